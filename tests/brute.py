"""Brute-force twins of the analyzer's definitions, in plain Python.

Written independently of both analyzers, straight from the definitions in
include/ta.h, with quadratic scans and tick bitmaps.  Only for tiny windows.
"""
import numpy as np


def log2_bin(v):
    if v <= 1:
        return 0
    return min(39, int(v).bit_length() - 1)


def load(ev, win_off, t0, t1):
    n = len(ev)
    W = len(t0)
    win = np.zeros(n, dtype=np.int64)
    dropped = np.zeros(n, dtype=bool)
    summ = [dict(n_events=0, n_valid=0, n_bad_kind=0, n_bad_interval=0, n_out_of_window=0)
            for _ in range(W)]
    for w in range(W):
        for k in range(win_off[w], win_off[w + 1]):
            win[k] = w
            s = summ[w]
            s["n_events"] += 1
            e = ev[k]
            if not (0 <= e["kind"] <= 5):
                dropped[k] = True
                s["n_bad_kind"] += 1
            elif e["ts_end"] < e["ts_start"]:
                dropped[k] = True
                s["n_bad_interval"] += 1
            elif e["ts_start"] < t0[w] or e["ts_start"] >= t1[w]:
                dropped[k] = True
                s["n_out_of_window"] += 1
            else:
                s["n_valid"] += 1
    return win, dropped, summ


def canonical_perm(ev, win, dropped):
    def key(k):
        e = ev[k]
        return (bool(dropped[k]), int(win[k]), int(e["pid"]), 1 if e["kind"] >= 3 else 0,
                int(e["stream"]), int(e["ts_start"]), -int(e["ts_end"]), k)
    return sorted(range(len(ev)), key=key)


def lanes(sv, wins, n_valid):
    """sv: records in sorted order; returns list of (window, pid, domain, stream, begin, end)."""
    out = []
    for p in range(n_valid):
        k = (int(wins[p]), int(sv[p]["pid"]), 1 if sv[p]["kind"] >= 3 else 0, int(sv[p]["stream"]))
        if not out or out[-1][:4] != k:
            if out:
                out[-1] = out[-1][:5] + (p,)
            out.append(k + (p, None))
    if out:
        out[-1] = out[-1][:5] + (n_valid,)
    return out


def join(sv, wins, n_valid):
    n = len(sv)
    launch_of = [-1] * n
    lat = [0] * n
    qd = [0] * n
    kol = [0] * n
    for i in range(n_valid):
        if sv[i]["kind"] not in (3, 4):
            continue
        for l in range(n_valid):
            if (sv[l]["kind"] == 2 and wins[l] == wins[i] and sv[l]["pid"] == sv[i]["pid"]
                    and sv[l]["corr_id"] == sv[i]["corr_id"]):
                launch_of[i] = l
                lat[i] = int(sv[i]["ts_start"]) - int(sv[l]["ts_start"])
                qd[i] = max(0, int(sv[i]["ts_start"]) - int(sv[l]["ts_end"]))
                kol[l] += 1
                break
    return launch_of, lat, qd, kol


def attribution(sv, wins, n_valid, lane_list):
    """O(n^2) scan of the enclosure definition.  Returns parent, depth, bad_nesting, the
    number of enclosers and the enclosers themselves."""
    n = len(sv)
    parent = [-1] * n
    depth = [0] * n
    n_enc = [0] * n
    enc_of = [()] * n
    bad = False
    for (w, pid, dom, st, b, e) in lane_list:
        if dom != 0:
            continue
        for i in range(b, e):
            si, ei = int(sv[i]["ts_start"]), int(sv[i]["ts_end"])
            enc = []
            for j in range(b, e):
                if j == i or sv[j]["kind"] != 0:
                    continue
                sj, ej = int(sv[j]["ts_start"]), int(sv[j]["ts_end"])
                if sj < si < ej < ei:
                    bad = True
                if sj <= si and ei <= ej and ((sj, ej) != (si, ei) or j < i):
                    enc.append(j)
            n_enc[i] = len(enc)
            enc_of[i] = tuple(enc)
            if enc:
                parent[i] = max(enc, key=lambda j: (int(sv[j]["ts_start"]), -int(sv[j]["ts_end"]), j))
    # depth = level in the forest the parents define
    for i in range(n):
        d, c = 0, parent[i]
        while c >= 0:
            d += 1
            c = parent[c]
        depth[i] = min(d, 255)
    return parent, depth, bad, n_enc, enc_of


def gaps_bitmap(sv, lane, W0, W1):
    """Marks every tick of [W0, W1) covered by a record of the lane; returns busy, idle,
    list of (start, len) of idle runs.  A zero-length record covers no tick but is still an
    observation of the stream, so an idle run is cut at the start time of such a record."""
    (_, _, _, _, b, e) = lane
    cov = np.zeros(W1 - W0, dtype=bool)
    for i in range(b, e):
        s, t = int(sv[i]["ts_start"]), min(int(sv[i]["ts_end"]), W1)
        if t > s:
            cov[s - W0:t - W0] = True
    busy = int(cov.sum())
    runs = []
    t = 0
    L = len(cov)
    while t < L:
        if not cov[t]:
            u = t
            while u < L and not cov[u]:
                u += 1
            cuts = sorted({int(sv[i]["ts_start"]) - W0 for i in range(b, e)
                           if t < int(sv[i]["ts_start"]) - W0 < u})
            a = t
            for c in cuts + [u]:
                runs.append((W0 + a, c - a))
                a = c
            t = u
        else:
            t += 1
    return busy, L - busy, runs


def aggregate(sv, wins, n_valid, kind_mask, values):
    """values: per sorted position value or None (not in the population)."""
    rows = {}
    for p in range(n_valid):
        if not ((1 << int(sv[p]["kind"])) & kind_mask) or values[p] is None:
            continue
        key = (int(wins[p]), int(sv[p]["pid"]), int(sv[p]["name_id"]))
        v = int(values[p])
        r = rows.setdefault(key, dict(count=0, sum=0, min=v, max=v, hist=[0] * 40))
        r["count"] += 1
        r["sum"] += v
        r["min"] = min(r["min"], v)
        r["max"] = max(r["max"], v)
        r["hist"][log2_bin(v)] += 1
    return [(k, rows[k]) for k in sorted(rows)]


def collectives(sv, wins, n_valid, sizes):
    exp = dict(sizes)
    groups = {}
    for p in range(n_valid):
        if sv[p]["kind"] == 5:
            groups.setdefault((int(wins[p]), int(sv[p]["corr_id"]), int(sv[p]["seq"])), []).append(p)
    out = []
    wait = {}
    ranks = {}
    for key in sorted(groups):
        m = groups[key]
        starts = [int(sv[p]["ts_start"]) for p in m]
        mx = max(starts)
        strag = min(int(sv[p]["pid"]) for p in m if int(sv[p]["ts_start"]) == mx)
        flags = 0
        if key[1] in exp:
            if len(m) != exp[key[1]]:
                flags |= 1
        elif len(m) < 2:
            flags |= 1
        pids = [int(sv[p]["pid"]) for p in m]
        if len(set(pids)) != len(pids):
            flags |= 2
        for p in m:
            wait[p] = mx - int(sv[p]["ts_start"])
            r = ranks.setdefault((key[0], int(sv[p]["pid"])), [0, 0, 0, 0])
            if flags == 0:
                r[0] += 1
                r[1] += wait[p]
                r[2] = max(r[2], wait[p])
        if flags == 0:
            ranks[(key[0], strag)][3] += 1
        out.append((key, dict(n=len(m), min_start=min(starts), max_start=mx, skew=mx - min(starts),
                              max_end=max(int(sv[p]["ts_end"]) for p in m), straggler=strag,
                              flags=flags)))
    return out, wait, [(k, ranks[k]) for k in sorted(ranks)]


def device_overlap(sv, wins, n_valid, t0, t1):
    """Per (window, pid): marks every tick of the window covered by a KERNEL record and every
    tick covered by a MEMCPY or COLL record; returns {(w, pid): (n, busy, idle, compute, comm,
    overlap, exposed)} counted tick by tick."""
    rows = {}
    for p in range(n_valid):
        k = int(sv[p]["kind"])
        if k < 3:
            continue
        w = int(wins[p])
        key = (w, int(sv[p]["pid"]))
        L = int(t1[w] - t0[w])
        if key not in rows:
            rows[key] = [0, np.zeros(L, dtype=bool), np.zeros(L, dtype=bool)]
        rows[key][0] += 1
        s, e = int(sv[p]["ts_start"]) - int(t0[w]), min(int(sv[p]["ts_end"]), int(t1[w])) - int(t0[w])
        if e > s:
            rows[key][1 if k == 3 else 2][s:e] = True
    out = {}
    for key, (cnt, comp, comm) in rows.items():
        busy = int((comp | comm).sum())
        both = int((comp & comm).sum())
        out[key] = (cnt, busy, len(comp) - busy, int(comp.sum()), int(comm.sum()), both,
                    int(comm.sum()) - both)
    return out


def blame(sv, wins, n_valid, lane_list, long_gaps, launch_of, t0, t1):
    """Classes of the long gaps (3 tail, 0 no launch, 1 submission, 2 queued) and, tick by tick,
    how many device streams of the operator's (window, pid) sit in a long gap while it runs."""
    cls = []
    for g in long_gaps:
        nxt = int(g["next_event"])
        if nxt < 0:
            cls.append(3)
        elif int(launch_of[nxt]) < 0:
            cls.append(0)
        else:
            cls.append(1 if int(sv[int(launch_of[nxt])]["ts_start"]) >= int(g["gap_start"]) else 2)
    idle = {}
    for g in long_gaps:
        w, pid = lane_list[int(g["lane"])][0], lane_list[int(g["lane"])][1]
        arr = idle.setdefault((w, pid), np.zeros(int(t1[w] - t0[w]), dtype=np.int64))
        a = int(g["gap_start"]) - int(t0[w])
        arr[a:a + int(g["gap_len"])] += 1
    op_gap = np.zeros(len(sv), dtype=np.int64)
    for p in range(n_valid):
        if int(sv[p]["kind"]) != 0:
            continue
        w = int(wins[p])
        arr = idle.get((w, int(sv[p]["pid"])))
        if arr is None:
            continue
        a = max(int(sv[p]["ts_start"]) - int(t0[w]), 0)
        b = min(int(sv[p]["ts_end"]) - int(t0[w]), len(arr))
        if b > a:
            op_gap[p] = int(arr[a:b].sum())
    return cls, op_gap


def rollup(sv, n_valid, parent, op_n, op_first, op_last, op_ns, launch_of, kol):
    """Inclusive figures: every OP that owns kernels is added to itself and to each OP on its
    parent chain.  Replays: the probes of every launch that owns two or more, collected in a
    dict.  Returns (incl_n, incl_first, incl_last, incl_ns, replays{launch: (first, last, ns)})."""
    n = len(sv)
    acc = {}
    for p in range(n_valid):
        if int(sv[p]["kind"]) != 0 or int(op_n[p]) <= 0:
            continue
        q = p
        hops = 0
        while q >= 0:
            a = acc.setdefault(q, [0, None, None, 0])
            a[0] += int(op_n[p])
            a[3] += int(op_ns[p])
            a[1] = int(op_first[p]) if a[1] is None else min(a[1], int(op_first[p]))
            a[2] = int(op_last[p]) if a[2] is None else max(a[2], int(op_last[p]))
            q = int(parent[q])
            hops += 1
            assert hops < 1000
    incl = [np.zeros(n, dtype=np.int64) for _ in range(4)]
    for q, a in acc.items():
        incl[0][q], incl[1][q], incl[2][q], incl[3][q] = a[0], a[1], a[2], a[3]
    replays = {}
    for p in range(n_valid):
        if int(sv[p]["kind"]) not in (3, 4):
            continue
        l = int(launch_of[p])
        if l < 0 or int(kol[l]) < 2:
            continue
        s, e = int(sv[p]["ts_start"]), int(sv[p]["ts_end"])
        r = replays.setdefault(l, [s, e, 0])
        r[0], r[1], r[2] = min(r[0], s), max(r[1], e), r[2] + (e - s)
    return incl[0], incl[1], incl[2], incl[3], replays


def critical_path(sv, wins, n_valid, launch_of):
    """The backward walk over START / END points, with every predecessor found by scanning all
    records for the one the definition names.  Returns {(window, pid): dict(sink, begin, end,
    reason, nodes (set of positions), ns (eight classes))}."""
    def slot(p):
        return (int(wins[p]), int(sv[p]["pid"]))

    def lane(p):
        return slot(p) + (1 if sv[p]["kind"] >= 3 else 0, int(sv[p]["stream"]))

    S = lambda p: int(sv[p]["ts_start"])
    E = lambda p: int(sv[p]["ts_end"])
    K = lambda p: int(sv[p]["kind"])
    out = {}
    for key in sorted({slot(p) for p in range(n_valid) if K(p) != 0}):
        mine = [p for p in range(n_valid) if K(p) != 0 and slot(p) == key]
        sink = max(mine, key=lambda p: (E(p), p))
        point = ("END", sink)
        ns = [0] * 8
        seen = set()
        reason = begin = None
        for _ in range(4 * n_valid + 4):
            what, v = point
            seen.add(v)
            if what == "END":
                if K(v) == 1:
                    cands = [d for d in mine if K(d) >= 3 and E(d) < E(v)]
                    if cands:
                        d = max(cands, key=lambda d: (E(d), d))
                        if E(d) >= S(v):
                            ns[7] += E(v) - E(d)
                            point = ("END", d)
                            continue
                ns[K(v) - 3 if K(v) >= 3 else 5] += E(v) - S(v)
                point = ("START", v)
            elif K(v) >= 3:
                before = [q for q in range(v) if lane(q) == lane(v)]
                q = before[-1] if before and E(before[-1]) <= S(v) else None
                l = int(launch_of[v]) if K(v) in (3, 4) else -1
                if l < 0 or S(l) > S(v):
                    l = None
                if q is not None and (l is None or E(q) > S(l)):
                    ns[4] += S(v) - E(q)
                    point = ("END", q)
                elif l is not None:
                    ns[3] += S(v) - S(l)
                    point = ("START", l)
                else:
                    reason, begin = 1, S(v)
                    break
            else:
                before = [u for u in range(v) if lane(u) == lane(v) and K(u) in (1, 2)]
                if not before:
                    reason, begin = 0, S(v)
                    break
                u = before[-1]
                if E(u) <= S(v):
                    ns[6] += S(v) - E(u)
                    point = ("END", u)
                else:
                    ns[5] += S(v) - S(u)
                    point = ("START", u)
        assert reason is not None, "the walk did not end"
        out[key] = dict(sink=sink, begin=begin, end=E(sink), reason=reason, nodes=seen, ns=ns)
    return out


def operator_sol(kind, perm, op_n, op_first, op_last, flops, nbytes, peak_flops, peak_bw):
    """MFU, MBU and SOL_op of every OP record as EXACT rationals (fractions.Fraction), from the
    definition: count / (T_op seconds x peak).  Returns (state, mfu, mbu, sol) lists."""
    from fractions import Fraction
    n = len(kind)
    state = [0] * n
    mfu = [Fraction(0)] * n
    mbu = [Fraction(0)] * n
    sol = [Fraction(0)] * n
    for p in range(n):
        if kind[p] != 0:
            continue
        top = int(op_last[p]) - int(op_first[p])
        if op_n[p] <= 0 or top <= 0:
            state[p] = 2
            continue
        f, b = float(flops[perm[p]]), float(nbytes[perm[p]])
        if not (f >= 0) or not (b >= 0):
            state[p] = 3
            continue
        seconds = Fraction(top, 10**9)
        mfu[p] = Fraction(f) / (seconds * Fraction(peak_flops))
        mbu[p] = Fraction(b) / (seconds * Fraction(peak_bw))
        sol[p] = max(mfu[p], mbu[p])
        state[p] = 1
    return state, mfu, mbu, sol
