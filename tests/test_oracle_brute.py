"""Pins the CPU oracle to brute-force twins of the definitions (tests/brute.py)
on random tiny adversarial windows: quadratic scans and tick bitmaps."""
from fractions import Fraction

import numpy as np
import pytest

import brute
from runners import DEVICE_MASK, run_oracle
from tiny import random_window, schedule_window

SEEDS = list(range(12))


def _sorted_view(ev, r):
    return ev[r["perm"]]


@pytest.mark.parametrize("seed", SEEDS)
def test_load_and_canonical_order(seed):
    ev, off, t0, t1, sizes = random_window(seed)
    r = run_oracle(ev, off, t0, t1, min_gap=5, comm_sizes=sizes)
    win, dropped, summ = brute.load(ev, off, t0, t1)
    for w, s in enumerate(summ):
        for k, v in s.items():
            assert int(r["load_sum"][w][k]) == v
    perm = brute.canonical_perm(ev, win, dropped)
    assert r["perm"].tolist() == perm
    assert r["n_valid"] == int((~dropped).sum())
    sv = ev[perm]
    for k in ("ts_start", "ts_end", "corr_id", "pid", "name_id", "seq", "stream", "kind"):
        assert np.array_equal(r[k], sv[k])
    ll = brute.lanes(sv, win[perm], r["n_valid"])
    assert r["lane_off"].tolist() == [l[4] for l in ll] + [r["n_valid"]]
    assert r["lane_window"].tolist() == [l[0] for l in ll]
    assert r["lane_pid"].tolist() == [l[1] for l in ll]
    assert r["lane_domain"].tolist() == [l[2] for l in ll]
    assert r["lane_stream"].tolist() == [l[3] for l in ll]


@pytest.mark.parametrize("seed", SEEDS)
def test_join_against_quadratic_scan(seed):
    ev, off, t0, t1, sizes = random_window(seed)
    r = run_oracle(ev, off, t0, t1)
    sv = _sorted_view(ev, r)
    wins = np.searchsorted(np.asarray(off), r["perm"], side="right") - 1
    lo, lat, qd, kol = brute.join(sv, wins, r["n_valid"])
    assert r["launch_of"].tolist() == lo
    assert r["launch_latency"].tolist() == lat
    assert r["queue_delay"].tolist() == qd
    assert r["kernels_of_launch"].tolist() == kol
    # every probe is matched to exactly one launch or counted unmatched
    js = r["join_sum"]
    assert (js["n_matched"] + js["n_unmatched"] == js["n_probe"]).all()
    for w in range(len(t0)):
        sel = [i for i in range(r["n_valid"]) if wins[i] == w and sv[i]["kind"] in (3, 4)]
        assert js[w]["n_probe"] == len(sel)
        assert js[w]["n_matched"] == sum(1 for i in sel if lo[i] >= 0)
        assert js[w]["sum_latency"] == sum(lat[i] for i in sel)
        assert js[w]["sum_queue"] == sum(qd[i] for i in sel)
        m = [lat[i] for i in sel if lo[i] >= 0]
        assert js[w]["min_latency"] == (min(m) if m else 0)
        assert js[w]["max_latency"] == (max(m) if m else 0)
        launches = [i for i in range(r["n_valid"]) if wins[i] == w and sv[i]["kind"] == 2]
        assert js[w]["n_launch"] == len(launches)
        dup = 0
        orphan = 0
        for i in launches:
            first = min(j for j in launches if sv[j]["pid"] == sv[i]["pid"]
                        and sv[j]["corr_id"] == sv[i]["corr_id"])
            if first != i:
                dup += 1
            elif kol[i] == 0:
                orphan += 1
        assert js[w]["n_dup_launch"] == dup and js[w]["n_orphan_launch"] == orphan


@pytest.mark.parametrize("seed", SEEDS)
def test_attribution_against_quadratic_scan(seed):
    ev, off, t0, t1, sizes = random_window(seed)
    r = run_oracle(ev, off, t0, t1)
    sv = _sorted_view(ev, r)
    wins = np.searchsorted(np.asarray(off), r["perm"], side="right") - 1
    ll = brute.lanes(sv, wins, r["n_valid"])
    parent, depth, bad, n_enc, enc_of = brute.attribution(sv, wins, r["n_valid"], ll)
    assert not bad and r["attr_status"] in (0, 8)
    assert r["parent"].tolist() == parent
    assert r["depth"].tolist() == depth
    # what the depth is, said through the enclosure rule alone: every ancestor of a record
    # encloses it, and the enclosers the depth leaves out are exactly those that are no
    # ancestors (ranges that end at the very instant a zero-length record sits on)
    for i in range(r["n_valid"]):
        if sv[i]["kind"] > 2:
            continue
        chain, c = set(), int(r["parent"][i])
        while c >= 0:
            chain.add(c)
            c = int(r["parent"][c])
        assert chain <= set(enc_of[i])
        off_chain = set(enc_of[i]) - chain
        assert n_enc[i] - min(int(r["depth"][i]), n_enc[i]) == len(off_chain) or r["depth"][i] == 255
        for j in off_chain:
            assert sv[i]["ts_start"] == sv[i]["ts_end"] == sv[j]["ts_end"]
    # the forest level equals the number of enclosers for every record of non-zero length
    for i in range(r["n_valid"]):
        if sv[i]["kind"] <= 2 and sv[i]["ts_end"] > sv[i]["ts_start"]:
            assert depth[i] == min(n_enc[i], 255)
        assert depth[i] <= n_enc[i]
    assert (r["attr_status"] == 8) == (max(depth) > 8)
    # for properly nested lanes the parent is the nearest earlier OP that ends no earlier
    for (w, pid, dom, st, b, e) in ll:
        if dom:
            continue
        for i in range(b, e):
            near = -1
            for j in range(i - 1, b - 1, -1):
                if sv[j]["kind"] == 0 and sv[j]["ts_end"] >= sv[i]["ts_end"]:
                    near = j
                    break
            assert parent[i] == near
    # device records inherit the parent of their launch; per-OP sums are direct
    n = len(ev)
    op_of = [-1] * n
    for i in range(r["n_valid"]):
        if sv[i]["kind"] in (3, 4) and r["launch_of"][i] >= 0:
            op_of[i] = parent[r["launch_of"][i]]
    assert r["op_of"].tolist() == op_of
    for p in range(n):
        mem = [i for i in range(n) if op_of[i] == p]
        assert r["op_n_kernels"][p] == len(mem)
        if mem:
            assert r["op_first_start"][p] == min(int(sv[i]["ts_start"]) for i in mem)
            assert r["op_last_end"][p] == max(int(sv[i]["ts_end"]) for i in mem)
            assert r["op_kernel_ns"][p] == sum(int(sv[i]["ts_end"] - sv[i]["ts_start"]) for i in mem)
        else:
            assert r["op_first_start"][p] == r["op_last_end"][p] == r["op_kernel_ns"][p] == 0
    a = r["attr_sum"]
    assert (a["n_attributed"] + a["n_no_launch"] + a["n_no_op"] == r["join_sum"]["n_probe"]).all()
    assert r["op_n_kernels"].sum() == a["n_attributed"].sum()


@pytest.mark.parametrize("seed", SEEDS)
def test_bad_nesting_flag(seed):
    ev, off, t0, t1, sizes = random_window(100 + seed, nested=False, defects=False)
    r = run_oracle(ev, off, t0, t1)
    sv = _sorted_view(ev, r)
    wins = np.searchsorted(np.asarray(off), r["perm"], side="right") - 1
    ll = brute.lanes(sv, wins, r["n_valid"])
    parent, depth, bad, _, _ = brute.attribution(sv, wins, r["n_valid"], ll)
    assert (r["attr_status"] == 9) == bad
    assert bool(r["attr_sum"]["bad_nesting"].any()) == bad
    # the oracle evaluates the definition even then
    assert r["parent"].tolist() == parent and r["depth"].tolist() == depth


@pytest.mark.parametrize("seed", SEEDS)
def test_gaps_against_tick_bitmap(seed):
    ev, off, t0, t1, sizes = random_window(seed)
    min_gap = 7
    r = run_oracle(ev, off, t0, t1, min_gap=min_gap)
    sv = _sorted_view(ev, r)
    wins = np.searchsorted(np.asarray(off), r["perm"], side="right") - 1
    ll = brute.lanes(sv, wins, r["n_valid"])
    want_long = []
    win_hist = np.zeros((len(t0), 40), dtype=np.int64)
    for li, lane in enumerate(ll):
        lg = r["lane_gaps"][li]
        if lane[2] == 0:
            assert all(int(lg[k]) == 0 for k in lg.dtype.names)
            assert r["lane_hist"][li].sum() == 0
            continue
        W0, W1 = t0[lane[0]], t1[lane[0]]
        busy, idle, runs = brute.gaps_bitmap(sv, lane, W0, W1)
        assert lg["busy"] == busy and lg["idle"] == idle
        assert lg["busy"] + lg["idle"] == W1 - W0
        assert lg["n_gaps"] == len(runs)
        assert lg["max_gap"] == max([x[1] for x in runs], default=0)
        assert lg["n_events"] == lane[5] - lane[4]
        hist = np.zeros(40, dtype=np.int64)
        for (_, ln) in runs:
            hist[brute.log2_bin(ln)] += 1
        assert r["lane_hist"][li].tolist() == hist.tolist()
        assert r["lane_hist"][li].sum() == lg["n_gaps"]
        win_hist[lane[0]] += hist
        # each idle run ends where a record starts (or at the window end)
        for (st, ln) in runs:
            if ln >= min_gap:
                end = st + ln
                nxt = -1
                if end < W1:
                    nxt = min(i for i in range(lane[4], lane[5]) if sv[i]["ts_start"] == end)
                want_long.append((li, nxt, st, ln))
        # gap_before of a record = length of the idle run that ends at its start, for the first
        # record (in canonical order) that starts there
        ends = {st + ln: ln for (st, ln) in runs}
        seen = set()
        for i in range(lane[4], lane[5]):
            s = int(sv[i]["ts_start"])
            g = ends.get(s, 0) if s not in seen else 0
            seen.add(s)
            assert r["gap_before"][i] == g
    assert r["win_hist"].tolist() == win_hist.tolist()
    got = [(int(x["lane"]), int(x["next_event"]), int(x["gap_start"]), int(x["gap_len"]))
           for x in r["long_gaps"]]
    assert got == want_long


@pytest.mark.parametrize("seed", SEEDS)
def test_aggregates_against_dict(seed):
    ev, off, t0, t1, sizes = random_window(seed)
    masks = (DEVICE_MASK, 1 << 2, 0b111111)
    r = run_oracle(ev, off, t0, t1, agg_masks=masks)
    sv = _sorted_view(ev, r)
    wins = np.searchsorted(np.asarray(off), r["perm"], side="right") - 1
    n = len(ev)
    dur = [int(sv[p]["ts_end"]) - int(sv[p]["ts_start"]) for p in range(n)]
    top = [int(r["op_last_end"][p] - r["op_first_start"][p]) if r["op_n_kernels"][p] > 0 else None
           for p in range(n)]
    cases = [(f"agg{i}_", m, dur) for i, m in enumerate(masks)] + [("aggT_", 1, top)]
    for pref, mask, vals in cases:
        rows = brute.aggregate(sv, wins, r["n_valid"], mask, vals)
        assert len(rows) == len(r[pref + "g_count"])
        for i, (key, row) in enumerate(rows):
            assert (int(r[pref + "g_window"][i]), int(r[pref + "g_pid"][i]),
                    int(r[pref + "g_name"][i])) == key
            assert int(r[pref + "g_count"][i]) == row["count"]
            assert int(r[pref + "g_sum"][i]) == row["sum"]
            assert int(r[pref + "g_min"][i]) == row["min"]
            assert int(r[pref + "g_max"][i]) == row["max"]
            assert r[pref + "g_hist"][i].tolist() == row["hist"]
            assert r[pref + "g_hist"][i].sum() == row["count"]
        pop = sum(1 for p in range(r["n_valid"])
                  if ((1 << int(sv[p]["kind"])) & mask) and vals[p] is not None)
        assert int(r[pref + "g_count"].sum()) == pop


def test_log2_bins_bracket_values():
    from helpers import make_events
    vals = [0, 1, 2, 3, 4, 7, 8, 1023, 1024, 2**38, 2**39 - 1, 2**39, 2**45]
    ev = make_events([("KERNEL", 1, 0, 10, 10 + v, 0, i, 0) for i, v in enumerate(vals)])
    r = run_oracle(ev, [0, len(ev)], [0], [100], agg_masks=(1 << 3,))
    for i, v in enumerate(vals):
        b = int(np.nonzero(r["agg0_g_hist"][i])[0][0])
        if v <= 1:
            assert b == 0
        elif b < 39:
            assert 2**b <= v < 2**(b + 1)
        else:
            assert v >= 2**39


@pytest.mark.parametrize("seed", SEEDS)
def test_collectives_against_dict(seed):
    ev, off, t0, t1, sizes = random_window(seed)
    r = run_oracle(ev, off, t0, t1, comm_sizes=sizes)
    sv = _sorted_view(ev, r)
    wins = np.searchsorted(np.asarray(off), r["perm"], side="right") - 1
    groups, wait, ranks = brute.collectives(sv, wins, r["n_valid"], sizes)
    assert len(groups) == len(r["c_seq"])
    for i, (key, g) in enumerate(groups):
        assert (int(r["c_window"][i]), int(r["c_comm"][i]), int(r["c_seq"][i])) == key
        assert (int(r["c_n_members"][i]), int(r["c_min_start"][i]), int(r["c_max_start"][i]),
                int(r["c_skew"][i]), int(r["c_max_end"][i]), int(r["c_straggler_pid"][i]),
                int(r["c_flags"][i])) == (g["n"], g["min_start"], g["max_start"], g["skew"],
                                          g["max_end"], g["straggler"], g["flags"])
    want = np.zeros(len(ev), dtype=np.int64)
    for p, v in wait.items():
        want[p] = v
    assert r["wait_ns"].tolist() == want.tolist()
    assert len(ranks) == len(r["r_pid"])
    for i, (key, row) in enumerate(ranks):
        assert (int(r["r_window"][i]), int(r["r_pid"][i])) == key
        assert [int(r["r_n_coll"][i]), int(r["r_sum_wait"][i]), int(r["r_max_wait"][i]),
                int(r["r_n_straggler"][i])] == row
    # in every unflagged group somebody waits 0 and somebody waits the whole skew
    for i, (key, g) in enumerate(groups):
        if g["flags"] == 0:
            ws = [wait[p] for p in range(r["n_valid"]) if sv[p]["kind"] == 5
                  and (int(wins[p]), int(sv[p]["corr_id"]), int(sv[p]["seq"])) == key]
            assert min(ws) == 0 and max(ws) == g["skew"]


@pytest.mark.parametrize("seed", SEEDS)
def test_device_overlap_against_tick_bitmaps(seed):
    ev, off, t0, t1, sizes = random_window(seed)
    r = run_oracle(ev, off, t0, t1, min_gap=5, comm_sizes=sizes)
    sv = _sorted_view(ev, r)
    wins = np.searchsorted(np.asarray(off), r["perm"], side="right") - 1
    rows = brute.device_overlap(sv, wins, r["n_valid"], t0, t1)
    got = {(int(w), int(p)): tuple(int(r[k][i]) for k in ("d_n_events", "d_busy", "d_idle", "d_compute",
                                                          "d_comm", "d_overlap", "d_exposed"))
           for i, (w, p) in enumerate(zip(r["d_window"], r["d_pid"]))}
    assert got == rows
    assert list(got) == sorted(got)  # rows come in (window, pid) order
    assert len(rows) > 0


@pytest.mark.parametrize("seed", SEEDS)
def test_gap_blame_against_ticks(seed):
    ev, off, t0, t1, sizes = random_window(seed)
    r = run_oracle(ev, off, t0, t1, min_gap=5, comm_sizes=sizes)
    sv = _sorted_view(ev, r)
    wins = np.searchsorted(np.asarray(off), r["perm"], side="right") - 1
    ll = brute.lanes(sv, wins, r["n_valid"])
    cls, op_gap = brute.blame(sv, wins, r["n_valid"], ll, r["long_gaps"], r["launch_of"], t0, t1)
    assert r["b_class"].tolist() == cls
    assert np.array_equal(r["op_gap_ns"], op_gap)
    assert len(cls) > 0 and len(set(cls)) >= 2
    cnt = np.zeros((len(t0), 4), dtype=np.int64)
    ns = np.zeros((len(t0), 4), dtype=np.int64)
    for g, c in zip(r["long_gaps"], cls):
        w = ll[int(g["lane"])][0]
        cnt[w, c] += 1
        ns[w, c] += int(g["gap_len"])
    assert np.array_equal(r["b_win_count"], cnt) and np.array_equal(r["b_win_ns"], ns)
    # the per-name table is the plain aggregate of the per-operator figures
    rows = brute.aggregate(sv, wins, r["n_valid"], 1, [int(v) if v > 0 else None for v in op_gap])
    assert len(rows) == len(r["aggG_g_count"])
    for i, (key, row) in enumerate(rows):
        assert (int(r["aggG_g_window"][i]), int(r["aggG_g_pid"][i]), int(r["aggG_g_name"][i])) == key
        assert int(r["aggG_g_count"][i]) == row["count"] and int(r["aggG_g_sum"][i]) == row["sum"]
        assert int(r["aggG_g_min"][i]) == row["min"] and int(r["aggG_g_max"][i]) == row["max"]


@pytest.mark.parametrize("seed", SEEDS)
def test_rollup_against_parent_chains(seed):
    ev, off, t0, t1, sizes = random_window(seed)
    r = run_oracle(ev, off, t0, t1, min_gap=5, comm_sizes=sizes)
    if r["attr_status"] != 0:
        pytest.skip("window with a nesting error: no roll-up")
    sv = _sorted_view(ev, r)
    wins = np.searchsorted(np.asarray(off), r["perm"], side="right") - 1
    n, first, last, ns, replays = brute.rollup(sv, r["n_valid"], r["parent"], r["op_n_kernels"],
                                               r["op_first_start"], r["op_last_end"], r["op_kernel_ns"],
                                               r["launch_of"], r["kernels_of_launch"])
    assert np.array_equal(r["incl_n_kernels"], n) and np.array_equal(r["incl_kernel_ns"], ns)
    assert np.array_equal(r["incl_first_start"], first) and np.array_equal(r["incl_last_end"], last)
    want = np.zeros((3, len(sv)), dtype=np.int64)
    for l, (a, b, c) in replays.items():
        want[:, l] = (a, b, c)
    assert np.array_equal(r["replay_first_start"], want[0]) and np.array_equal(r["replay_last_end"], want[1])
    assert np.array_equal(r["replay_kernel_ns"], want[2])
    summ = np.zeros((len(t0), 3), dtype=np.int64)
    for l in replays:
        w = wins[l]
        k = int(r["kernels_of_launch"][l])
        summ[w] = (summ[w][0] + 1, summ[w][1] + k, max(summ[w][2], k))
    assert np.array_equal(r["roll_sum"], summ)
    # roots of the forest hold everything that was attributed below them
    roots = (sv["kind"][:r["n_valid"]] == 0) & (r["parent"][:r["n_valid"]] < 0)
    assert int(r["incl_n_kernels"][:r["n_valid"]][roots].sum()) == int(r["attr_sum"]["n_attributed"].sum())


def _critical_path_matches_brute(ev, off, t0, t1, sizes=()):
    r = run_oracle(ev, off, t0, t1, min_gap=5, comm_sizes=sizes)
    sv = _sorted_view(ev, r)
    wins = np.searchsorted(np.asarray(off), r["perm"], side="right") - 1
    want = brute.critical_path(sv, wins, r["n_valid"], r["launch_of"])
    keys = list(zip(r["cp_window"].tolist(), r["cp_pid"].tolist()))
    assert keys == list(want)
    on = np.zeros(len(sv), dtype=np.uint8)
    tot = np.zeros((len(t0), 10), dtype=np.int64)
    for i, key in enumerate(keys):
        b = want[key]
        assert int(r["cp_sink"][i]) == b["sink"] and int(r["cp_reason"][i]) == b["reason"]
        assert int(r["cp_begin"][i]) == b["begin"] and int(r["cp_end"][i]) == b["end"]
        assert int(r["cp_n_nodes"][i]) == len(b["nodes"])
        assert r["cp_ns"].reshape(-1, 8)[i].tolist() == b["ns"]
        assert sum(b["ns"]) == b["end"] - b["begin"]  # the classes telescope
        on[list(b["nodes"])] = 1
        tot[key[0], 0] += 1
        tot[key[0], 1] += len(b["nodes"])
        tot[key[0], 2:] += b["ns"]
    assert np.array_equal(r["on_path"], on)
    assert np.array_equal(r["cp_sum"].reshape(-1, 10), tot)
    # the per-symbol table of the records on a path is the plain aggregate of their durations
    rows = brute.aggregate(sv, wins, r["n_valid"], 62,
                           [int(sv[p]["ts_end"]) - int(sv[p]["ts_start"]) if on[p] else None
                            for p in range(len(sv))])
    assert len(rows) == len(r["aggP_g_count"])
    for i, (key, row) in enumerate(rows):
        assert (int(r["aggP_g_window"][i]), int(r["aggP_g_pid"][i]), int(r["aggP_g_name"][i])) == key
        assert int(r["aggP_g_count"][i]) == row["count"] and int(r["aggP_g_sum"][i]) == row["sum"]
        assert int(r["aggP_g_min"][i]) == row["min"] and int(r["aggP_g_max"][i]) == row["max"]
        assert r["aggP_g_hist"][i].tolist() == row["hist"]
    assert int(r["aggP_g_count"].sum()) == int(on.sum())
    return r, want


@pytest.mark.parametrize("seed", SEEDS)
def test_critical_path_against_point_walk_random(seed):
    ev, off, t0, t1, sizes = random_window(seed)
    _critical_path_matches_brute(ev, off, t0, t1, sizes)


@pytest.mark.parametrize("seed", SEEDS)
def test_critical_path_against_point_walk_schedules(seed):
    ev, off, t0, t1, _ = schedule_window(seed)
    r, want = _critical_path_matches_brute(ev, off, t0, t1)
    ns = r["cp_ns"].reshape(-1, 8).sum(0)
    assert ns[7] > 0 and ns[3] > 0 and ns[6] > 0  # waits, submission edges and host time all occur


@pytest.mark.parametrize("seed", SEEDS)
def test_critical_path_of_a_tight_schedule_is_the_longest_path(seed):
    """In a schedule without slack (a kernel starts the moment its launch call starts or its
    stream frees up, a wait returns a fixed time after the last kernel) the chain of binding
    dependencies is a longest path of the full dependency graph: it reaches the first call of the
    thread, spans the makespan, and holds neither launch latency nor stream delay."""
    ev, off, t0, t1, info = schedule_window(seed, tight=True)
    r = run_oracle(ev, off, t0, t1)
    for i, pid in enumerate(r["cp_pid"].tolist()):
        g = info[pid]
        # longest path over ALL dependencies: relax every edge until nothing changes
        dist = {g["source"]: 0}
        changed = True
        while changed:
            changed = False
            for a, b, w in g["edges"]:
                if a in dist and dist[a] + w > dist.get(b, -1):
                    dist[b] = dist[a] + w
                    changed = True
        longest = max(dist.values())
        assert longest == g["makespan"]
        ns = r["cp_ns"].reshape(-1, 8)[i]
        assert int(r["cp_reason"][i]) == 0 and int(r["cp_begin"][i]) == g["first"]
        assert int(r["cp_end"][i]) - int(r["cp_begin"][i]) == longest == int(ns.sum())
        assert ns[3] == 0 and ns[4] == 0


@pytest.mark.parametrize("seed", SEEDS[:6])
def test_operator_sol_against_exact_rationals(seed):
    """The efficiency step against the definition evaluated in exact rational arithmetic: each
    double must lie within a few units in the last place of the exact quotient (two roundings
    in the denominator, one in the division); plus the identities the definition implies."""
    ev, off, t0, t1, sizes = random_window(seed)
    rng = np.random.default_rng(seed)
    flops = rng.integers(0, 10**12, size=len(ev)).astype(np.float64)
    nbytes = rng.integers(0, 10**9, size=len(ev)).astype(np.float64)
    flops[rng.random(len(ev)) < 0.1] = -1.0
    nbytes[rng.random(len(ev)) < 0.05] = np.nan
    pf, pb = 2.25e15, 7.7e12
    r = run_oracle(ev, off, t0, t1, op_work=(flops, nbytes, pf, pb))
    if r["attr_status"] != 0:
        pytest.skip("window without a legal operator nesting")
    nv = r["n_valid"]
    state, mfu, mbu, sol = brute.operator_sol(r["kind"][:nv], r["perm"], r["op_n_kernels"],
                                              r["op_first_start"], r["op_last_end"], flops, nbytes, pf, pb)
    assert r["sol_state"][:nv].tolist() == state and not r["sol_state"][nv:].any()
    for got, want in ((r["sol_mfu"], mfu), (r["sol_mbu"], mbu), (r["sol_op"], sol)):
        for p in range(nv):
            assert abs(Fraction(float(got[p])) - want[p]) <= abs(want[p]) * Fraction(4, 2**53), p
    res = r["sol_state"] == 1
    assert (r["sol_op"] >= r["sol_mfu"]).all() and (r["sol_op"] >= r["sol_mbu"]).all()
    assert ((r["sol_op"] == r["sol_mfu"]) | (r["sol_op"] == r["sol_mbu"])).all()
    assert not r["sol_op"][~res].any() and not r["sol_mfu"][~res].any()
    wins = np.searchsorted(np.asarray(off), r["perm"], side="right") - 1
    for w in range(len(t0)):
        s = r["sol_sum"][w]
        m = res & (wins == w)
        assert (s["n_resolved"], s["n_no_kernels"], s["n_no_counts"]) == \
            (int(m.sum()), int(((r["sol_state"] == 2) & (wins == w)).sum()),
             int(((r["sol_state"] == 3) & (wins == w)).sum()))
        top = (r["op_last_end"] - r["op_first_start"])[m]
        assert s["sum_top_ns"] == int(top.sum())
        assert s["max_sol"] == (r["sol_op"][m].max() if m.any() else 0.0)
        assert np.isclose(s["sum_flops"], flops[r["perm"][m]].sum(), rtol=1e-12)
        assert np.isclose(s["sum_bytes"], nbytes[r["perm"][m]].sum(), rtol=1e-12)
    # scaling laws that hold exactly in binary floating point: twice the work doubles the
    # utilisation, twice the peak halves it
    r2 = run_oracle(ev, off, t0, t1, op_work=(flops * 2, nbytes * 2, pf, pb * 2))
    assert np.array_equal(r2["sol_mfu"], r["sol_mfu"] * 2) and np.array_equal(r2["sol_mbu"], r["sol_mbu"])
