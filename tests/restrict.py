"""Full-size parity by sub-problem.

The analysis decomposes: a record only ever interacts with records of its own
(window, pid) - except collectives, whose groups span the pids of one window.
So the result of the whole analysis, restricted to the records of a subset that is
closed under those interactions, must equal the analysis of the subset alone
(positions renumbered).  `run_gpu_restricted` runs the CUDA library once on the
full input, keeps the results on the device, and for each requested subset builds
that restricted, renumbered view with torch indexing; only the views travel to the
host, where they are compared with the oracle run on the subset.
"""
import numpy as np

from paper_2609_40247_b200.ta import NBINS
from runners import (AGG_KEYS, ATTR_KEYS, BLAME_KEYS, COLL_KEYS, CRITPATH_KEYS, DEVICE_MASK, GAP_KEYS,
                     JOIN_KEYS, OP_MASK, OVERLAP_KEYS, ROLLUP_KEYS)

_POSITIONAL = {"launch_of", "parent", "op_of"}  # values are sorted positions (or -1)
_PER_RECORD_SORT = ["ts_start", "ts_end", "corr_id", "pid", "name_id", "seq", "stream", "kind"]
_LANE_COLS = ["lane_window", "lane_pid", "lane_stream", "lane_domain"]


class Subset:
    """sel: bool mask over the input records; windows: kept window indices (None = all);
    pid: restrict aggregate rows to this pid (None = all); groups: which result groups
    are meaningful for the subset (any of "sort", "join", "attr", "gaps", "agg", "coll",
    "overlap")."""

    def __init__(self, name, sel, groups, windows=None, pid=None):
        self.name, self.sel, self.groups, self.windows, self.pid = name, sel, groups, windows, pid


def _typed(res, name):
    import torch
    dt, cnt = res._spec(res._names.get(name, name) if hasattr(res, "_names") else name)
    t = res.tensor(name)
    if dt.names:  # struct array: rows of bytes
        return t.view(torch.uint8).reshape(cnt, dt.itemsize), dt
    tdt = {"<i4": torch.int32, "<i8": torch.int64, "<i2": torch.int16, "|u1": torch.uint8,
           "<u4": torch.int32}[dt.str]
    return (t.view(tdt) if cnt else torch.empty(0, dtype=tdt, device=t.device)), dt


def _host(t, dt):
    a = t.contiguous().cpu().numpy()
    if dt.names:
        return a.reshape(-1).view(dt).copy()
    return a.view(dt).copy()


def run_gpu_restricted(events, win_off, t0, t1, subsets, min_gap=500_000, comm_sizes=(),
                       checks=None):
    """Returns {subset.name: result dict in the subset's own coordinates}.  `checks(full)`,
    if given, is called with the device-side results (dict of result objects) so that
    whole-window properties can be tested without copying per-record arrays."""
    import torch
    from paper_2609_40247_b200 import ta
    W = len(win_off) - 1
    buf = torch.from_numpy(np.ascontiguousarray(events).view(np.uint8).reshape(-1)).cuda()
    out = {}
    with ta.Window(buf, win_off, t0, t1) as w:
        s = w.sort_timeline()
        j = w.correlate_launches()
        a = w.attribute_operators(check=False)
        g = w.stream_gaps(min_gap)
        ag_dev = w.aggregate_ops(DEVICE_MASK, 0)
        ag_op = w.aggregate_ops(OP_MASK, 1) if a.status == 0 else None
        c = w.match_collectives(comm_sizes)
        ov = w.device_overlap()
        ru = w.rollup_operators() if a.status == 0 else None
        bl = w.blame_gaps(g)
        ag_gap = w.aggregate_ops(OP_MASK, 2)
        cp = w.critical_path()
        ag_path = w.aggregate_ops(62, 3)
        del buf
        if checks is not None:
            checks(dict(window=w, sort=s, join=j, attr=a, gaps=g, agg_dev=ag_dev, agg_op=ag_op,
                        coll=c, overlap=ov, blame=bl, critpath=cp))
        n, n_valid = s.n, s.n_valid
        perm = _typed(s, "perm")[0].long()
        lane_off = _typed(s, "lane_off")[0].long()
        for sub in subsets:
            r = {}
            sel = torch.from_numpy(np.ascontiguousarray(sub.sel)).cuda()
            pos_sel = sel[perm]
            pos_idx = pos_sel.nonzero().squeeze(1)
            pos_map = (torch.cumsum(pos_sel, 0) - 1).to(torch.int32)
            pos_map[~pos_sel] = -1
            inv = (torch.cumsum(sel, 0) - 1).to(torch.int32)
            nv_sub = int(pos_sel[:n_valid].sum())
            r["n_valid"] = nv_sub
            wkeep = list(range(W)) if sub.windows is None else list(sub.windows)
            wmap = torch.full((W,), -1, dtype=torch.int32, device=perm.device)
            wmap[torch.tensor(wkeep, device=perm.device)] = torch.arange(
                len(wkeep), dtype=torch.int32, device=perm.device)

            def per_record(res, name):
                t, dt = _typed(res, name)
                v = t[pos_idx]
                if name in _POSITIONAL:
                    v = torch.where(v >= 0, pos_map[v.clamp(min=0).long()], v)
                return _host(v, dt)

            # lanes that keep at least one record, their new offsets
            csum = torch.cat([torch.zeros(1, dtype=torch.int64, device=perm.device),
                              torch.cumsum(pos_sel[:n_valid], 0)])
            lo, hi = csum[lane_off[:-1]], csum[lane_off[1:]]
            lkeep = hi > lo
            lane_new = (torch.cumsum(lkeep, 0) - 1).to(torch.int32)
            if "sort" in sub.groups:
                r["perm"] = _host(inv[perm[pos_idx]], np.dtype("<i4"))
                for k in _PER_RECORD_SORT:
                    r[k] = per_record(s, k)
                for k in _LANE_COLS:
                    t, dt = _typed(s, k)
                    v = t[lkeep]
                    if k == "lane_window":
                        v = wmap[v.long()]
                    r[k] = _host(v, dt)
                r["lane_off"] = _host(torch.cat([lo[lkeep], torch.tensor([nv_sub], device=lo.device)])
                                      .to(torch.int32), np.dtype("<i4"))
                if sub.windows is not None:
                    r["load_sum"] = w.load_summary[wkeep]
            if "join" in sub.groups:
                for k in JOIN_KEYS[:-1]:
                    r[k] = per_record(j, k)
                if sub.windows is not None:
                    r["join_sum"] = j.numpy("join_sum")[wkeep]
            if "attr" in sub.groups:
                r["attr_status"] = a.status
                for k in ATTR_KEYS[:-1]:
                    r[k] = per_record(a, k)
                if sub.windows is not None:
                    r["attr_sum"] = a.numpy("attr_sum")[wkeep]
            if "gaps" in sub.groups:
                r["gap_before"] = per_record(g, "gap_before")
                t, dt = _typed(g, "lane_gaps")
                r["lane_gaps"] = _host(t[lkeep], dt)
                t, dt = _typed(g, "lane_hist")
                r["lane_hist"] = _host(t.reshape(-1, NBINS)[lkeep], dt).reshape(-1, NBINS)
                if sub.windows is not None:
                    t, dt = _typed(g, "win_hist")
                    r["win_hist"] = _host(t.reshape(-1, NBINS)[torch.tensor(wkeep, device=t.device)],
                                          dt).reshape(-1, NBINS)
                t, dt = _typed(g, "long_gaps")
                if t.shape[0]:
                    cols = t.reshape(-1).view(torch.int32).reshape(-1, dt.itemsize // 4).clone()
                    rows = lkeep[cols[:, 0].long()]
                    cols = cols[rows]
                    cols[:, 0] = lane_new[cols[:, 0].long()]
                    nxt = cols[:, 1]
                    cols[:, 1] = torch.where(nxt >= 0, pos_map[nxt.clamp(min=0).long()], nxt)
                    r["long_gaps"] = cols.contiguous().cpu().numpy().reshape(-1).view(dt).copy()
                else:
                    r["long_gaps"] = np.empty(0, dtype=dt)
            if "rollup" in sub.groups and ru is not None:
                for k in ROLLUP_KEYS[:-1]:
                    r[k] = per_record(ru, k)
                if sub.windows is not None:
                    r["roll_sum"] = ru.numpy("roll_sum")[wkeep]
            if "blame" in sub.groups:
                r["op_gap_ns"] = per_record(bl, "op_gap_ns")
                t, dt = _typed(g, "long_gaps")
                if t.shape[0]:
                    lanes_of = t.reshape(-1).view(torch.int32).reshape(-1, dt.itemsize // 4)[:, 0]
                    rows = lkeep[lanes_of.long()]
                    r["b_class"] = _host(_typed(bl, "b_class")[0][rows], np.dtype("<i4"))
                    v = _typed(bl, "b_launch")[0][rows]
                    r["b_launch"] = _host(torch.where(v >= 0, pos_map[v.clamp(min=0).long()], v),
                                          np.dtype("<i4"))
                else:
                    r["b_class"] = np.empty(0, dtype=np.int32)
                    r["b_launch"] = np.empty(0, dtype=np.int32)
                if sub.windows is not None:
                    r["b_win_count"] = bl.numpy("b_win_count")[wkeep]
                    r["b_win_ns"] = bl.numpy("b_win_ns")[wkeep]
            if "agg" in sub.groups:
                for tag, res in (("agg0", ag_dev), ("aggT", ag_op), ("aggG", ag_gap), ("aggP", ag_path)):
                    if tag == "aggG" and "blame" not in sub.groups:
                        continue
                    if tag == "aggP" and "critpath" not in sub.groups:
                        continue
                    if res is None:
                        continue
                    gw = _typed(res, "g_window")[0]
                    rows = wmap[gw.long()] >= 0
                    if sub.pid is not None:
                        rows &= _typed(res, "g_pid")[0] == sub.pid
                    for k in AGG_KEYS:
                        t, dt = _typed(res, k)
                        if k == "g_hist":
                            v = t.reshape(-1, NBINS)[rows]
                            r[f"{tag}_{k}"] = _host(v, dt).reshape(-1, NBINS)
                            continue
                        v = t[rows]
                        if k == "g_window":
                            v = wmap[v.long()]
                        r[f"{tag}_{k}"] = _host(v, dt)
            if "coll" in sub.groups:
                cw = _typed(c, "c_window")[0]
                crow = wmap[cw.long()] >= 0
                rw = _typed(c, "r_window")[0]
                rrow = wmap[rw.long()] >= 0
                for k in COLL_KEYS:
                    t, dt = _typed(c, k)
                    if k == "wait_ns":
                        r[k] = _host(t[pos_idx], dt)
                        continue
                    v = t[crow] if k.startswith("c_") else t[rrow]
                    if k in ("c_window", "r_window"):
                        v = wmap[v.long()]
                    r[k] = _host(v, dt)
            if "overlap" in sub.groups:
                rows = wmap[_typed(ov, "d_window")[0].long()] >= 0
                if sub.pid is not None:
                    rows &= _typed(ov, "d_pid")[0] == sub.pid
                for k in OVERLAP_KEYS:
                    t, dt = _typed(ov, k)
                    v = t[rows]
                    if k == "d_window":
                        v = wmap[v.long()]
                    r[k] = _host(v, dt)
            if "critpath" in sub.groups:
                r["on_path"] = per_record(cp, "on_path")
                rows = wmap[_typed(cp, "cp_window")[0].long()] >= 0
                if sub.pid is not None:
                    rows &= _typed(cp, "cp_pid")[0] == sub.pid
                for k in CRITPATH_KEYS[1:-1]:
                    t, dt = _typed(cp, k)
                    if k == "cp_ns":
                        r[k] = _host(t.reshape(-1, 8)[rows].reshape(-1), dt)
                        continue
                    v = t[rows]
                    if k == "cp_window":
                        v = wmap[v.long()]
                    elif k == "cp_sink":
                        v = pos_map[v.long()]
                    r[k] = _host(v, dt)
                if sub.windows is not None:
                    r["cp_sum"] = cp.numpy("cp_sum").reshape(-1, 10)[wkeep].reshape(-1)
            out[sub.name] = r
            del sel, pos_sel, pos_idx, pos_map, inv, csum
    return out


def subset_input(events, win_off, sel, windows=None):
    """The subset as an input of its own: (events, win_off, kept window indices)."""
    W = len(win_off) - 1
    wkeep = list(range(W)) if windows is None else list(windows)
    cs = np.concatenate([[0], np.cumsum(sel, dtype=np.int64)])
    off = np.asarray(win_off, dtype=np.int64)
    counts = cs[off[1:]] - cs[off[:-1]]
    sub_off = np.concatenate([[0], np.cumsum(counts[wkeep])]).astype(np.int64)
    return events[sel], sub_off, wkeep
