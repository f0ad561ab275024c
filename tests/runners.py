"""Runs one analysis end to end and returns every output as numpy arrays under
common names, once through the CPU oracle and once through the CUDA library,
so that golden checks and parity checks can treat both alike."""
import numpy as np

SORT_KEYS = ["perm", "ts_start", "ts_end", "corr_id", "pid", "name_id", "seq", "stream", "kind",
             "lane_window", "lane_pid", "lane_stream", "lane_domain", "lane_off"]
JOIN_KEYS = ["launch_of", "launch_latency", "queue_delay", "kernels_of_launch", "join_sum"]
ATTR_KEYS = ["parent", "depth", "op_of", "op_first_start", "op_last_end", "op_kernel_ns",
             "op_n_kernels", "attr_sum"]
GAP_KEYS = ["gap_before", "lane_gaps", "lane_hist", "win_hist", "long_gaps"]
AGG_KEYS = ["g_window", "g_pid", "g_name", "g_count", "g_sum", "g_min", "g_max", "g_hist"]
COLL_KEYS = ["c_window", "c_comm", "c_seq", "c_n_members", "c_min_start", "c_max_start", "c_skew",
             "c_max_end", "c_straggler_pid", "c_flags", "wait_ns", "r_window", "r_pid", "r_n_coll",
             "r_sum_wait", "r_max_wait", "r_n_straggler"]

ROLLUP_KEYS = ["incl_n_kernels", "incl_first_start", "incl_last_end", "incl_kernel_ns",
               "replay_first_start", "replay_last_end", "replay_kernel_ns", "roll_sum"]
BLAME_KEYS = ["b_class", "b_launch", "b_win_count", "b_win_ns", "op_gap_ns"]
OVERLAP_KEYS = ["d_window", "d_pid", "d_n_events", "d_busy", "d_idle", "d_compute", "d_comm",
                "d_overlap", "d_exposed"]

SOL_KEYS = ["sol_mfu", "sol_mbu", "sol_op", "sol_state", "sol_sum"]
CRITPATH_KEYS = ["on_path", "cp_window", "cp_pid", "cp_sink", "cp_n_nodes", "cp_reason", "cp_begin",
                 "cp_end", "cp_ns", "cp_sum"]

DEVICE_MASK = (1 << 3) | (1 << 4) | (1 << 5)
OP_MASK = 1
NODE_MASK = 62  # API, LAUNCH and the device kinds: what a critical path is made of


def run_oracle(events, win_off, t0, t1, min_gap=500_000, comm_sizes=(), agg_masks=(DEVICE_MASK,),
               op_work=None):
    """op_work = (flops, bytes, peak_flops, peak_bw): also the operator efficiency step."""
    from oracle.ta_oracle import Oracle
    o = Oracle(events, win_off, t0, t1)
    r = {}
    r["load_sum"] = o.load()
    o.sort()
    r["n_valid"] = o.n_valid
    for k in SORT_KEYS:
        r[k] = o.get(k)
    o.correlate()
    for k in JOIN_KEYS:
        r[k] = o.get(k)
    r["attr_status"] = o.attribute()
    for k in ATTR_KEYS:
        r[k] = o.get(k)
    o.gaps(min_gap)
    for k in GAP_KEYS:
        r[k] = o.get(k)
    for i, m in enumerate(agg_masks):
        assert o.aggregate(m, 0) == 0
        for k in AGG_KEYS:
            r[f"agg{i}_{k}"] = o.get(k)
    assert o.aggregate(OP_MASK, 1) == 0
    for k in AGG_KEYS:
        r[f"aggT_{k}"] = o.get(k)
    o.collectives(comm_sizes)
    for k in COLL_KEYS:
        r[k] = o.get(k)
    if r["attr_status"] == 0:
        o.rollup()
        for k in ROLLUP_KEYS:
            r[k] = o.get(k)
        if op_work is not None:
            o.sol(*op_work)
            for k in SOL_KEYS:
                r[k] = o.get(k)
    o.blame()
    for k in BLAME_KEYS:
        r[k] = o.get(k)
    assert o.aggregate(OP_MASK, 2) == 0
    for k in AGG_KEYS:
        r[f"aggG_{k}"] = o.get(k)
    o.device_overlap()
    for k in OVERLAP_KEYS:
        r[k] = o.get(k)
    o.critical_path()
    for k in CRITPATH_KEYS:
        r[k] = o.get(k)
    assert o.aggregate(NODE_MASK, 3) == 0
    for k in AGG_KEYS:
        r[f"aggP_{k}"] = o.get(k)
    o.close()
    return r


def run_gpu(events, win_off, t0, t1, min_gap=500_000, comm_sizes=(), agg_masks=(DEVICE_MASK,),
            on_device=True, use_torch_allocator=True, op_work=None):
    """Same analysis through the C ABI of the CUDA library (torch supplies memory + stream)."""
    import torch
    from paper_2609_40247_b200 import ta
    if on_device:
        buf = torch.from_numpy(np.ascontiguousarray(events).view(np.uint8).reshape(-1)).cuda()
    else:
        buf = np.ascontiguousarray(events)
    r = {}
    with ta.Window(buf, win_off, t0, t1, use_torch_allocator=use_torch_allocator) as w:
        r["load_sum"] = w.load_summary
        s = w.sort_timeline()
        r["n_valid"] = s.n_valid
        for k in SORT_KEYS:
            r[k] = s.numpy(k)
        j = w.correlate_launches()
        for k in JOIN_KEYS:
            r[k] = j.numpy(k)
        a = w.attribute_operators(check=False)
        r["attr_status"] = a.status
        for k in ATTR_KEYS:
            r[k] = a.numpy(k)
        g = w.stream_gaps(min_gap)
        for k in GAP_KEYS:
            r[k] = g.numpy(k)
        for i, m in enumerate(agg_masks):
            ag = w.aggregate_ops(m, 0)
            for k in AGG_KEYS:
                r[f"agg{i}_{k}"] = ag.numpy(k)
        if a.status == 0:
            ag = w.aggregate_ops(OP_MASK, 1)
            for k in AGG_KEYS:
                r[f"aggT_{k}"] = ag.numpy(k)
        c = w.match_collectives(comm_sizes)
        for k in COLL_KEYS:
            r[k] = c.numpy(k)
        if a.status == 0:
            ru = w.rollup_operators()
            for k in ROLLUP_KEYS:
                r[k] = ru.numpy(k)
            if op_work is not None:
                so = w.operator_sol(*op_work)
                for k in SOL_KEYS:
                    r[k] = so.numpy(k)
        b = w.blame_gaps(g)
        for k in BLAME_KEYS:
            r[k] = b.numpy(k)
        ag = w.aggregate_ops(OP_MASK, 2)
        for k in AGG_KEYS:
            r[f"aggG_{k}"] = ag.numpy(k)
        d = w.device_overlap()
        for k in OVERLAP_KEYS:
            r[k] = d.numpy(k)
        cp = w.critical_path()
        for k in CRITPATH_KEYS:
            r[k] = cp.numpy(k)
        ag = w.aggregate_ops(NODE_MASK, 3)
        for k in AGG_KEYS:
            r[f"aggP_{k}"] = ag.numpy(k)
    return r


def assert_same(a, b, skip=()):
    """Bit-exact comparison of two result dicts (b may lack keys that a has)."""
    for k in a:
        if k in skip or k not in b:
            continue
        x, y = a[k], b[k]
        if k == "sol_sum":
            # the two float sums are accumulated in no particular order on the GPU; everything
            # else in the row (counts, the exact T_op sum, the maximum) is compared exactly
            assert x.dtype == y.dtype and x.shape == y.shape
            for f in x.dtype.names:
                if f in ("sum_flops", "sum_bytes"):
                    assert np.allclose(x[f], y[f], rtol=1e-9, atol=0), (k, f)
                else:
                    assert np.array_equal(x[f], y[f]), (k, f)
            continue
        if isinstance(x, np.ndarray):
            assert x.dtype == y.dtype, (k, x.dtype, y.dtype)
            assert x.shape == y.shape, (k, x.shape, y.shape)
            if not np.array_equal(x, y):
                if x.dtype.names:
                    bad = np.nonzero(x != y)[0]
                else:
                    bad = np.argwhere(x != y)
                raise AssertionError(f"{k}: {len(bad)} mismatches, first at {bad[0]}: "
                                     f"{x[tuple(np.atleast_1d(bad[0]))]} vs {y[tuple(np.atleast_1d(bad[0]))]}")
        else:
            assert x == y, (k, x, y)
