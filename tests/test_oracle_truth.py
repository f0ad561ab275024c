"""Pins the CPU oracle to the generator's ground truth and to invariants that
hold at any size, on scaled-down copies of the five benchmark workloads."""
import numpy as np
import pytest

from paper_2609_40247_b200 import synth
from runners import run_oracle

CASES = [("c0", 1.0, 0), ("c0", 0.2, 1), ("c1", 0.02, 0), ("c2", 0.005, 0), ("c3", 0.002, 0),
         ("c4", 0.0004, 0)]


def check_against_truth(wl, r):
    """Shared by the oracle tests and the GPU tests: r is a result dict of runners.py."""
    ev = wl.events
    n = len(ev)
    perm = r["perm"].astype(np.int64)
    assert np.array_equal(np.sort(perm), np.arange(n))
    assert r["n_valid"] == n  # the generator emits no defective records
    inv = np.empty(n, dtype=np.int64)
    inv[perm] = np.arange(n)
    link = np.concatenate([t["link"].astype(np.int64) + (off if True else 0)
                           for t, off in zip(wl.truth, wl.win_off[:-1])])
    neg = np.concatenate([t["link"] < 0 for t in wl.truth])
    link[neg] = -1
    val = np.concatenate([t["val"] for t in wl.truth])
    wait = np.concatenate([t["wait"] for t in wl.truth])
    kind = ev["kind"]
    # canonical order: keys never decrease
    win_sorted = np.searchsorted(wl.win_off, perm, side="right") - 1
    dom = (r["kind"] >= 3).astype(np.int64)
    keys = list(zip(win_sorted.tolist(), r["pid"].tolist(), dom.tolist(), r["stream"].tolist(),
                    r["ts_start"].tolist(), (-r["ts_end"]).tolist(), perm.tolist())) if n <= 200000 else None
    if keys is not None:
        assert all(keys[i] < keys[i + 1] for i in range(n - 1))
    # attribution: innermost open operator at emission time; depth = number of open operators
    host = np.nonzero(kind <= 2)[0]
    par_sorted = r["parent"][inv[host]].astype(np.int64)
    par_input = np.where(par_sorted >= 0, perm[np.maximum(par_sorted, 0)], -1)
    assert np.array_equal(par_input, link[host])
    assert np.array_equal(r["depth"][inv[host]].astype(np.int64), val[host])
    assert r["attr_status"] == 0
    # join: the launch the simulation issued for each kernel; deleted launches are unmatched
    probe = np.nonzero((kind == 3) | (kind == 4))[0]
    lo_sorted = r["launch_of"][inv[probe]].astype(np.int64)
    lo_input = np.where(lo_sorted >= 0, perm[np.maximum(lo_sorted, 0)], -1)
    assert np.array_equal(lo_input, link[probe])
    n_deleted = sum(t["n_deleted"] for t in wl.truth)
    assert int(r["join_sum"]["n_unmatched"].sum()) == n_deleted
    assert int(r["join_sum"]["n_dup_launch"].sum()) == 0
    assert (r["join_sum"]["n_matched"] + r["join_sum"]["n_unmatched"] == r["join_sum"]["n_probe"]).all()
    # gaps: streams are in order, so the idle time before a record is known to the simulation
    dev = np.nonzero(kind >= 3)[0]
    assert np.array_equal(r["gap_before"][inv[dev]], val[dev])
    lg = r["lane_gaps"]
    isdev = r["lane_domain"] == 1
    span = (wl.win_t1 - wl.win_t0)[r["lane_window"]]
    assert np.array_equal((lg["busy"] + lg["idle"])[isdev], span[isdev])
    assert np.array_equal(r["lane_hist"].sum(axis=1), lg["n_gaps"])
    assert np.array_equal(r["win_hist"].sum(axis=1),
                          np.bincount(r["lane_window"], weights=lg["n_gaps"], minlength=len(wl.win_t0)).astype(np.int64))
    # collectives: waits until the latest arrival; complete groups everywhere
    coll = np.nonzero(kind == 5)[0]
    assert np.array_equal(r["wait_ns"][inv[coll]], wait[coll])
    if len(coll):
        assert (r["c_flags"] == 0).all()
        assert int(r["r_n_coll"].sum()) == len(coll)
        assert int(r["r_n_straggler"].sum()) == len(r["c_seq"])
        assert int(r["r_sum_wait"].sum()) == int(wait.sum())
    # aggregates cover the population exactly once
    assert int(r["agg0_g_count"].sum()) == len(dev)
    assert int(r["agg0_g_sum"].sum()) == int((ev["ts_end"][dev] - ev["ts_start"][dev]).sum())
    assert np.array_equal(r["agg0_g_hist"].sum(axis=1), r["agg0_g_count"])
    assert (r["agg0_g_min"] <= r["agg0_g_max"]).all()
    assert int(r["aggT_g_count"].sum()) == int((r["op_n_kernels"] > 0).sum())
    # inclusive figures: the roots hold every attributed kernel; a subtree covers its own kernels
    if r["attr_status"] == 0:
        nv = r["n_valid"]
        roots = (r["kind"][:nv] == 0) & (r["parent"][:nv] < 0)
        assert int(r["incl_n_kernels"][:nv][roots].sum()) == int(r["attr_sum"]["n_attributed"].sum())
        assert int(r["incl_kernel_ns"][:nv][roots].sum()) == int(r["op_kernel_ns"].sum())
        own = r["op_n_kernels"] > 0
        assert (r["incl_n_kernels"] >= r["op_n_kernels"]).all()
        assert (r["incl_first_start"][own] <= r["op_first_start"][own]).all()
        assert (r["incl_last_end"][own] >= r["op_last_end"][own]).all()
        many = r["kernels_of_launch"] >= 2
        assert int(many.sum()) == int(r["roll_sum"][:, 0].sum())
        assert int(r["kernels_of_launch"][many].sum()) == int(r["roll_sum"][:, 1].sum())
    # device-level coverage: set identities, and bounds from the per-stream figures
    span = (np.asarray(wl.win_t1) - np.asarray(wl.win_t0))[r["d_window"]]
    assert np.array_equal(r["d_busy"] + r["d_idle"], span)
    assert np.array_equal(r["d_busy"], r["d_compute"] + r["d_comm"] - r["d_overlap"])
    assert np.array_equal(r["d_exposed"], r["d_comm"] - r["d_overlap"])
    assert (r["d_overlap"] <= np.minimum(r["d_compute"], r["d_comm"])).all()
    assert int(r["d_n_events"].sum()) == len(dev)
    devl = np.nonzero(r["lane_domain"] == 1)[0]
    key = {(int(w), int(p)): i for i, (w, p) in enumerate(zip(r["d_window"], r["d_pid"]))}
    lane_max = np.zeros(len(key), dtype=np.int64)
    lane_sum = np.zeros(len(key), dtype=np.int64)
    for l in devl:
        i = key[(int(r["lane_window"][l]), int(r["lane_pid"][l]))]
        b = int(r["lane_gaps"]["busy"][l])
        lane_max[i] = max(lane_max[i], b)
        lane_sum[i] += b
    assert (r["d_busy"] >= lane_max).all() and (r["d_busy"] <= lane_sum).all()
    if not (kind == 5).any() and not (kind == 4).any():
        assert not r["d_comm"].any()


@pytest.mark.parametrize("name,scale,shuffle", CASES)
def test_oracle_reproduces_generator_truth(name, scale, shuffle):
    wl = synth.make_workload(name, scale, shuffle_mode=shuffle, n_windows=6 if name == "c4" else None)
    r = run_oracle(wl.events, wl.win_off, wl.win_t0, wl.win_t1, min_gap=500_000,
                   comm_sizes=wl.comm_sizes)
    check_against_truth(wl, r)


def test_injected_stalls_show_up_as_long_gaps():
    wl = synth.make_workload("c2", 0.004)
    r = run_oracle(wl.events, wl.win_off, wl.win_t0, wl.win_t1, min_gap=500_000)
    val = wl.truth[0]["val"]
    dev = wl.events["kind"] >= 3
    n_long_truth = int(((val >= 500_000) & dev).sum())
    assert n_long_truth > 10
    interior = r["long_gaps"][r["long_gaps"]["next_event"] >= 0]
    assert len(interior) == n_long_truth
    assert np.array_equal(np.sort(r["gap_before"][interior["next_event"]]), np.sort(val[dev & (val >= 500_000)]))
    # a host stall right before a launch leaves the stream idle until the host submits: every
    # such gap is submission-bound
    cls = r["b_class"][r["long_gaps"]["next_event"] >= 0]
    assert (cls == 1).mean() > 0.95 and not (cls == 3).any()
    assert int(r["b_win_count"].sum()) == len(r["long_gaps"])
    assert int(r["b_win_ns"].sum()) == int(r["long_gaps"]["gap_len"].sum())
