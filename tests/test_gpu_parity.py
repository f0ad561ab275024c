"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle,
bit for bit, on the hand-worked windows, on random adversarial tiny windows and
on scaled-down copies of the five benchmark workloads."""
import numpy as np
import pytest

import golden_checks
from helpers import make_events
from paper_2609_40247_b200 import synth
from runners import DEVICE_MASK, assert_same, run_gpu, run_oracle
from test_oracle_truth import check_against_truth
from tiny import random_window, schedule_window

pytestmark = pytest.mark.gpu


def both(ev, off, t0, t1, **kw):
    o = run_oracle(ev, off, t0, t1, **kw)
    g = run_gpu(ev, off, t0, t1, **kw)
    skip = ()
    if o["attr_status"] != 0:
        # outputs of the attribution are unspecified after a nesting / depth error; the status
        # and the flags must agree
        assert g["attr_status"] == o["attr_status"]
        assert np.array_equal(g["attr_sum"]["bad_nesting"] > 0, o["attr_sum"]["bad_nesting"] > 0) \
            or o["attr_status"] == 8
        skip = ("parent", "depth", "op_of", "op_first_start", "op_last_end", "op_kernel_ns",
                "op_n_kernels", "attr_sum") + tuple(k for k in o if k.startswith("aggT_"))
    assert_same(o, g, skip=skip)
    return o, g


@pytest.mark.parametrize("check", golden_checks.ALL, ids=lambda f: f.__name__)
def test_hand_worked_windows(check):
    check(run_gpu)


@pytest.mark.parametrize("seed", range(16))
def test_tiny_adversarial_windows(seed):
    ev, off, t0, t1, sizes = random_window(seed)
    both(ev, off, t0, t1, min_gap=7, comm_sizes=sizes, agg_masks=(DEVICE_MASK, 1 << 2, 63))


@pytest.mark.parametrize("seed", range(8))
def test_tiny_windows_with_partial_overlap(seed):
    ev, off, t0, t1, sizes = random_window(100 + seed, nested=False, defects=False)
    both(ev, off, t0, t1, min_gap=3, comm_sizes=sizes)


@pytest.mark.parametrize("seed,tight", [(s, t) for s in range(6) for t in (False, True)])
def test_simulated_schedules(seed, tight):
    """Launches, kernels in stream order and waits of a simulated run: every kind of edge of the
    critical path occurs (submission, stream order, program order, synchronisation)."""
    ev, off, t0, t1, _ = schedule_window(seed, tight=tight, n_actions=300, n_streams=3, n_pid=3)
    o, g = both(ev, off, t0, t1, min_gap=20)
    assert int(o["cp_ns"].reshape(-1, 8)[:, 7].sum()) > 0


@pytest.mark.parametrize("seed", [5598, 6030, 6746, 7166, 7226, 8514])
def test_equal_operator_ends_across_tile_boundaries(seed):
    """Windows found by differential fuzzing: an operator and one nested in it end at the same
    instant, and the records they enclose continue in the next tile of the attribution kernels
    (the stack carried from tile to tile has to keep both)."""
    rng = np.random.default_rng(seed)
    ev, off, t0, t1, sizes = random_window(seed, span=int(rng.integers(200, 20000)),
                                           n_dev=int(rng.integers(10, 6000)),
                                           max_depth=int(rng.integers(1, 8)), n_pid=int(rng.integers(1, 5)))
    both(ev, off, t0, t1, min_gap=1, comm_sizes=sizes)


def test_larger_random_window_spans_tiles():
    ev, off, t0, t1, sizes = random_window(50, span=6000, n_dev=9000, max_depth=7, n_pid=3)
    both(ev, off, t0, t1, min_gap=1, comm_sizes=sizes)


def test_sparse_correlation_ids_take_the_sort_merge_join():
    """Correlation ids spread over a range far wider than the record count: the direct-address
    table is not used, launches and probes are matched by sorting (several tiles of each)."""
    wl = synth.make_workload("c1", 0.02, truth=False)
    ev = wl.events.copy()
    dev_or_launch = ev["kind"] != 5
    ev["corr_id"][dev_or_launch] = ev["corr_id"][dev_or_launch] * 1_000_003 - 2**45
    o, g = both(ev, wl.win_off, wl.win_t0, wl.win_t1, comm_sizes=wl.comm_sizes)
    assert int(o["join_sum"]["n_matched"].sum()) > 20_000


def test_widely_spread_symbol_ids_are_grouped_by_sorting():
    """name_id values a million apart: the dense aggregate table does not apply and the rows of
    all three aggregate selectors come from the sort-based path."""
    wl = synth.make_workload("c1", 0.05, truth=False)
    ev = wl.events.copy()
    ev["name_id"] = (ev["name_id"].astype(np.int64) * 1_048_573 - 2**30).astype(np.int32)
    o, g = both(ev, wl.win_off, wl.win_t0, wl.win_t1, comm_sizes=wl.comm_sizes,
                agg_masks=(DEVICE_MASK, 1 << 2, 63))
    assert len(o["agg0_g_count"]) > 100 and len(o["aggT_g_count"]) > 10


@pytest.mark.parametrize("run_len,ordinary", [(2, 300), (5, 300), (31, 300), (48, 300), (49, 300),
                                              (400, 300), (60, 12000)])
def test_runs_of_equal_start_times(run_len, ordinary):
    """Many records of one stream start at the same time: their order (longer first, then
    input order) comes from the run ranking of the gather up to 48 members, and from the
    full-resolution pair sort with its duration key beyond that."""
    rng = np.random.default_rng(run_len + ordinary)
    rows = []
    for pid in (4, 9):
        for s0 in (100, 5000, 5001):
            for i in range(run_len):
                dur = int(rng.integers(0, 6))  # few distinct durations: equal intervals too
                rows.append(("KERNEL", pid, 1, s0, s0 + dur, int(rng.integers(0, 50)), i % 3, 0))
        for i in range(ordinary):  # ordinary traffic around the runs
            s = int(rng.integers(0, 9000))
            rows.append(("KERNEL", pid, int(rng.integers(0, 2)), s, s + int(rng.integers(0, 40)),
                         int(rng.integers(0, 50)), int(rng.integers(0, 4)), 0))
            rows.append(("LAUNCH", pid, 0, s // 2, s // 2 + 1, int(rng.integers(0, 50)), 0, 0))
    order = rng.permutation(len(rows))
    ev = make_events([rows[i] for i in order])
    both(ev, [0, len(ev)], [0], [10000], min_gap=5)


def test_defects_sprinkled_over_a_multi_window_batch():
    """A few percent of the records of a nine-window batch are made defective (bad kind, negative
    length, start outside the window): the dropped tail spans many tiles and every window."""
    wl = synth.make_workload("c4", 0.002, truth=False, n_windows=9)
    ev = wl.events.copy()
    rng = np.random.default_rng(11)
    n = len(ev)
    bad = rng.choice(n, size=n // 25, replace=False)
    third = len(bad) // 3
    ev["kind"][bad[:third]] = 9
    ev["ts_end"][bad[third:2 * third]] = ev["ts_start"][bad[third:2 * third]] - 1 - rng.integers(0, 1000, third)
    ev["ts_start"][bad[2 * third:]] -= 10**12
    o, g = both(ev, wl.win_off, wl.win_t0, wl.win_t1, min_gap=500_000, comm_sizes=wl.comm_sizes)
    assert o["n_valid"] < n - third and int(o["load_sum"]["n_bad_kind"].sum()) == third


def test_one_overlong_kernel_sends_the_critical_path_to_its_sorted_search():
    """In-order streams end their records in ascending order and the critical path searches
    each stream lane directly; a single kernel that outlives its successors makes it sort the
    device records by end time instead (several tiles, sixteen processes)."""
    wl = synth.make_workload("c3", 0.01, truth=False)
    ev = wl.events.copy()
    k = np.nonzero(ev["kind"] == 3)[0]
    ev["ts_end"][k[len(k) // 2]] += 10_000_000
    o, g = both(ev, wl.win_off, wl.win_t0, wl.win_t1, min_gap=500_000, comm_sizes=wl.comm_sizes)
    assert int(o["cp_n_nodes"].sum()) > 10_000


def test_deep_nesting_is_reported():
    rows = [("OP", 1, 0, 10 + i, 1000 - i, 0, i, 0) for i in range(12)]
    rows.append(("LAUNCH", 1, 0, 100, 110, 1, 0, 0))
    ev = make_events(rows)
    o, g = both(ev, [0, len(ev)], [0], [2000])
    assert o["attr_status"] == 8 and g["attr_status"] == 8
    assert g["attr_sum"]["max_depth"][0] == 12


def test_defective_records_pin():
    rows = [("KERNEL", 1, 0, 10, 20, 0, 0, 0), (7, 1, 0, 10, 20, 0, 0, 0), (-1, 1, 0, 10, 20, 0, 0, 0),
            ("KERNEL", 1, 0, 30, 20, 0, 0, 0), ("OP", 1, 0, 5, 50, 0, 0, 0), ("OP", 1, 0, -5, 50, 0, 0, 0),
            ("LAUNCH", 1, 0, 100, 120, 0, 0, 0), ("LAUNCH", 1, 0, 99, 120, 0, 0, 0),
            ("COLL", 2, 0, 99, 2000, 0, 0, 0), ("API", 2, 1, 0, 0, 0, 0, 0),
            ("MEMCPY", 2, 0, 100, 100, 0, 0, 0), (6, -3, 0, 100, 100, 0, 0, 0)]
    ev = make_events(rows)
    o, g = both(ev, [0, len(ev)], [0], [100])
    s = g["load_sum"][0]
    assert (s["n_events"], s["n_valid"], s["n_bad_kind"], s["n_bad_interval"], s["n_out_of_window"]) \
        == (12, 5, 3, 1, 3)


def test_empty_inputs():
    ev = make_events([])
    both(ev, [0, 0], [0], [100])
    ev = make_events([("KERNEL", 1, 0, 10, 20, 0, 0, 0)])
    both(ev, [0, 0, 1, 1], [0, 0, 0], [100, 100, 100])


def test_host_buffer_input_matches_device_input():
    ev, off, t0, t1, sizes = random_window(3)
    a = run_gpu(ev, off, t0, t1, comm_sizes=sizes, on_device=True)
    b = run_gpu(ev, off, t0, t1, comm_sizes=sizes, on_device=False)
    assert_same(a, b)


# c0 x 10: one process, one host thread, two streams - three lanes of 200 000 records each
# (long look-back chains, a deep tree of tile stacks)
CASES = [("c0", 1.0, 0), ("c0", 1.0, 1), ("c1", 0.1, 0), ("c1", 0.03, 1), ("c2", 0.02, 0),
         ("c3", 0.01, 0), ("c4", 0.002, 0), ("c0", 10.0, 0)]


@pytest.mark.parametrize("name,scale,shuffle", CASES)
def test_scaled_workloads(name, scale, shuffle):
    wl = synth.make_workload(name, scale, shuffle_mode=shuffle, n_windows=9 if name == "c4" else None)
    flops, nbytes = synth.op_work(wl.events, seed=7)
    o, g = both(wl.events, wl.win_off, wl.win_t0, wl.win_t1, min_gap=500_000,
                comm_sizes=wl.comm_sizes, op_work=(flops, nbytes, synth.PEAK_FLOPS, synth.PEAK_BW))
    assert int((o["sol_state"] == 1).sum()) > 100 and int((o["sol_state"] == 3).sum()) > 0
    check_against_truth(wl, g)


def test_operator_sol_counts_on_the_device_and_unknown_counts():
    """The side table as CUDA tensors (no copy inside the call), NaN and negative counts, a
    window batch (the warp fold meets window boundaries)."""
    import torch
    wl = synth.make_workload("c4", 0.002, truth=False, n_windows=9)
    flops, nbytes = synth.op_work(wl.events, seed=3, unknown_frac=0.2)
    nbytes[::7] = np.nan
    args = (wl.events, wl.win_off, wl.win_t0, wl.win_t1)
    o = run_oracle(*args, comm_sizes=wl.comm_sizes, op_work=(flops, nbytes, 1e15, 5e12))
    g = run_gpu(*args, comm_sizes=wl.comm_sizes,
                op_work=(torch.from_numpy(flops).cuda(), torch.from_numpy(nbytes).cuda(), 1e15, 5e12))
    assert_same(o, g)
    assert int(o["sol_sum"]["n_no_counts"].sum()) > 100
