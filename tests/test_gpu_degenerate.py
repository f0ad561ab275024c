"""Degenerate and extreme inputs through the CUDA library and the oracle alike, run-to-run
determinism, and two handles alive at once on different streams."""
import numpy as np
import pytest

from helpers import make_events
from paper_2609_40247_b200 import synth
from runners import assert_same, run_gpu, run_oracle
from tiny import random_window

pytestmark = pytest.mark.gpu
I32, I16 = 2**31, 2**15
T0 = 1_700_000_000_000_000_000  # wall-clock nanoseconds: the full 64-bit range is in play


def _both(rows, off=None, t0=(0,), t1=(10_000,), **kw):
    ev = make_events(rows)
    off = [0, len(ev)] if off is None else off
    o = run_oracle(ev, off, list(t0), list(t1), **kw)
    g = run_gpu(ev, off, list(t0), list(t1), **kw)
    skip = ()
    if o["attr_status"] != 0:
        skip = tuple(k for k in o if k.startswith(("parent", "depth", "op_", "attr_sum", "aggT_", "incl_",
                                                   "replay_", "roll_")))
        assert g["attr_status"] == o["attr_status"]
    assert_same(o, g, skip=skip)
    return o


CASES = {
    "one kernel": [("KERNEL", 1, 0, 10, 20, 0, 0, 0)],
    "one host record": [("OP", 1, 0, 10, 20, 0, 0, 0)],
    "host records only": [("OP", 1, 0, 0, 100, 0, 0, 0), ("LAUNCH", 1, 0, 5, 6, 1, 0, 0), ("API", 1, 0, 7, 7, 0, 0, 0)],
    "device records only": [("KERNEL", 1, s, 10 * s, 10 * s + 5, s, 0, 0) for s in range(7)],
    "everything dropped": [("KERNEL", 1, 0, 20_000, 20_001, 0, 0, 0), (9, 1, 0, 1, 2, 0, 0, 0), ("OP", 1, 0, 9, 3, 0, 0, 0)],
    "extreme ids": [("KERNEL", -I32, -I16, 10, 20, -2**63, -I32, 0), ("KERNEL", I32 - 1, I16 - 1, 10, 20, 2**63 - 1, I32 - 1, 0),
                    ("LAUNCH", -I32, -I16, 1, 2, -2**63, 0, 0), ("LAUNCH", I32 - 1, I16 - 1, 1, 2, 2**63 - 1, 0, 0),
                    ("OP", -I32, -I16, 0, 9000, 0, -I32, 0), ("OP", I32 - 1, I16 - 1, 0, 9000, 0, I32 - 1, 0),
                    ("COLL", -I32, 3, 50, 60, 2**63 - 2, 0, -I32), ("COLL", I32 - 1, 3, 55, 60, 2**63 - 2, 0, -I32)],
    "all zero length at one instant": [("KERNEL", 1, 0, 500, 500, i, 0, 0) for i in range(40)]
    + [("OP", 1, 0, 500, 500, 0, i, 0) for i in range(6)] + [("LAUNCH", 1, 0, 500, 500, i, 0, 0) for i in range(40)],
    "kernel that outlives the window": [("LAUNCH", 1, 0, 10, 11, 1, 0, 0), ("KERNEL", 1, 0, 20, 10**12, 1, 0, 0),
                                        ("KERNEL", 1, 0, 30, 40, 2, 0, 0)],
    # a kernel that ends exactly when the wait returns did not release it (strictly before), one that
    # ends exactly when the wait begins did; calls nested in a call; zero-length waits; equal last ends
    "waits, ties and nested calls": [
        ("LAUNCH", 1, 0, 10, 12, 1, 0, 0), ("LAUNCH", 1, 0, 13, 14, 2, 0, 0), ("KERNEL", 1, 0, 15, 50, 1, 0, 0),
        ("KERNEL", 1, 1, 16, 20, 2, 0, 0), ("API", 1, 0, 20, 50, 0, 0, 0),
        ("API", 1, 0, 60, 100, 0, 1, 0), ("LAUNCH", 1, 0, 70, 72, 3, 0, 0), ("API", 1, 0, 95, 98, 0, 2, 0),
        ("KERNEL", 1, 0, 75, 96, 3, 0, 0), ("API", 1, 0, 200, 200, 0, 3, 0), ("KERNEL", 1, 1, 150, 199, 9, 0, 0),
        ("LAUNCH", 1, 0, 250, 260, 4, 0, 0), ("KERNEL", 1, 0, 255, 300, 4, 0, 0), ("API", 1, 0, 270, 300, 0, 4, 0),
        ("API", 2, 0, 10, 300, 0, 0, 0), ("COLL", 2, 7, 20, 40, 5, 0, 0), ("COLL", 2, 7, 40, 290, 5, 0, 1),
        ("KERNEL", 2, 7, 100, 120, 6, 0, 0), ("LAUNCH", 2, 0, 5, 6, 6, 0, 0),
        ("LAUNCH", 3, 0, 500, 510, 8, 0, 0), ("KERNEL", 3, 0, 400, 450, 8, 0, 0)],  # launch after its kernel
    "many kernels per launch": [("OP", 1, 0, 0, 5000, 0, 0, 0), ("LAUNCH", 1, 0, 10, 20, 7, 0, 0)]
    + [("KERNEL", 1, i % 3, 100 + 10 * i, 105 + 10 * i, 7, 0, 0) for i in range(100)],
}


@pytest.mark.parametrize("name", sorted(CASES))
def test_degenerate_windows(name):
    _both(CASES[name], min_gap=3)


def test_wall_clock_timestamps_and_empty_windows_between_full_ones():
    rows, off, t0, t1 = [], [0], [], []
    rng = np.random.default_rng(5)
    for w in range(9):
        a = T0 + w * 60_000_000_000
        t0.append(a)
        t1.append(a + 30_000_000_000)
        if w % 3 != 1:  # every third window is empty
            for i in range(50):
                s = a + int(rng.integers(0, 29_000_000_000))
                rows.append(("LAUNCH", 1 + w % 2, 0, s, s + 1000, i, 0, 0))
                rows.append(("KERNEL", 1 + w % 2, i % 2, s + 5000, s + 5000 + int(rng.integers(0, 10**9)), i, i % 5, 0))
        off.append(len(rows))
    _both(rows, off=off, t0=t0, t1=t1, min_gap=10**6)


def test_two_runs_give_identical_results():
    wl = synth.make_workload("c3", 0.01, truth=False)
    a = (wl.events, wl.win_off, wl.win_t0, wl.win_t1)
    assert_same(run_gpu(*a, comm_sizes=wl.comm_sizes), run_gpu(*a, comm_sizes=wl.comm_sizes))


def test_two_handles_on_two_streams_do_not_disturb_each_other():
    import torch
    from paper_2609_40247_b200 import ta
    ev1, off1, a1, b1, _ = random_window(21)
    wl = synth.make_workload("c1", 0.02, truth=False)
    want1 = run_gpu(ev1, off1, a1, b1)
    want2 = run_gpu(wl.events, wl.win_off, wl.win_t0, wl.win_t1)
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    buf1 = torch.from_numpy(np.ascontiguousarray(ev1).view(np.uint8).reshape(-1)).cuda()
    buf2 = torch.from_numpy(np.ascontiguousarray(wl.events).view(np.uint8).reshape(-1)).cuda()
    torch.cuda.synchronize()
    with ta.Window(buf1, off1, a1, b1, stream=s1) as w1, \
            ta.Window(buf2, wl.win_off, wl.win_t0, wl.win_t1, stream=s2) as w2:
        r2 = w2.sort_timeline()
        r1 = w1.sort_timeline()
        j1 = w1.correlate_launches()
        j2 = w2.correlate_launches()
        g2 = w2.stream_gaps(500_000)
        g1 = w1.stream_gaps(500_000)
        for k in ("perm", "ts_start", "kind", "lane_off"):
            assert np.array_equal(r1.numpy(k), want1[k]) and np.array_equal(r2.numpy(k), want2[k])
        for k in ("launch_of", "launch_latency"):
            assert np.array_equal(j1.numpy(k), want1[k]) and np.array_equal(j2.numpy(k), want2[k])
        assert np.array_equal(g1.numpy("gap_before"), want1["gap_before"])
        assert np.array_equal(g2.numpy("gap_before"), want2["gap_before"])


def test_two_threads_with_a_handle_each():
    """ctypes releases the interpreter lock during a call, so two Python threads really are
    inside the library at the same time, each with its own handle and stream."""
    import threading
    import torch
    wl = [synth.make_workload("c1", 0.03, truth=False, seed_offset=k) for k in range(2)]
    want = [run_gpu(w.events, w.win_off, w.win_t0, w.win_t1, comm_sizes=w.comm_sizes) for w in wl]
    got = [None, None]
    errors = []

    def work(k):
        try:
            torch.cuda.set_device(0)
            with torch.cuda.stream(torch.cuda.Stream()):
                for _ in range(3):
                    got[k] = run_gpu(wl[k].events, wl[k].win_off, wl[k].win_t0, wl[k].win_t1,
                                     comm_sizes=wl[k].comm_sizes)
        except Exception as e:  # surfaced in the main thread below
            errors.append(e)

    threads = [threading.Thread(target=work, args=(k,)) for k in range(2)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors
    for k in range(2):
        assert_same(want[k], got[k])


def test_library_pool_serves_windows_of_changing_sizes():
    """Without allocator callbacks the library keeps released blocks by size and hands them out
    again; windows of alternating sizes must not disturb each other's results, and blocks that
    nobody asks for any more are given back (device memory in use stays bounded)."""
    import torch
    wls = [synth.make_workload("c1", s, truth=False) for s in (0.05, 0.02, 0.05, 0.01, 0.03, 0.05)]
    want = [run_gpu(w.events, w.win_off, w.win_t0, w.win_t1, comm_sizes=w.comm_sizes) for w in wls]
    used = []
    for rep in range(3):
        for w, ref in zip(wls, want):
            got = run_gpu(w.events, w.win_off, w.win_t0, w.win_t1, comm_sizes=w.comm_sizes,
                          use_torch_allocator=False)
            assert_same(ref, got)
        free, total = torch.cuda.mem_get_info()
        used.append(total - free)
    assert used[2] <= used[0] + (64 << 20)  # no growth from round to round
