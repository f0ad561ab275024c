"""Error behaviour of the C ABI on a GPU: every failure is a status code, the handle stays
freeable, and the next analysis on the same device is unaffected.  All cases are rejected by
argument checks, call-order bookkeeping or bounded device tables; none faults the device."""
import numpy as np
import pytest

from helpers import make_events
from paper_2609_40247_b200 import synth, ta
from runners import assert_same, run_gpu, run_oracle

pytestmark = pytest.mark.gpu

TA_ERR_INVALID_ARG, TA_ERR_ORDER, TA_ERR_TOO_LARGE = 1, 4, 5


def _small():
    wl = synth.make_workload("c0", 0.05, truth=False)
    import torch
    buf = torch.from_numpy(np.ascontiguousarray(wl.events).view(np.uint8).reshape(-1)).cuda()
    return wl, buf


def _status(fn):
    with pytest.raises(ta.TaError) as e:
        fn()
    return e.value.status


def test_call_order_is_enforced():
    wl, buf = _small()
    with ta.Window(buf, wl.win_off, wl.win_t0, wl.win_t1) as w:
        assert _status(w.correlate_launches) == TA_ERR_ORDER  # before the sort
        assert _status(w.device_overlap) == TA_ERR_ORDER
        w.sort_timeline()
        assert _status(w.sort_timeline) == TA_ERR_ORDER       # twice
        assert _status(w.attribute_operators) == TA_ERR_ORDER  # before the join
        assert _status(lambda: w.aggregate_ops(1, 1)) == TA_ERR_ORDER  # T_op before attribution
        g = w.stream_gaps(1000)
        assert _status(lambda: w.blame_gaps(g)) == TA_ERR_ORDER  # before the join
        assert _status(w.rollup_operators) == TA_ERR_ORDER
        assert _status(w.critical_path) == TA_ERR_ORDER          # before the join
        w.correlate_launches()
        assert _status(lambda: w.aggregate_ops(62, 3)) == TA_ERR_ORDER  # on-path table before the path
        assert w.critical_path().n_rows > 0
        assert w.aggregate_ops(62, 3).n_groups > 0
        assert _status(lambda: w.aggregate_ops(1, 2)) == TA_ERR_ORDER  # idle charged before the blame
        w.attribute_operators()
        w.blame_gaps(g)
        assert w.aggregate_ops(1, 2).n_groups >= 0
        assert w.rollup_operators() is not None


def test_invalid_arguments():
    wl, buf = _small()
    with ta.Window(buf, wl.win_off, wl.win_t0, wl.win_t1) as w:
        w.sort_timeline()
        assert _status(lambda: w.aggregate_ops(1, 4)) == TA_ERR_INVALID_ARG
        assert _status(lambda: w.aggregate_ops(1 << 3, 1)) == TA_ERR_INVALID_ARG  # T_op needs the OP mask
    with pytest.raises((ta.TaError, ValueError)):
        ta.Window(buf, [0, len(wl.events)], [10], [10])  # empty window span
    # the largest communicator id is reserved
    import torch
    ev = make_events([("COLL", 1, 0, 10, 20, 2**63 - 1, 0, 0), ("COLL", 2, 0, 10, 20, 2**63 - 1, 0, 0)])
    cbuf = torch.from_numpy(ev.view(np.uint8).reshape(-1)).cuda()
    assert _status(lambda: ta.Window(cbuf, [0, 2], [0], [1000])) == TA_ERR_INVALID_ARG


def test_documented_limits_return_too_large():
    import torch
    # more distinct (pid, domain, stream) triples than the lane table holds
    rows = [("KERNEL", 1, s, 10 + s, 20 + s, 0, 0, 0) for s in range(5000)]
    ev = make_events(rows)
    buf = torch.from_numpy(ev.view(np.uint8).reshape(-1)).cuda()
    assert _status(lambda: ta.Window(buf, [0, len(ev)], [0], [10**6])) == TA_ERR_TOO_LARGE
    # a window longer than 2^40 ns
    ev = make_events([("KERNEL", 1, 0, 10, 20, 0, 0, 0)])
    buf = torch.from_numpy(ev.view(np.uint8).reshape(-1)).cuda()

    def too_long():
        with ta.Window(buf, [0, 1], [0], [2**41]) as w:
            w.sort_timeline()
    assert _status(too_long) == TA_ERR_TOO_LARGE
    # windows x 2^ceil(log2(triples)) beyond 2^24: 2^21 windows and 16 streams
    W = 1 << 21
    rows = [("KERNEL", 1, s, 10, 20, 0, 0, 0) for s in range(16)]
    ev = make_events(rows)
    buf = torch.from_numpy(ev.view(np.uint8).reshape(-1)).cuda()
    off = np.full(W + 1, len(ev), dtype=np.int64)
    off[0] = 0
    assert _status(lambda: ta.Window(buf, off, np.zeros(W, dtype=np.int64),
                                     np.full(W, 1000, dtype=np.int64))) == TA_ERR_TOO_LARGE
    # 2^22 lanes (one record in each of 2^22 windows): the gap scan's lane limit
    W = 1 << 22
    ev = np.zeros(W, dtype=ta.EVENT_DTYPE)
    ev["ts_start"], ev["ts_end"], ev["pid"], ev["kind"] = 10, 20, 1, 3
    buf = torch.from_numpy(ev.view(np.uint8).reshape(-1)).cuda()

    def too_many_lanes():
        with ta.Window(buf, np.arange(W + 1, dtype=np.int64), np.zeros(W, dtype=np.int64),
                       np.full(W, 1000, dtype=np.int64)) as w:
            assert w.sort_timeline().n_lanes == W
            w.stream_gaps(1)
    assert _status(too_many_lanes) == TA_ERR_TOO_LARGE


def test_device_is_fine_after_errors():
    wl = synth.make_workload("c0", 0.1, truth=False)
    a = (wl.events, wl.win_off, wl.win_t0, wl.win_t1)
    assert_same(run_oracle(*a), run_gpu(*a))


# ---- failure paths: bounded waits and allocation failures -------------------------------
TA_ERR_OOM, TA_ERR_TIMEOUT = 2, 7


def _every_call(w, comm_sizes=()):
    """All entry points in a legal order; returns the statuses of those that fail."""
    failed = []

    def step(fn):
        try:
            return fn()
        except ta.TaError as e:
            failed.append(e.status)
            return None

    step(w.sort_timeline)
    step(w.correlate_launches)
    step(lambda: w.attribute_operators(check=False))
    g = step(lambda: w.stream_gaps(500_000))
    step(lambda: w.aggregate_ops(ta.DEVICE_KINDS, 0))
    step(lambda: w.aggregate_ops(1, 1))
    step(lambda: w.match_collectives(comm_sizes))
    step(w.device_overlap)
    step(w.rollup_operators)
    if g is not None:
        step(lambda: w.blame_gaps(g))
    step(w.critical_path)
    return failed


def test_bounded_wait_gives_up_and_the_device_stays_usable():
    """A wait on a tile descriptor that nothing ever publishes must end by itself after its
    poll limit and leave TA_ERR_TIMEOUT behind (no trap, no hang); the context stays usable."""
    assert ta.selftest_wait_timeout(3) == TA_ERR_TIMEOUT
    assert ta.selftest_wait_timeout(1000) == TA_ERR_TIMEOUT
    wl = synth.make_workload("c0", 0.1, truth=False)
    a = (wl.events, wl.win_off, wl.win_t0, wl.win_t1)
    assert_same(run_oracle(*a), run_gpu(*a))


def test_a_failed_handle_fails_every_later_call_and_frees():
    """The error word of a handle is set from the host, as a wait that gave up would set it,
    at every point of the call sequence: each later call returns that error, none faults, the
    handle frees, and the next analysis is bit-exact."""
    import torch
    wl = synth.make_workload("c1", 0.02, truth=False)
    buf = torch.from_numpy(np.ascontiguousarray(wl.events).view(np.uint8).reshape(-1)).cuda()
    for after in range(5):
        with ta.Window(buf, wl.win_off, wl.win_t0, wl.win_t1) as w:
            if after >= 1:
                w.sort_timeline()
            if after >= 2:
                w.correlate_launches()
            if after >= 3:
                w.attribute_operators()
            g = w.stream_gaps(500_000) if after >= 4 else None
            w.inject_device_error(TA_ERR_TIMEOUT)
            calls = [w.sort_timeline, w.correlate_launches, w.attribute_operators,
                     lambda: w.stream_gaps(500_000), lambda: w.aggregate_ops(ta.DEVICE_KINDS, 0),
                     lambda: w.match_collectives(wl.comm_sizes), w.device_overlap, w.critical_path,
                     w.rollup_operators]
            if g is not None:
                calls.append(lambda: w.blame_gaps(g))
            got = [_status(c) for c in calls]
            assert set(got) <= {TA_ERR_TIMEOUT, TA_ERR_ORDER}, got
            assert got.count(TA_ERR_TIMEOUT) >= (1 if after == 0 else 3), got
    torch.cuda.synchronize()
    a = (wl.events, wl.win_off, wl.win_t0, wl.win_t1)
    assert_same(run_oracle(*a, comm_sizes=wl.comm_sizes), run_gpu(*a, comm_sizes=wl.comm_sizes))


def test_waits_limited_to_one_poll_fail_cleanly_under_a_whole_analysis():
    """With the poll limit at 1 the chained scans of a window of hundreds of tiles give up
    almost at once.  Whatever each call returns must be TA_OK (every predecessor happened to
    be published in time), TA_ERR_TIMEOUT, or TA_ERR_ORDER after a failed prerequisite; a
    window that came through is bit-exact; the default limit afterwards gives a bit-exact run."""
    import torch
    wl = synth.make_workload("c1", 0.25, truth=False)
    buf = torch.from_numpy(np.ascontiguousarray(wl.events).view(np.uint8).reshape(-1)).cuda()
    ta.set_spin_limit(1)
    try:
        seen = []
        for _ in range(3):
            with ta.Window(buf, wl.win_off, wl.win_t0, wl.win_t1) as w:
                seen += _every_call(w, wl.comm_sizes)
        assert set(seen) <= {TA_ERR_TIMEOUT, TA_ERR_ORDER}, seen
    finally:
        ta.set_spin_limit(0)
    torch.cuda.synchronize()
    a = (wl.events, wl.win_off, wl.win_t0, wl.win_t1)
    assert_same(run_oracle(*a, comm_sizes=wl.comm_sizes), run_gpu(*a, comm_sizes=wl.comm_sizes))


def test_allocation_failure_at_every_request():
    """The k-th request to the caller's allocator fails, for every k of a whole analysis: the
    call in progress returns TA_ERR_OOM, ta_free hands back exactly what was handed out, and a
    run with a working allocator afterwards is bit-exact."""
    import torch
    wl = synth.make_workload("c0", 0.05, truth=False)
    buf = torch.from_numpy(np.ascontiguousarray(wl.events).view(np.uint8).reshape(-1)).cuda()
    dev = buf.device.index
    sptr = torch.cuda.current_stream(dev).cuda_stream

    class Counting:
        def __init__(self, fail_at):
            self.fail_at, self.calls, self.live = fail_at, 0, {}

        def alloc(self, nbytes):
            self.calls += 1
            if self.calls == self.fail_at:
                return None
            p = torch.cuda.caching_allocator_alloc(nbytes, dev, sptr)
            self.live[p] = nbytes
            return p

        def release(self, p):
            assert p in self.live, "released a block that was not handed out (or twice)"
            del self.live[p]
            torch.cuda.caching_allocator_delete(p)

    def run(fail_at):
        c = Counting(fail_at)
        failed = []
        try:
            w = ta.Window(buf, wl.win_off, wl.win_t0, wl.win_t1, alloc_fn=c.alloc, release_fn=c.release)
        except ta.TaError as e:
            failed.append(e.status)
        else:
            with w:
                failed += _every_call(w, wl.comm_sizes)
        assert not c.live, f"{len(c.live)} blocks not released after ta_free"
        return c.calls, failed

    total, failed = run(0)
    assert failed == [] and total > 20
    for k in range(1, total + 1):
        calls, failed = run(k)
        assert calls >= k and failed and failed[0] == TA_ERR_OOM, (k, failed)
        assert set(failed) <= {TA_ERR_OOM, TA_ERR_ORDER}, (k, failed)
    torch.cuda.synchronize()
    a = (wl.events, wl.win_off, wl.win_t0, wl.win_t1)
    assert_same(run_oracle(*a), run_gpu(*a))
