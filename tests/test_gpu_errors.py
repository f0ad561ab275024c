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


def test_device_is_fine_after_errors():
    wl = synth.make_workload("c0", 0.1, truth=False)
    a = (wl.events, wl.win_off, wl.win_t0, wl.win_t1)
    assert_same(run_oracle(*a), run_gpu(*a))
