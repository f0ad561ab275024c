"""ta_lane_gaps_noalloc: the entry point for callers that cannot allocate device
memory (a resident monitoring agent in a serving process whose device heap is
fully reserved, a plug-in whose host forbids cudaMalloc in callbacks).  It keeps
its scratch in a fixed array inside the library, so its results must not depend
on what an earlier call left there.  The test calls it through the C ABI twice
in a row, on lanes of different length, and compares each result bit for bit
with what ta_stream_gaps gives for the same lane.

Collected last on purpose (file name): a run that stops at the first failure
has then already run every other test.
"""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu


def _device_lanes(w, s, g):
    dom = s.numpy("lane_domain")
    off = s.numpy("lane_off")
    lg = g.numpy("lane_gaps")
    return [(int(off[l]), int(off[l + 1]), lg[l]) for l in range(len(dom)) if dom[l] == 1]


def test_no_alloc_entry_matches_stream_gaps_on_two_calls_in_a_row():
    import torch
    from paper_2609_40247_b200 import synth, ta

    wl = synth.make_workload("c1", 0.02)
    buf = torch.from_numpy(np.ascontiguousarray(wl.events).view(np.uint8).reshape(-1)).cuda()
    with ta.Window(buf, wl.win_off, wl.win_t0, wl.win_t1) as w:
        s = w.sort_timeline()
        g = w.stream_gaps(500_000)
        ts = s.tensor("ts_start").view(torch.int64)
        te = s.tensor("ts_end").view(torch.int64)
        want_gap = g.tensor("gap_before").view(torch.int64)
        lanes = _device_lanes(w, s, g)
        assert len(lanes) >= 2
        # two lanes of different length, the longer one first: the second call must not see
        # anything of the first in the shared scratch
        lanes.sort(key=lambda x: x[0] - x[1])
        picked = [lanes[0], lanes[-1]]
        for lo, hi, want_row in picked:
            assert hi - lo <= ta.NOALLOC_MAX_RECORDS
            a = ts[lo:hi].contiguous()
            b = te[lo:hi].contiguous()
            gap, row = ta.lane_gaps_noalloc(a, b, int(wl.win_t0[0]), int(wl.win_t1[0]))
            torch.cuda.synchronize()
            assert torch.equal(gap, want_gap[lo:hi])
            for k in ta.LANE_GAPS.names:
                assert int(row[k]) == int(want_row[k]), k
            assert int(row["busy"]) + int(row["idle"]) == int(wl.win_t1[0] - wl.win_t0[0])


def test_no_alloc_entry_rejects_sizes_beyond_its_scratch():
    import torch
    from paper_2609_40247_b200 import ta

    n = ta.NOALLOC_MAX_RECORDS + 1
    a = torch.zeros(n, dtype=torch.int64, device="cuda")
    with pytest.raises(ta.TaError) as e:
        ta.lane_gaps_noalloc(a, a, 0, 1000)
    assert e.value.status == 5  # TA_ERR_TOO_LARGE
