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


def test_no_alloc_entry_on_lanes_of_many_tiles():
    """Two device lanes of 150 000 records, 74 scan tiles each (a tile is 2048 records), one
    after the other and twice over, so that the chained scan really looks back through
    descriptors in the fixed scratch and every call starts from what the one before left there.  Each call is compared
    element by element with ta_stream_gaps on the same lane; the calls are given buffers the
    caller already owns and must leave the device's free memory and torch's allocation count
    unchanged (the warm-up call pays for the module load, which does take device memory)."""
    import torch
    from paper_2609_40247_b200 import synth, ta

    wl = synth.make_workload("c0", 15.0, truth=False)
    buf = torch.from_numpy(np.ascontiguousarray(wl.events).view(np.uint8).reshape(-1)).cuda()
    with ta.Window(buf, wl.win_off, wl.win_t0, wl.win_t1) as w:
        s = w.sort_timeline()
        g = w.stream_gaps(500_000)
        ts = s.tensor("ts_start").view(torch.int64)
        te = s.tensor("ts_end").view(torch.int64)
        want_gap = g.tensor("gap_before").view(torch.int64)
        lanes = _device_lanes(w, s, g)
        lanes.sort(key=lambda x: x[0] - x[1])
        assert len(lanes) == 2 and lanes[-1][1] - lanes[-1][0] > 50 * 2048
        t0, t1 = int(wl.win_t0[0]), int(wl.win_t1[0])
        cols = [(ts[lo:hi].contiguous(), te[lo:hi].contiguous()) for lo, hi, _ in lanes]
        outs = [(torch.empty(hi - lo, dtype=torch.int64, device="cuda"),
                 torch.empty(ta.LANE_GAPS.itemsize, dtype=torch.uint8, device="cuda")) for lo, hi, _ in lanes]
        ta.lane_gaps_noalloc(cols[0][0], cols[0][1], t0, t1, gap_before=outs[0][0], lane_out=outs[0][1])
        torch.cuda.synchronize()
        L = ta.lib()
        stream = torch.cuda.current_stream().cuda_stream
        for rep in range(2):
            for (a, b), (gap, row_buf), (lo, hi, want_row) in zip(cols, outs, lanes):
                free0, alloc0 = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated()
                st = L.ta_lane_gaps_noalloc(a.data_ptr(), b.data_ptr(), hi - lo, t0, t1, gap.data_ptr(),
                                            row_buf.data_ptr(), stream)
                assert st == 0
                assert torch.cuda.mem_get_info()[0] == free0 and torch.cuda.memory_allocated() == alloc0
                assert torch.equal(gap, want_gap[lo:hi])
                row = row_buf.cpu().numpy().view(ta.LANE_GAPS)[0]
                for k in ta.LANE_GAPS.names:
                    assert int(row[k]) == int(want_row[k]), k


def test_no_alloc_entry_on_a_lane_of_exactly_the_maximum_size():
    """An ascending synthetic lane of exactly TA_NOALLOC_MAX_RECORDS records (2048 tiles: every
    descriptor of the fixed scratch is used), against ta_stream_gaps on the same records."""
    import torch
    from paper_2609_40247_b200 import ta

    n = ta.NOALLOC_MAX_RECORDS
    rng = np.random.default_rng(5)
    start = np.cumsum(rng.integers(1, 40, size=n)).astype(np.int64)
    dur = rng.integers(0, 60, size=n).astype(np.int64)
    dur[::1000] += 5000  # a few records outlive their successors: the running maximum matters
    ev = np.zeros(n, dtype=ta.EVENT_DTYPE)
    ev["ts_start"], ev["ts_end"], ev["pid"], ev["stream"], ev["kind"] = start, start + dur, 1, 3, 3
    t0, t1 = 0, int(start[-1] + 10_000)
    buf = torch.from_numpy(ev.view(np.uint8).reshape(-1)).cuda()
    with ta.Window(buf, [0, n], [t0], [t1]) as w:
        s = w.sort_timeline()
        g = w.stream_gaps(1000)
        assert s.n_lanes == 1
        ts = s.tensor("ts_start").view(torch.int64).contiguous()
        te = s.tensor("ts_end").view(torch.int64).contiguous()
        want_gap = g.tensor("gap_before").view(torch.int64)
        want_row = g.numpy("lane_gaps")[0]
        for _ in range(2):
            gap, row = ta.lane_gaps_noalloc(ts, te, t0, t1)
            assert torch.equal(gap, want_gap)
            for k in ta.LANE_GAPS.names:
                assert int(row[k]) == int(want_row[k]), k


def test_no_alloc_entry_rejects_sizes_beyond_its_scratch():
    import torch
    from paper_2609_40247_b200 import ta

    n = ta.NOALLOC_MAX_RECORDS + 1
    a = torch.zeros(n, dtype=torch.int64, device="cuda")
    with pytest.raises(ta.TaError) as e:
        ta.lane_gaps_noalloc(a, a, 0, 1000)
    assert e.value.status == 5  # TA_ERR_TOO_LARGE
