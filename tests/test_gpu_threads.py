"""Handles on different host threads at the same time.  The header allows it (one handle per
thread, each on a stream of its own); the library shares three things between handles - the
page-locked staging blocks, the cache of released device blocks and the stream-ordered pool - so
the test runs different windows on four threads at once, several times over and with both
allocators, and compares every result with the oracle."""
import threading

import numpy as np
import pytest

from paper_2609_40247_b200 import synth
from runners import assert_same, run_gpu, run_oracle

pytestmark = pytest.mark.gpu

CASES = [("c0", 1.0), ("c1", 0.05), ("c2", 0.01), ("c3", 0.004)]


@pytest.mark.parametrize("torch_alloc", [False, True])
def test_four_threads_analyse_different_windows_at_once(torch_alloc):
    import torch

    work = []
    for name, scale in CASES:
        wl = synth.make_workload(name, scale, truth=False)
        args = (wl.events, wl.win_off, wl.win_t0, wl.win_t1)
        work.append((args, wl.comm_sizes, run_oracle(*args, comm_sizes=wl.comm_sizes)))
    errors = []

    def worker(k):
        try:
            torch.cuda.set_device(0)
            stream = torch.cuda.Stream()
            with torch.cuda.stream(stream):
                for rep in range(3):
                    args, sizes, want = work[(k + rep) % len(work)]
                    got = run_gpu(*args, comm_sizes=sizes, use_torch_allocator=torch_alloc)
                    assert_same(want, got)
                stream.synchronize()
        except BaseException as exc:  # reported in the main thread
            errors.append((k, exc))

    threads = [threading.Thread(target=worker, args=(k,)) for k in range(4)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    torch.cuda.synchronize()
    if errors:
        raise errors[0][1]
    # and the library is as usable afterwards as before
    args, sizes, want = work[0]
    assert_same(want, run_gpu(*args, comm_sizes=sizes, use_torch_allocator=torch_alloc))
    assert np.array_equal(want["perm"], run_gpu(*args, comm_sizes=sizes)["perm"])
