"""The byte models bench.py divides by: checked on a scaled copy of the 64 M-record workload
against the figures the mix of that workload gives by hand (a layer is 10 kernels, 10 launches,
2 collectives and 3 operators, plus one step operator and one API call per step)."""
import numpy as np

import bench
from paper_2609_40247_b200 import synth


def _mix(ev):
    n = len(ev)
    k = np.bincount(ev["kind"].astype(np.int64), minlength=6)[:6] / n
    return dict(op=k[0], api=k[1], launch=k[2], kernel=k[3], memcpy=k[4], coll=k[5])


def test_lsd_model_on_the_c3_mix():
    wl = synth.make_workload("c3", 0.01, truth=False)
    total, key_bits, passes, parts = bench.lsd_model_bytes_per_event(wl)
    # 0 window bits + 4 (16 pids) + 1 (domain) + 2 (4 streams) + 35 (30 s in ns) = 42 bits, six passes
    assert key_bits == 42 and passes == 6
    assert parts["load"] == 52.0 and parts["gather"] == 84.0 and parts["sort"] == 8.0 + 6 * 24.0
    m = _mix(wl.events)
    assert abs(m["launch"] - 0.40) < 0.01 and abs(m["kernel"] - 0.40) < 0.01 and abs(m["coll"] - 0.08) < 0.005
    f_h = m["op"] + m["api"] + m["launch"]
    f_d = m["kernel"] + m["memcpy"] + m["coll"]
    f_K = m["kernel"] + m["memcpy"]
    want = (52 + 152 + 84 + m["launch"] * 44 + f_K * 64 + f_h * 23 + f_K * 40 + m["op"] * 28 + f_d * 26
            + (2 + f_d * 24) + (2 + m["op"] * 32) + m["coll"] * 100)
    assert abs(total - want) < 1e-9
    assert 395.0 < total < 410.0  # about 400 B per record on this mix


def test_built_path_model_adds_its_parts_and_takes_the_radix_bytes_as_given():
    wl = synth.make_workload("c3", 0.01, truth=False)
    total, parts = bench.built_path_bytes_per_event(wl, 64.0)
    assert abs(total - sum(parts.values())) < 1e-9
    assert parts["radix passes"] == 64.0 and parts["discover"] == 48.0 and parts["gather"] == 92.0
    more, parts2 = bench.built_path_bytes_per_event(wl, 96.0)
    assert abs((more - total) - 32.0) < 1e-9
    # every other part depends on the kind mix only
    assert all(parts[k] == parts2[k] for k in parts if k != "radix passes")
    assert 380.0 < total < 410.0
