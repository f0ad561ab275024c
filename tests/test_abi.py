"""The C-ABI library loads and exports every symbol that include/ta.h declares
(no compute calls: this runs without a GPU)."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    src = open(os.path.join(ROOT, "include", "ta.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(ta_[a-z_]+)\s*\(", src)))


def test_library_exports_every_declared_symbol():
    from paper_2609_40247_b200 import build, ta
    if not os.path.exists(build.LIB):
        build.build()
    lib = ctypes.CDLL(build.LIB)
    names = declared_functions()
    assert {"ta_load_window", "ta_sort_timeline", "ta_correlate_launches", "ta_attribute_operators",
            "ta_stream_gaps", "ta_aggregate_ops", "ta_match_collectives", "ta_free"} <= set(names)
    for n in names:
        assert hasattr(lib, n), f"libta.so does not export {n}"
    assert set(ta.EXPORTS) == set(names)


def test_record_and_summary_layouts_match_the_header():
    from paper_2609_40247_b200 import ta
    assert ta.EVENT_DTYPE.itemsize == 40
    assert [ta.EVENT_DTYPE.fields[k][1] for k in
            ("ts_start", "ts_end", "corr_id", "pid", "name_id", "seq", "stream", "kind")] == \
        [0, 8, 16, 24, 28, 32, 36, 38]
    assert ta.LOAD_SUM.itemsize == 40 and ta.JOIN_SUM.itemsize == 88
    assert ta.ATTR_SUM.itemsize == 32 and ta.LANE_GAPS.itemsize == 56 and ta.LONG_GAP.itemsize == 24


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    from paper_2609_40247_b200 import ta
    monkeypatch.setattr(ta, "_lib", None)
    monkeypatch.setattr(ta, "_LIB_PATH", str(tmp_path / "nope.so"))
    try:
        ta.lib()
    except RuntimeError as e:
        assert "no CPU fallback" in str(e)
    else:
        raise AssertionError("loading a missing library must raise")


def test_arguments_are_rejected_before_any_device_work():
    """Argument checks of ta_load_window come before the first CUDA call, so they can be
    exercised here: a record count of 2^31, a window of 2^40 ns, offsets that do not end at n,
    a null handle pointer."""
    import numpy as np
    from paper_2609_40247_b200 import ta
    L = ta.lib()
    env = ta._Env()
    env.device = 0
    handle = ctypes.c_void_p()
    ev = np.zeros(4, dtype=ta.EVENT_DTYPE)
    summ = np.zeros(1, dtype=ta.LOAD_SUM)

    def load(n, off, t0, t1, hp=ctypes.byref(handle)):
        off = np.asarray(off, dtype=np.int64)
        t0 = np.asarray(t0, dtype=np.int64)
        t1 = np.asarray(t1, dtype=np.int64)
        return L.ta_load_window(ctypes.byref(env), ev.ctypes.data, n, 0, off.ctypes.data, t0.ctypes.data,
                                t1.ctypes.data, 1, summ.ctypes.data, hp)

    assert load(2**31, [0, 2**31], [0], [1000]) == 5          # TA_ERR_TOO_LARGE
    assert load(4, [0, 4], [0], [2**40]) == 5                 # window of 2^40 ns
    assert load(4, [0, 3], [0], [1000]) == 1                  # TA_ERR_INVALID_ARG: offsets end before n
    assert load(4, [0, 4], [10], [10]) == 1                   # empty window
    assert load(-1, [0, 0], [0], [10]) == 1
    assert load(4, [0, 4], [0], [1000], hp=None) == 1
    assert not handle.value
    L.ta_free(None)                                           # NULL-safe
    assert L.ta_strerror(5) and L.ta_version() > 0
    # the analyses on top of the seven calls reject a missing handle or output before any CUDA call
    out = ctypes.create_string_buffer(256)
    vp = ctypes.c_void_p
    for fn, nargs in ((L.ta_critical_path, 3), (L.ta_device_overlap, 2), (L.ta_rollup_operators, 3),
                      (L.ta_blame_gaps, 4)):
        raw = ctypes.CFUNCTYPE(ctypes.c_int, *([vp] * nargs))(ctypes.cast(fn, vp).value)
        assert raw(None, *([ctypes.addressof(out)] * (nargs - 1))) == 1
