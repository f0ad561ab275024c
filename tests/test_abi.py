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
