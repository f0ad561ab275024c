"""ctypes wrapper of the CPU oracle (ta_oracle.cpp).  TEST INFRASTRUCTURE ONLY.

Used by tests/, by the smoke check and by the benchmark's CPU-baseline leg.
The product path never imports this module.  It shares no code with the CUDA
binding; the record and summary layouts are restated here on purpose.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ta_oracle.cpp")
_LIB = os.path.join(_HERE, "libta_oracle.so")

LOAD_SUM = np.dtype([(k, "<i8") for k in
                     ("n_events", "n_valid", "n_bad_kind", "n_bad_interval", "n_out_of_window")])
JOIN_SUM = np.dtype([(k, "<i8") for k in
                     ("n_probe", "n_matched", "n_unmatched", "n_launch", "n_dup_launch",
                      "n_orphan_launch", "sum_latency", "min_latency", "max_latency",
                      "sum_queue", "max_queue")])
ATTR_SUM = np.dtype([("n_attributed", "<i8"), ("n_no_launch", "<i8"), ("n_no_op", "<i8"),
                     ("max_depth", "<i4"), ("bad_nesting", "<i4")])
LANE_GAPS = np.dtype([(k, "<i8") for k in
                      ("busy", "idle", "n_events", "n_gaps", "max_gap", "first_start", "last_end")])
LONG_GAP = np.dtype([("lane", "<i4"), ("next_event", "<i4"), ("gap_start", "<i8"), ("gap_len", "<i8")])
COMM_SIZE = np.dtype([("comm_id", "<i8"), ("n_ranks", "<i4"), ("reserved", "<i4")])
SOL_SUM = np.dtype([("n_resolved", "<i8"), ("n_no_kernels", "<i8"), ("n_no_counts", "<i8"),
                    ("sum_top_ns", "<i8"), ("sum_flops", "<f8"), ("sum_bytes", "<f8"),
                    ("max_sol", "<f8")])

_DTYPES = {
    "load_sum": LOAD_SUM, "dropped": np.uint8, "win_of": np.int32,
    "perm": np.int32, "ts_start": np.int64, "ts_end": np.int64, "corr_id": np.int64,
    "pid": np.int32, "name_id": np.int32, "seq": np.int32, "stream": np.int16, "kind": np.int16,
    "win_sorted": np.int32,
    "lane_window": np.int32, "lane_pid": np.int32, "lane_stream": np.int16,
    "lane_domain": np.int16, "lane_off": np.int32,
    "launch_of": np.int32, "kernels_of_launch": np.int32, "launch_latency": np.int64,
    "queue_delay": np.int64, "join_sum": JOIN_SUM,
    "parent": np.int32, "depth": np.uint8, "op_of": np.int32, "op_n_kernels": np.int32,
    "op_first_start": np.int64, "op_last_end": np.int64, "op_kernel_ns": np.int64,
    "attr_sum": ATTR_SUM,
    "gap_before": np.int64, "lane_gaps": LANE_GAPS, "lane_hist": np.uint32, "win_hist": np.uint32,
    "long_gaps": LONG_GAP,
    "g_window": np.int32, "g_pid": np.int32, "g_name": np.int32, "g_count": np.int64,
    "g_sum": np.int64, "g_min": np.int64, "g_max": np.int64, "g_hist": np.uint32,
    "c_window": np.int32, "c_comm": np.int64, "c_seq": np.int32, "c_n_members": np.int32,
    "c_min_start": np.int64, "c_max_start": np.int64, "c_skew": np.int64, "c_max_end": np.int64,
    "c_straggler_pid": np.int32, "c_flags": np.int32, "wait_ns": np.int64,
    "r_window": np.int32, "r_pid": np.int32, "r_n_coll": np.int64, "r_sum_wait": np.int64,
    "r_max_wait": np.int64, "r_n_straggler": np.int64,
    "incl_n_kernels": np.int32, "incl_first_start": np.int64, "incl_last_end": np.int64,
    "incl_kernel_ns": np.int64, "replay_first_start": np.int64, "replay_last_end": np.int64,
    "replay_kernel_ns": np.int64, "roll_sum": np.int64,
    "b_class": np.int32, "b_launch": np.int32, "b_win_count": np.int64, "b_win_ns": np.int64,
    "op_gap_ns": np.int64,
    "d_window": np.int32, "d_pid": np.int32, "d_n_events": np.int64, "d_busy": np.int64,
    "d_idle": np.int64, "d_compute": np.int64, "d_comm": np.int64, "d_overlap": np.int64,
    "d_exposed": np.int64,
    "on_path": np.uint8, "cp_window": np.int32, "cp_pid": np.int32, "cp_sink": np.int32,
    "cp_n_nodes": np.int32, "cp_reason": np.int32, "cp_begin": np.int64, "cp_end": np.int64,
    "cp_ns": np.int64, "cp_sum": np.int64,
    "sol_mfu": np.float64, "sol_mbu": np.float64, "sol_op": np.float64, "sol_state": np.uint8,
    "sol_sum": SOL_SUM,
}

_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with g++ -O2 (in-tree); returns the library path."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        subprocess.check_call(
            ["g++", "-O2", "-std=c++17", "-shared", "-fPIC", _SRC, "-o", _LIB + ".tmp"])
        os.replace(_LIB + ".tmp", _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.orc_create.restype = ctypes.c_void_p
        lib.orc_create.argtypes = [ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p,
                                   ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int32]
        lib.orc_destroy.argtypes = [ctypes.c_void_p]
        for f in ("orc_load", "orc_sort", "orc_correlate"):
            getattr(lib, f).argtypes = [ctypes.c_void_p]
            getattr(lib, f).restype = None
        lib.orc_attribute.argtypes = [ctypes.c_void_p]
        lib.orc_attribute.restype = ctypes.c_int32
        lib.orc_gaps.argtypes = [ctypes.c_void_p, ctypes.c_int64]
        lib.orc_gaps.restype = None
        lib.orc_aggregate.argtypes = [ctypes.c_void_p, ctypes.c_uint32, ctypes.c_int32]
        lib.orc_aggregate.restype = ctypes.c_int32
        lib.orc_collectives.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int32]
        lib.orc_collectives.restype = None
        lib.orc_device_overlap.argtypes = [ctypes.c_void_p]
        lib.orc_device_overlap.restype = None
        lib.orc_blame.argtypes = [ctypes.c_void_p]
        lib.orc_blame.restype = None
        lib.orc_rollup.argtypes = [ctypes.c_void_p]
        lib.orc_rollup.restype = None
        lib.orc_critical_path.argtypes = [ctypes.c_void_p]
        lib.orc_critical_path.restype = None
        lib.orc_sol.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_double,
                                ctypes.c_double]
        lib.orc_sol.restype = None
        lib.orc_n_valid.argtypes = [ctypes.c_void_p]
        lib.orc_n_valid.restype = ctypes.c_int64
        lib.orc_get.argtypes = [ctypes.c_void_p, ctypes.c_char_p, ctypes.POINTER(ctypes.c_void_p),
                                ctypes.POINTER(ctypes.c_int64), ctypes.POINTER(ctypes.c_int32)]
        lib.orc_get.restype = ctypes.c_int32
        _lib = lib
    return _lib


class Oracle:
    """One analysis of one batch of windows; methods mirror the seven steps."""

    def __init__(self, events: np.ndarray, win_off, win_t0, win_t1):
        lib = _load()
        ev = np.ascontiguousarray(events)
        assert ev.dtype.itemsize == 40
        self._off = np.ascontiguousarray(win_off, dtype=np.int64)
        self._t0 = np.ascontiguousarray(win_t0, dtype=np.int64)
        self._t1 = np.ascontiguousarray(win_t1, dtype=np.int64)
        self.W = len(self._t0)
        self.n = len(ev)
        assert len(self._off) == self.W + 1 and self._off[0] == 0 and self._off[-1] == self.n
        self._lib = lib
        self._h = lib.orc_create(ev.ctypes.data, self.n, self._off.ctypes.data,
                                 self._t0.ctypes.data, self._t1.ctypes.data, self.W)

    def close(self):
        if self._h:
            self._lib.orc_destroy(self._h)
            self._h = None

    def __del__(self):
        self.close()

    def get(self, name: str) -> np.ndarray:
        ptr = ctypes.c_void_p()
        cnt = ctypes.c_int64()
        el = ctypes.c_int32()
        if self._lib.orc_get(self._h, name.encode(), ctypes.byref(ptr), ctypes.byref(cnt),
                             ctypes.byref(el)) != 0:
            raise KeyError(name)
        dt = np.dtype(_DTYPES[name])
        assert dt.itemsize == el.value, (name, dt.itemsize, el.value)
        if cnt.value == 0:
            out = np.empty(0, dtype=dt)
        else:
            buf = (ctypes.c_char * (cnt.value * el.value)).from_address(ptr.value)
            out = np.frombuffer(buf, dtype=dt).copy()
        if name in ("lane_hist", "win_hist", "g_hist"):
            out = out.reshape(-1, 40)
        if name in ("b_win_count", "b_win_ns"):
            out = out.reshape(-1, 4)
        if name == "roll_sum":
            out = out.reshape(-1, 3)
        return out

    @property
    def n_valid(self) -> int:
        return int(self._lib.orc_n_valid(self._h))

    def load(self):
        self._lib.orc_load(self._h)
        return self.get("load_sum")

    def sort(self):
        self._lib.orc_sort(self._h)

    def correlate(self):
        self._lib.orc_correlate(self._h)
        return self.get("join_sum")

    def attribute(self) -> int:
        """Returns 0, 8 (depth) or 9 (bad nesting), the analyzer's status codes."""
        return int(self._lib.orc_attribute(self._h))

    def gaps(self, min_gap_ns: int):
        self._lib.orc_gaps(self._h, int(min_gap_ns))

    def aggregate(self, kind_mask: int, value_sel: int) -> int:
        return int(self._lib.orc_aggregate(self._h, kind_mask, value_sel))

    def collectives(self, comm_sizes=()):
        arr = np.zeros(len(comm_sizes), dtype=COMM_SIZE)
        for i, (cid, nr) in enumerate(comm_sizes):
            arr[i] = (cid, nr, 0)
        self._sizes = arr
        self._lib.orc_collectives(self._h, arr.ctypes.data if len(arr) else None, len(arr))

    def rollup(self):
        """Inclusive per-operator kernel figures and graph replays (needs attribute() == 0)."""
        self._lib.orc_rollup(self._h)

    def blame(self):
        """Classifies the long gaps of the last gaps() call and charges them to the operators
        they coincide with (needs correlate() and gaps())."""
        self._lib.orc_blame(self._h)

    def device_overlap(self):
        """Per (window, process): busy / idle over all device streams, compute and
        communication coverage, their overlap and the exposed communication (needs sort())."""
        self._lib.orc_device_overlap(self._h)

    def critical_path(self):
        """Per (window, process): the chain of binding submission, stream-order, program-order
        and synchronisation dependencies that ends at the last record to finish, and the split
        of its length into eight classes (needs correlate())."""
        self._lib.orc_critical_path(self._h)

    def sol(self, flops, bytes_, peak_flops: float, peak_bw: float):
        """MFU, MBU and SOL_op = max(MFU, MBU) of every operator invocation from its T_op, the
        operation count and data volume given per INPUT record (float64, negative or NaN =
        not known) and the device peaks in FLOP/s and B/s (needs attribute() == 0)."""
        f = np.ascontiguousarray(flops, dtype=np.float64)
        b = np.ascontiguousarray(bytes_, dtype=np.float64)
        assert len(f) == self.n and len(b) == self.n
        self._lib.orc_sol(self._h, f.ctypes.data, b.ctypes.data, float(peak_flops), float(peak_bw))

    def run_all(self, min_gap_ns: int = 500_000, comm_sizes=()):
        """load, sort, correlate, attribute, gaps, collectives; returns attribute's status."""
        self.load()
        self.sort()
        self.correlate()
        st = self.attribute()
        self.gaps(min_gap_ns)
        self.collectives(comm_sizes)
        return st
