"""Python binding of the C ABI in include/ta.h (argument marshalling only).

Every step runs in the CUDA library (libta.so, built by
`python -m paper_2609_40247_b200.build`); PyTorch supplies device memory (its
caching allocator, through the ta_env callbacks) and the stream.  There is no
CPU fallback: if the library is missing, loading fails with an error.

    with ta.Window(events_u8_cuda, win_off, t0, t1) as w:
        s = w.sort_timeline();  j = w.correlate_launches();  a = w.attribute_operators()
        g = w.stream_gaps(500_000);  k = w.aggregate_ops(ta.DEVICE_KINDS, 0)
        c = w.match_collectives([(comm_id, n_ranks), ...])
"""
from __future__ import annotations

import ctypes
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libta.so")

KIND_OP, KIND_API, KIND_LAUNCH, KIND_KERNEL, KIND_MEMCPY, KIND_COLL = range(6)
DEVICE_KINDS = (1 << KIND_KERNEL) | (1 << KIND_MEMCPY) | (1 << KIND_COLL)
NBINS = 40

STATUS_NAMES = ["TA_OK", "TA_ERR_INVALID_ARG", "TA_ERR_OOM", "TA_ERR_CUDA", "TA_ERR_ORDER",
                "TA_ERR_TOO_LARGE", "TA_ERR_OVERFLOW", "TA_ERR_TIMEOUT", "TA_ERR_DEPTH",
                "TA_ERR_BAD_NESTING"]
TA_ERR_DEPTH, TA_ERR_BAD_NESTING = 8, 9

EVENT_DTYPE = np.dtype([("ts_start", "<i8"), ("ts_end", "<i8"), ("corr_id", "<i8"), ("pid", "<i4"),
                        ("name_id", "<i4"), ("seq", "<i4"), ("stream", "<i2"), ("kind", "<i2")])
LOAD_SUM = np.dtype([(k, "<i8") for k in
                     ("n_events", "n_valid", "n_bad_kind", "n_bad_interval", "n_out_of_window")])
JOIN_SUM = np.dtype([(k, "<i8") for k in
                     ("n_probe", "n_matched", "n_unmatched", "n_launch", "n_dup_launch",
                      "n_orphan_launch", "sum_latency", "min_latency", "max_latency", "sum_queue",
                      "max_queue")])
ATTR_SUM = np.dtype([("n_attributed", "<i8"), ("n_no_launch", "<i8"), ("n_no_op", "<i8"),
                     ("max_depth", "<i4"), ("bad_nesting", "<i4")])
LANE_GAPS = np.dtype([(k, "<i8") for k in
                      ("busy", "idle", "n_events", "n_gaps", "max_gap", "first_start", "last_end")])
LONG_GAP = np.dtype([("lane", "<i4"), ("next_event", "<i4"), ("gap_start", "<i8"), ("gap_len", "<i8")])
COMM_SIZE = np.dtype([("comm_id", "<i8"), ("n_ranks", "<i4"), ("reserved", "<i4")])

_vp = ctypes.c_void_p
_ALLOC_T = ctypes.CFUNCTYPE(ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p)
_RELEASE_T = ctypes.CFUNCTYPE(None, ctypes.c_void_p, ctypes.c_void_p)


class _Env(ctypes.Structure):
    _fields_ = [("alloc", _ALLOC_T), ("release", _RELEASE_T), ("ctx", _vp), ("cuda_stream", _vp),
                ("device", ctypes.c_int32)]


def _ptr_struct(name, fields):
    return type(name, (ctypes.Structure,), {"_fields_": fields})


_SortResult = _ptr_struct("_SortResult", [
    ("n", ctypes.c_int64), ("n_valid", ctypes.c_int64), ("n_lanes", ctypes.c_int32),
    ("n_windows", ctypes.c_int32), ("perm", _vp), ("ts_start", _vp), ("ts_end", _vp),
    ("corr_id", _vp), ("pid", _vp), ("name_id", _vp), ("seq", _vp), ("stream", _vp), ("kind", _vp),
    ("lane_window", _vp), ("lane_pid", _vp), ("lane_stream", _vp), ("lane_domain", _vp),
    ("lane_off", _vp)])
_JoinResult = _ptr_struct("_JoinResult", [
    ("launch_of", _vp), ("launch_latency", _vp), ("queue_delay", _vp), ("kernels_of_launch", _vp)])
_AttrResult = _ptr_struct("_AttrResult", [
    ("parent", _vp), ("depth", _vp), ("op_of", _vp), ("op_first_start", _vp), ("op_last_end", _vp),
    ("op_kernel_ns", _vp), ("op_n_kernels", _vp)])
_GapResult = _ptr_struct("_GapResult", [
    ("gap_before", _vp), ("lane_gaps", _vp), ("lane_hist", _vp), ("win_hist", _vp),
    ("long_gaps", _vp), ("n_long_gaps", ctypes.c_int64)])
_AggResult = _ptr_struct("_AggResult", [
    ("n_groups", ctypes.c_int64), ("g_window", _vp), ("g_pid", _vp), ("g_name", _vp),
    ("g_count", _vp), ("g_sum", _vp), ("g_min", _vp), ("g_max", _vp), ("g_hist", _vp)])
_CollResult = _ptr_struct("_CollResult", [
    ("n_groups", ctypes.c_int64), ("n_ranks", ctypes.c_int64), ("g_window", _vp), ("g_comm", _vp),
    ("g_seq", _vp), ("g_n_members", _vp), ("g_min_start", _vp), ("g_max_start", _vp),
    ("g_skew", _vp), ("g_max_end", _vp), ("g_straggler_pid", _vp), ("g_flags", _vp),
    ("wait_ns", _vp), ("r_window", _vp), ("r_pid", _vp), ("r_n_coll", _vp), ("r_sum_wait", _vp),
    ("r_max_wait", _vp), ("r_n_straggler", _vp)])
_RollupResult = _ptr_struct("_RollupResult", [
    ("incl_n_kernels", _vp), ("incl_first_start", _vp), ("incl_last_end", _vp), ("incl_kernel_ns", _vp),
    ("replay_first_start", _vp), ("replay_last_end", _vp), ("replay_kernel_ns", _vp)])
_BlameResult = _ptr_struct("_BlameResult", [
    ("n_long_gaps", ctypes.c_int64), ("g_class", _vp), ("g_launch", _vp), ("op_gap_ns", _vp)])
_SolResult = _ptr_struct("_SolResult", [("mfu", _vp), ("mbu", _vp), ("sol", _vp), ("state", _vp)])
_OverlapResult = _ptr_struct("_OverlapResult", [
    ("n_rows", ctypes.c_int64), ("d_window", _vp), ("d_pid", _vp), ("d_n_events", _vp),
    ("d_busy", _vp), ("d_idle", _vp), ("d_compute", _vp), ("d_comm", _vp), ("d_overlap", _vp),
    ("d_exposed", _vp)])

_CritpathResult = _ptr_struct("_CritpathResult", [
    ("n_rows", ctypes.c_int64), ("on_path", _vp), ("p_window", _vp), ("p_pid", _vp), ("p_sink", _vp),
    ("p_n_nodes", _vp), ("p_reason", _vp), ("p_begin", _vp), ("p_end", _vp), ("p_ns", _vp)])

EXPORTS = ["ta_load_window", "ta_sort_timeline", "ta_correlate_launches", "ta_attribute_operators",
           "ta_stream_gaps", "ta_aggregate_ops", "ta_match_collectives", "ta_free", "ta_strerror",
           "ta_version", "ta_launch_count", "ta_profile_enable", "ta_profile_radix",
           "ta_lane_gaps_noalloc", "ta_device_overlap", "ta_blame_gaps",
           "ta_rollup_operators", "ta_critical_path", "ta_set_spin_limit",
           "ta_selftest_wait_timeout", "ta_inject_device_error", "ta_operator_sol"]
NOALLOC_MAX_RECORDS = 1 << 22

_lib = None


class TaError(RuntimeError):
    def __init__(self, status, where):
        self.status = status
        name = STATUS_NAMES[status] if 0 <= status < len(STATUS_NAMES) else str(status)
        super().__init__(f"{where}: {name}")


def lib():
    """Loads libta.so; raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise RuntimeError(
                f"{_LIB_PATH} is missing: build it with `python -m paper_2609_40247_b200.build` "
                "(nvcc, sm_100a). The analyzer has no CPU fallback.")
        L = ctypes.CDLL(_LIB_PATH)
        L.ta_load_window.restype = ctypes.c_int
        L.ta_load_window.argtypes = [ctypes.POINTER(_Env), _vp, ctypes.c_int64, ctypes.c_int32, _vp,
                                     _vp, _vp, ctypes.c_int32, _vp, ctypes.POINTER(_vp)]
        L.ta_sort_timeline.restype = ctypes.c_int
        L.ta_sort_timeline.argtypes = [_vp, ctypes.POINTER(_SortResult)]
        L.ta_correlate_launches.restype = ctypes.c_int
        L.ta_correlate_launches.argtypes = [_vp, ctypes.POINTER(_JoinResult), _vp]
        L.ta_attribute_operators.restype = ctypes.c_int
        L.ta_attribute_operators.argtypes = [_vp, ctypes.POINTER(_AttrResult), _vp]
        L.ta_stream_gaps.restype = ctypes.c_int
        L.ta_stream_gaps.argtypes = [_vp, ctypes.c_int64, ctypes.POINTER(_GapResult)]
        L.ta_aggregate_ops.restype = ctypes.c_int
        L.ta_aggregate_ops.argtypes = [_vp, ctypes.c_uint32, ctypes.c_int32, ctypes.POINTER(_AggResult)]
        L.ta_match_collectives.restype = ctypes.c_int
        L.ta_match_collectives.argtypes = [_vp, _vp, ctypes.c_int32, ctypes.POINTER(_CollResult)]
        L.ta_rollup_operators.restype = ctypes.c_int
        L.ta_rollup_operators.argtypes = [_vp, ctypes.POINTER(_RollupResult), _vp]
        L.ta_critical_path.restype = ctypes.c_int
        L.ta_critical_path.argtypes = [_vp, ctypes.POINTER(_CritpathResult), _vp]
        L.ta_blame_gaps.restype = ctypes.c_int
        L.ta_blame_gaps.argtypes = [_vp, _vp, ctypes.POINTER(_BlameResult), _vp]
        L.ta_operator_sol.restype = ctypes.c_int
        L.ta_operator_sol.argtypes = [_vp, _vp, _vp, ctypes.c_int32, ctypes.c_double, ctypes.c_double,
                                      ctypes.POINTER(_SolResult), _vp]
        L.ta_device_overlap.restype = ctypes.c_int
        L.ta_device_overlap.argtypes = [_vp, ctypes.POINTER(_OverlapResult)]
        L.ta_free.restype = None
        L.ta_free.argtypes = [_vp]
        L.ta_strerror.restype = ctypes.c_char_p
        L.ta_strerror.argtypes = [ctypes.c_int]
        L.ta_version.restype = ctypes.c_int32
        L.ta_lane_gaps_noalloc.restype = ctypes.c_int
        L.ta_lane_gaps_noalloc.argtypes = [_vp, _vp, ctypes.c_int64, ctypes.c_int64, ctypes.c_int64,
                                           _vp, _vp, _vp]
        L.ta_launch_count.restype = ctypes.c_int64
        L.ta_set_spin_limit.restype = None
        L.ta_set_spin_limit.argtypes = [ctypes.c_int32]
        L.ta_inject_device_error.restype = ctypes.c_int
        L.ta_inject_device_error.argtypes = [_vp, ctypes.c_int]
        L.ta_selftest_wait_timeout.restype = ctypes.c_int
        L.ta_selftest_wait_timeout.argtypes = [_vp, ctypes.c_int32]
        L.ta_profile_enable.restype = None
        L.ta_profile_enable.argtypes = [ctypes.c_int32]
        L.ta_profile_radix.restype = ctypes.c_int32
        L.ta_profile_radix.argtypes = [ctypes.POINTER(ctypes.c_int64), ctypes.POINTER(ctypes.c_double),
                                       ctypes.POINTER(ctypes.c_double)]
        _lib = L
    return _lib


def lane_gaps_noalloc(ts_start, ts_end, win_t0: int, win_t1: int, gap_before=None, lane_out=None,
                      stream=None):
    """Gap scan of one device lane through ta_lane_gaps_noalloc, the entry point for
    callers that may not allocate device memory: the library call itself allocates
    nothing (its scratch is a fixed array inside libta.so).  The output buffers are
    the caller's; pass `gap_before` (int64, n) and `lane_out` (uint8, 56 bytes) to
    reuse buffers you already own, otherwise this wrapper creates them with torch.
    Inputs: int64 CUDA tensors of one lane in canonical order.  Calls must not
    overlap on the GPU (they share the scratch array); at most NOALLOC_MAX_RECORDS
    records.  Returns (gap_before tensor, lane summary as a LANE_GAPS numpy record)."""
    import torch
    L = lib()
    if not (ts_start.is_cuda and ts_end.is_cuda and ts_start.dtype == torch.int64
            and ts_end.dtype == torch.int64 and ts_start.is_contiguous() and ts_end.is_contiguous()):
        raise ValueError("ts_start / ts_end must be contiguous int64 CUDA tensors")
    n = ts_start.numel()
    if ts_end.numel() != n:
        raise ValueError("ts_start and ts_end differ in length")
    dev = ts_start.device
    if gap_before is None:
        gap_before = torch.empty(max(n, 1), dtype=torch.int64, device=dev)
    if lane_out is None:
        lane_out = torch.empty(LANE_GAPS.itemsize, dtype=torch.uint8, device=dev)
    s = stream if stream is not None else torch.cuda.current_stream(dev)
    with torch.cuda.device(dev):
        st = L.ta_lane_gaps_noalloc(ts_start.data_ptr(), ts_end.data_ptr(), n, int(win_t0), int(win_t1),
                                    gap_before.data_ptr(), lane_out.data_ptr(), s.cuda_stream)
    if st != 0:
        raise TaError(st, "ta_lane_gaps_noalloc")
    return gap_before[:n], lane_out.cpu().numpy().view(LANE_GAPS)[0]


def launch_count() -> int:
    """Kernels launched by the library since it was loaded."""
    return int(lib().ta_launch_count())


def set_spin_limit(polls: int) -> None:
    """Poll limit of the device-side waits of windows created from now on (0 = default)."""
    lib().ta_set_spin_limit(int(polls))


def selftest_wait_timeout(polls: int, stream=None) -> int:
    """Runs a wait that nothing ever ends, limited to `polls` polls; returns the status the
    kernel recorded (7 = TA_ERR_TIMEOUT when the bounded wait works)."""
    import torch
    s = stream if stream is not None else torch.cuda.current_stream()
    return int(lib().ta_selftest_wait_timeout(s.cuda_stream, int(polls)))


def profile_enable(on: bool) -> None:
    """Start (and reset) / stop the CUDA-event timing of the radix-sort passes."""
    lib().ta_profile_enable(1 if on else 0)


def profile_radix():
    """(number of radix passes timed, their summed duration in ms, algorithmic bytes moved)."""
    n = ctypes.c_int64()
    ms = ctypes.c_double()
    nb = ctypes.c_double()
    if lib().ta_profile_radix(ctypes.byref(n), ctypes.byref(ms), ctypes.byref(nb)) != 0:
        raise RuntimeError("ta_profile_radix: CUDA error")
    return n.value, ms.value, nb.value


class _DevView:
    """Exposes a raw device range to torch through __cuda_array_interface__."""

    def __init__(self, ptr, nbytes, owner):
        self.owner = owner
        self.__cuda_array_interface__ = {"shape": (nbytes,), "typestr": "|u1",
                                         "data": (int(ptr), False), "version": 2}


class _Result:
    """Device pointers owned by the window handle, with typed access."""
    _layout: dict = {}

    def __init__(self, window, raw, extra=None):
        self._w = window
        self._raw = raw
        self.__dict__.update(extra or {})

    def _spec(self, name):
        dt, count = self._layout[name]
        cnt = count(self) if callable(count) else count
        return np.dtype(dt), int(cnt)

    def tensor(self, name):
        """Zero-copy torch view (uint8 for struct arrays) of a device result; valid while
        the window is open."""
        import torch
        dt, cnt = self._spec(name)
        ptr = getattr(self._raw, name)
        nbytes = cnt * dt.itemsize
        if nbytes == 0 or not ptr:
            return torch.empty(0, dtype=torch.uint8, device=f"cuda:{self._w.device}")
        return torch.as_tensor(_DevView(ptr, nbytes, self._w), device=f"cuda:{self._w.device}")

    def numpy(self, name):
        if name in self.__dict__ and isinstance(self.__dict__[name], np.ndarray):
            return self.__dict__[name]
        dt, cnt = self._spec(name)
        if cnt == 0:
            out = np.empty(0, dtype=dt)
        else:
            import torch
            with torch.cuda.stream(self._w.torch_stream):
                out = self.tensor(name).cpu().numpy().view(dt).copy()
        if name.endswith("_hist"):
            out = out.reshape(-1, NBINS)
        return out


class SortResult(_Result):
    _layout = {
        "perm": ("<i4", lambda r: r.n), "ts_start": ("<i8", lambda r: r.n),
        "ts_end": ("<i8", lambda r: r.n), "corr_id": ("<i8", lambda r: r.n),
        "pid": ("<i4", lambda r: r.n), "name_id": ("<i4", lambda r: r.n),
        "seq": ("<i4", lambda r: r.n), "stream": ("<i2", lambda r: r.n),
        "kind": ("<i2", lambda r: r.n),
        "lane_window": ("<i4", lambda r: r.n_lanes), "lane_pid": ("<i4", lambda r: r.n_lanes),
        "lane_stream": ("<i2", lambda r: r.n_lanes), "lane_domain": ("<i2", lambda r: r.n_lanes),
        "lane_off": ("<i4", lambda r: r.n_lanes + 1),
    }


class JoinResult(_Result):
    _layout = {"launch_of": ("<i4", lambda r: r.n), "launch_latency": ("<i8", lambda r: r.n),
               "queue_delay": ("<i8", lambda r: r.n), "kernels_of_launch": ("<i4", lambda r: r.n)}


class AttrResult(_Result):
    _layout = {"parent": ("<i4", lambda r: r.n), "depth": ("|u1", lambda r: r.n),
               "op_of": ("<i4", lambda r: r.n), "op_first_start": ("<i8", lambda r: r.n),
               "op_last_end": ("<i8", lambda r: r.n), "op_kernel_ns": ("<i8", lambda r: r.n),
               "op_n_kernels": ("<i4", lambda r: r.n)}


class GapResult(_Result):
    _layout = {"gap_before": ("<i8", lambda r: r.n), "lane_gaps": (LANE_GAPS, lambda r: r.n_lanes),
               "lane_hist": ("<u4", lambda r: r.n_lanes * NBINS),
               "win_hist": ("<u4", lambda r: r.n_windows * NBINS),
               "long_gaps": (LONG_GAP, lambda r: r.n_long_gaps)}


class AggResult(_Result):
    _layout = {"g_window": ("<i4", lambda r: r.n_groups), "g_pid": ("<i4", lambda r: r.n_groups),
               "g_name": ("<i4", lambda r: r.n_groups), "g_count": ("<i8", lambda r: r.n_groups),
               "g_sum": ("<i8", lambda r: r.n_groups), "g_min": ("<i8", lambda r: r.n_groups),
               "g_max": ("<i8", lambda r: r.n_groups),
               "g_hist": ("<u4", lambda r: r.n_groups * NBINS)}


class CollResult(_Result):
    _names = {"c_window": "g_window", "c_comm": "g_comm", "c_seq": "g_seq",
              "c_n_members": "g_n_members", "c_min_start": "g_min_start",
              "c_max_start": "g_max_start", "c_skew": "g_skew", "c_max_end": "g_max_end",
              "c_straggler_pid": "g_straggler_pid", "c_flags": "g_flags"}
    _layout = {"g_window": ("<i4", lambda r: r.n_groups), "g_comm": ("<i8", lambda r: r.n_groups),
               "g_seq": ("<i4", lambda r: r.n_groups), "g_n_members": ("<i4", lambda r: r.n_groups),
               "g_min_start": ("<i8", lambda r: r.n_groups),
               "g_max_start": ("<i8", lambda r: r.n_groups), "g_skew": ("<i8", lambda r: r.n_groups),
               "g_max_end": ("<i8", lambda r: r.n_groups),
               "g_straggler_pid": ("<i4", lambda r: r.n_groups),
               "g_flags": ("<i4", lambda r: r.n_groups), "wait_ns": ("<i8", lambda r: r.n),
               "r_window": ("<i4", lambda r: r.n_ranks), "r_pid": ("<i4", lambda r: r.n_ranks),
               "r_n_coll": ("<i8", lambda r: r.n_ranks), "r_sum_wait": ("<i8", lambda r: r.n_ranks),
               "r_max_wait": ("<i8", lambda r: r.n_ranks),
               "r_n_straggler": ("<i8", lambda r: r.n_ranks)}

    def numpy(self, name):
        return super().numpy(self._names.get(name, name))

    def tensor(self, name):
        return super().tensor(self._names.get(name, name))


ROLLUP_SUM = np.dtype([(k, "<i8") for k in ("n_graph_launches", "n_graph_kernels",
                                            "max_kernels_per_launch")])


class RollupResult(_Result):
    _layout = dict([("incl_n_kernels", ("<i4", lambda r: r.n))] +
                   [(k, ("<i8", lambda r: r.n)) for k in
                    ("incl_first_start", "incl_last_end", "incl_kernel_ns", "replay_first_start",
                     "replay_last_end", "replay_kernel_ns")])

    def numpy(self, name):
        if name == "roll_sum":
            s = self.rollup_sum
            return np.stack([s["n_graph_launches"], s["n_graph_kernels"], s["max_kernels_per_launch"]],
                            axis=1).astype(np.int64)
        return super().numpy(name)


CRITPATH_SUM = np.dtype([("n_paths", "<i8"), ("n_nodes", "<i8"), ("ns", "<i8", (8,))])


class CritpathResult(_Result):
    """on_path per sorted position; one row per (window, process): cp_window, cp_pid, cp_sink,
    cp_n_nodes, cp_reason, cp_begin, cp_end, cp_ns[row][8]; cp_sum[window][10] = paths, nodes and
    the eight class totals."""
    _names = {"cp_window": "p_window", "cp_pid": "p_pid", "cp_sink": "p_sink", "cp_n_nodes": "p_n_nodes",
              "cp_reason": "p_reason", "cp_begin": "p_begin", "cp_end": "p_end", "cp_ns": "p_ns"}
    _layout = dict([("on_path", ("u1", lambda r: r.n))] +
                   [(k, ("<i4", lambda r: r.n_rows)) for k in
                    ("p_window", "p_pid", "p_sink", "p_n_nodes", "p_reason")] +
                   [("p_begin", ("<i8", lambda r: r.n_rows)), ("p_end", ("<i8", lambda r: r.n_rows)),
                    ("p_ns", ("<i8", lambda r: r.n_rows * 8))])

    def numpy(self, name):
        if name == "cp_sum":
            s = self.critpath_sum
            return np.concatenate([s["n_paths"][:, None], s["n_nodes"][:, None], s["ns"]],
                                  axis=1).astype(np.int64).reshape(-1)
        return super().numpy(self._names.get(name, name))

    def tensor(self, name):
        return super().tensor(self._names.get(name, name))


BLAME_SUM = np.dtype([("count", "<i8", (4,)), ("ns", "<i8", (4,))])


class BlameResult(_Result):
    _names = {"b_class": "g_class", "b_launch": "g_launch"}
    _layout = {"g_class": ("<i4", lambda r: r.n_long_gaps), "g_launch": ("<i4", lambda r: r.n_long_gaps),
               "op_gap_ns": ("<i8", lambda r: r.n)}

    def numpy(self, name):
        if name == "b_win_count":
            return self.blame_sum["count"].astype(np.int64).reshape(-1, 4)
        if name == "b_win_ns":
            return self.blame_sum["ns"].astype(np.int64).reshape(-1, 4)
        return super().numpy(self._names.get(name, name))

    def tensor(self, name):
        return super().tensor(self._names.get(name, name))


SOL_SUM = np.dtype([("n_resolved", "<i8"), ("n_no_kernels", "<i8"), ("n_no_counts", "<i8"),
                    ("sum_top_ns", "<i8"), ("sum_flops", "<f8"), ("sum_bytes", "<f8"),
                    ("max_sol", "<f8")])


class SolResult(_Result):
    """Per sorted position: sol_mfu, sol_mbu, sol_op (float64), sol_state (uint8); sol_sum per
    window (SOL_SUM)."""
    _names = {"sol_mfu": "mfu", "sol_mbu": "mbu", "sol_op": "sol", "sol_state": "state"}
    _layout = {"mfu": ("<f8", lambda r: r.n), "mbu": ("<f8", lambda r: r.n),
               "sol": ("<f8", lambda r: r.n), "state": ("|u1", lambda r: r.n)}

    def numpy(self, name):
        if name == "sol_sum":
            return self.sol_sum
        return super().numpy(self._names.get(name, name))

    def tensor(self, name):
        return super().tensor(self._names.get(name, name))


class OverlapResult(_Result):
    _layout = dict([("d_window", ("<i4", lambda r: r.n_rows)), ("d_pid", ("<i4", lambda r: r.n_rows))] +
                   [(k, ("<i8", lambda r: r.n_rows)) for k in
                    ("d_n_events", "d_busy", "d_idle", "d_compute", "d_comm", "d_overlap", "d_exposed")])


class Window:
    """One analysis handle (ta_window).  `events`: a CUDA tensor holding n 40-byte
    records (any dtype, contiguous) - borrowed until sort_timeline() returns - or a
    host numpy array of EVENT_DTYPE (copied to the device by the library)."""

    def __init__(self, events, win_off, win_t0, win_t1, device=None, stream=None,
                 use_torch_allocator=True, alloc_fn=None, release_fn=None):
        """alloc_fn(nbytes) -> device address or None, release_fn(address): replace torch's
        caching allocator behind the ta_env callbacks (both or neither)."""
        import torch
        L = lib()
        self._lib = L
        self._h = _vp()
        on_device = hasattr(events, "is_cuda")
        if on_device:
            if not events.is_cuda or not events.is_contiguous():
                raise ValueError("events tensor must be a contiguous CUDA tensor")
            nbytes = events.numel() * events.element_size()
            ev_ptr = events.data_ptr()
            device = events.device.index if device is None else device
        else:
            events = np.ascontiguousarray(events)
            nbytes = events.nbytes
            ev_ptr = events.ctypes.data
            device = torch.cuda.current_device() if device is None else device
        if nbytes % 40:
            raise ValueError("events must hold whole 40-byte records")
        self.n = nbytes // 40
        self.device = int(device)
        self._events = events  # keep the borrowed buffer alive
        self.torch_stream = stream if stream is not None else torch.cuda.current_stream(self.device)
        self._off = np.ascontiguousarray(win_off, dtype=np.int64)
        self._t0 = np.ascontiguousarray(win_t0, dtype=np.int64)
        self._t1 = np.ascontiguousarray(win_t1, dtype=np.int64)
        self.W = len(self._t0)
        if len(self._off) != self.W + 1 or len(self._t1) != self.W:
            raise ValueError("win_off needs W+1 entries, win_t0 / win_t1 W entries")
        dev, sptr = self.device, self.torch_stream.cuda_stream

        def _alloc(size, ctx):
            try:
                if alloc_fn is not None:
                    return alloc_fn(int(size))
                return torch.cuda.caching_allocator_alloc(int(size), dev, sptr)
            except Exception:
                return None

        def _release(ptr, ctx):
            if release_fn is not None:
                release_fn(ptr)
            else:
                torch.cuda.caching_allocator_delete(ptr)

        self._alloc_cb = _ALLOC_T(_alloc)
        self._release_cb = _RELEASE_T(_release)
        env = _Env()
        if use_torch_allocator:
            env.alloc, env.release = self._alloc_cb, self._release_cb
        env.ctx = None
        env.cuda_stream = sptr
        env.device = dev
        self._env = env
        self.load_summary = np.zeros(self.W, dtype=LOAD_SUM)
        st = L.ta_load_window(ctypes.byref(env), ev_ptr, self.n, 1 if on_device else 0,
                              self._off.ctypes.data, self._t0.ctypes.data, self._t1.ctypes.data,
                              self.W, self.load_summary.ctypes.data, ctypes.byref(self._h))
        if st != 0:
            self.close()
            raise TaError(st, "ta_load_window")
        self._sorted = None

    def inject_device_error(self, code: int) -> None:
        """Test hook: marks the handle as failed, as a device-side wait that gave up would."""
        st = self._lib.ta_inject_device_error(self._h, int(code))
        if st != 0:
            raise TaError(st, "ta_inject_device_error")

    # -- context manager / lifetime
    def close(self):
        if self._h:
            self._lib.ta_free(self._h)
            self._h = _vp()

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _dims(self):
        s = self._sorted
        return {"n": self.n, "n_lanes": s.n_lanes if s else 0, "n_windows": self.W}

    # -- the seven calls
    def sort_timeline(self) -> SortResult:
        raw = _SortResult()
        st = self._lib.ta_sort_timeline(self._h, ctypes.byref(raw))
        if st != 0:
            raise TaError(st, "ta_sort_timeline")
        self._sorted = SortResult(self, raw, {"n": raw.n, "n_valid": raw.n_valid,
                                              "n_lanes": raw.n_lanes, "n_windows": raw.n_windows})
        self._events = None  # the borrow ends here
        return self._sorted

    def correlate_launches(self) -> JoinResult:
        raw = _JoinResult()
        summ = np.zeros(self.W, dtype=JOIN_SUM)
        st = self._lib.ta_correlate_launches(self._h, ctypes.byref(raw), summ.ctypes.data)
        if st != 0:
            raise TaError(st, "ta_correlate_launches")
        return JoinResult(self, raw, dict(self._dims(), join_sum=summ))

    def attribute_operators(self, check=True) -> AttrResult:
        """check=False returns the result even for TA_ERR_DEPTH / TA_ERR_BAD_NESTING
        (see .status); the summaries are valid, the other outputs unspecified."""
        raw = _AttrResult()
        summ = np.zeros(self.W, dtype=ATTR_SUM)
        st = self._lib.ta_attribute_operators(self._h, ctypes.byref(raw), summ.ctypes.data)
        if st != 0 and (check or st not in (TA_ERR_DEPTH, TA_ERR_BAD_NESTING)):
            raise TaError(st, "ta_attribute_operators")
        return AttrResult(self, raw, dict(self._dims(), attr_sum=summ, status=st))

    def stream_gaps(self, min_gap_ns: int) -> GapResult:
        raw = _GapResult()
        st = self._lib.ta_stream_gaps(self._h, int(min_gap_ns), ctypes.byref(raw))
        if st != 0:
            raise TaError(st, "ta_stream_gaps")
        return GapResult(self, raw, dict(self._dims(), n_long_gaps=raw.n_long_gaps))

    def aggregate_ops(self, kind_mask: int, value_sel: int) -> AggResult:
        raw = _AggResult()
        st = self._lib.ta_aggregate_ops(self._h, kind_mask, value_sel, ctypes.byref(raw))
        if st != 0:
            raise TaError(st, "ta_aggregate_ops")
        return AggResult(self, raw, dict(self._dims(), n_groups=raw.n_groups))

    def rollup_operators(self) -> RollupResult:
        raw = _RollupResult()
        summ = np.zeros(self.W, dtype=ROLLUP_SUM)
        st = self._lib.ta_rollup_operators(self._h, ctypes.byref(raw), summ.ctypes.data)
        if st != 0:
            raise TaError(st, "ta_rollup_operators")
        return RollupResult(self, raw, dict(self._dims(), rollup_sum=summ))

    def critical_path(self) -> CritpathResult:
        raw = _CritpathResult()
        summ = np.zeros(self.W, dtype=CRITPATH_SUM)
        st = self._lib.ta_critical_path(self._h, ctypes.byref(raw), summ.ctypes.data)
        if st != 0:
            raise TaError(st, "ta_critical_path")
        return CritpathResult(self, raw, dict(self._dims(), n_rows=raw.n_rows, critpath_sum=summ))

    def blame_gaps(self, gaps) -> BlameResult:
        """gaps: the GapResult of an earlier stream_gaps() call on this window."""
        raw = _BlameResult()
        summ = np.zeros(self.W, dtype=BLAME_SUM)
        st = self._lib.ta_blame_gaps(self._h, ctypes.byref(gaps._raw), ctypes.byref(raw), summ.ctypes.data)
        if st != 0:
            raise TaError(st, "ta_blame_gaps")
        return BlameResult(self, raw, dict(self._dims(), n_long_gaps=raw.n_long_gaps, blame_sum=summ))

    def operator_sol(self, flops, nbytes, peak_flops: float, peak_bw: float) -> SolResult:
        """flops / nbytes: float64 per INPUT record (numpy arrays, or CUDA tensors on this
        window's device); negative or NaN = not known."""
        raw = _SolResult()
        summ = np.zeros(self.W, dtype=SOL_SUM)
        on_device = hasattr(flops, "is_cuda")
        if on_device:
            import torch
            if not (flops.is_cuda and nbytes.is_cuda and flops.dtype == torch.float64
                    and nbytes.dtype == torch.float64 and flops.is_contiguous() and nbytes.is_contiguous()):
                raise ValueError("counts must be contiguous float64 CUDA tensors")
            fp, bp, cnt = flops.data_ptr(), nbytes.data_ptr(), (flops.numel(), nbytes.numel())
        else:
            flops = np.ascontiguousarray(flops, dtype=np.float64)
            nbytes = np.ascontiguousarray(nbytes, dtype=np.float64)
            fp, bp, cnt = flops.ctypes.data, nbytes.ctypes.data, (len(flops), len(nbytes))
        if cnt != (self.n, self.n):
            raise ValueError("one operation count and one data volume per input record")
        st = self._lib.ta_operator_sol(self._h, fp, bp, 1 if on_device else 0, float(peak_flops),
                                       float(peak_bw), ctypes.byref(raw), summ.ctypes.data)
        if st != 0:
            raise TaError(st, "ta_operator_sol")
        return SolResult(self, raw, dict(self._dims(), sol_sum=summ))

    def device_overlap(self) -> OverlapResult:
        raw = _OverlapResult()
        st = self._lib.ta_device_overlap(self._h, ctypes.byref(raw))
        if st != 0:
            raise TaError(st, "ta_device_overlap")
        return OverlapResult(self, raw, dict(self._dims(), n_rows=raw.n_rows))

    def match_collectives(self, comm_sizes=()) -> CollResult:
        arr = np.zeros(len(comm_sizes), dtype=COMM_SIZE)
        for i, (cid, nr) in enumerate(comm_sizes):
            arr[i] = (cid, nr, 0)
        raw = _CollResult()
        st = self._lib.ta_match_collectives(self._h, arr.ctypes.data if len(arr) else None, len(arr),
                                            ctypes.byref(raw))
        if st != 0:
            raise TaError(st, "ta_match_collectives")
        return CollResult(self, raw, dict(self._dims(), n_groups=raw.n_groups, n_ranks=raw.n_ranks))
