"""Seeded synthetic profiling windows (inputs only; no analysis arithmetic).

The paper's traces are private, so every test and benchmark input is produced
here: a C++ simulation (ta_synth.cpp) of host threads, in-order device streams
and lock-step collectives whose shapes follow the five benchmark workloads
(c0..c4).  Besides the 40-byte records the generator returns what the
simulation knows to be true (parent operator, launch of each kernel, idle time
before each device record, collective waits), which the tests use as an
independent check.  Nothing in this module is shared with either analyzer.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading
from concurrent.futures import ThreadPoolExecutor

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ta_synth.cpp")
_LIB = os.path.join(_HERE, "libta_synth.so")

EVENT_DTYPE = np.dtype(
    [
        ("ts_start", "<i8"),
        ("ts_end", "<i8"),
        ("corr_id", "<i8"),
        ("pid", "<i4"),
        ("name_id", "<i4"),
        ("seq", "<i4"),
        ("stream", "<i2"),
        ("kind", "<i2"),
    ]
)
assert EVENT_DTYPE.itemsize == 40

KIND_OP, KIND_API, KIND_LAUNCH, KIND_KERNEL, KIND_MEMCPY, KIND_COLL = range(6)

T0_BASE = 1_700_000_000_000_000_000  # exercises full int64 timestamps
WINDOW_STRIDE_NS = 60_000_000_000
SPAN_30S = 30_000_000_000


class _Config(ctypes.Structure):
    _fields_ = [
        ("mode", ctypes.c_int32),
        ("n_pid", ctypes.c_int32),
        ("n_threads", ctypes.c_int32),
        ("n_streams", ctypes.c_int32),
        ("pid_base", ctypes.c_int32),
        ("n_steps", ctypes.c_int32),
        ("ops_per_step", ctypes.c_int32),
        ("launches_per_step", ctypes.c_int32),
        ("max_depth", ctypes.c_int32),
        ("layers_per_step", ctypes.c_int32),
        ("ops_per_layer", ctypes.c_int32),
        ("kernels_per_layer", ctypes.c_int32),
        ("colls_per_layer", ctypes.c_int32),
        ("sync_api", ctypes.c_int32),
        ("n_names", ctypes.c_int32),
        ("name_mode", ctypes.c_int32),
        ("shuffle_mode", ctypes.c_int32),
        ("comm_offset", ctypes.c_int32),
        ("seed", ctypes.c_uint64),
        ("span_ns", ctypes.c_int64),
        ("zipf_s", ctypes.c_double),
        ("k_med1_ns", ctypes.c_double),
        ("k_sigma1", ctypes.c_double),
        ("k_frac2", ctypes.c_double),
        ("k_med2_ns", ctypes.c_double),
        ("k_sigma2", ctypes.c_double),
        ("launch_delay_mean_ns", ctypes.c_double),
        ("coll_skew_sigma_ns", ctypes.c_double),
        ("stall_prob", ctypes.c_double),
        ("stall_min_ns", ctypes.c_double),
        ("stall_max_ns", ctypes.c_double),
        ("memcpy_frac", ctypes.c_double),
        ("delete_launch_frac", ctypes.c_double),
        ("tie_prob", ctypes.c_double),
        ("step_gap_mean_ns", ctypes.c_double),
    ]


_lib = None
_lock = threading.Lock()


def build(force: bool = False) -> str:
    """Compile the generator with g++ (in-tree); returns the library path."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        subprocess.check_call(
            ["g++", "-O2", "-std=c++17", "-shared", "-fPIC", _SRC, "-o", _LIB + ".tmp"]
        )
        os.replace(_LIB + ".tmp", _LIB)
    return _LIB


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = ctypes.CDLL(build())
            lib.tasynth_max_events.restype = ctypes.c_int64
            lib.tasynth_max_events.argtypes = [ctypes.POINTER(_Config)]
            lib.tasynth_generate.restype = ctypes.c_int32
            lib.tasynth_generate.argtypes = [
                ctypes.POINTER(_Config), ctypes.c_int64, ctypes.c_void_p, ctypes.c_int64,
                ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                ctypes.POINTER(ctypes.c_int64), ctypes.POINTER(ctypes.c_int64),
                ctypes.POINTER(ctypes.c_int64),
            ]
            _lib = lib
    return _lib


_DEFAULTS = dict(
    mode=0, n_pid=1, n_threads=1, n_streams=1, pid_base=100, n_steps=1,
    ops_per_step=1, launches_per_step=0, max_depth=4,
    layers_per_step=1, ops_per_layer=1, kernels_per_layer=1, colls_per_layer=0,
    sync_api=1, n_names=64, name_mode=0, shuffle_mode=0, comm_offset=0, seed=0,
    span_ns=SPAN_30S, zipf_s=1.0,
    k_med1_ns=20000.0, k_sigma1=1.0, k_frac2=0.0, k_med2_ns=0.0, k_sigma2=0.0,
    launch_delay_mean_ns=8000.0, coll_skew_sigma_ns=30000.0,
    stall_prob=0.0, stall_min_ns=0.0, stall_max_ns=0.0,
    memcpy_frac=0.0, delete_launch_frac=0.0, tie_prob=0.002, step_gap_mean_ns=0.0,
)


def window_params(family: str, target_events: int, seed: int) -> dict:
    """Generator parameters of one window of a workload family, scaled to
    about `target_events` records.  Families: 'c0' tiny single process,
    'c1' tensor-parallel decode, 'c2' prefill-heavy mixed batch, 'c3' MoE
    expert-parallel decode."""
    p = dict(_DEFAULTS)
    p["seed"] = seed
    if family == "c0":
        p.update(mode=0, n_pid=1, n_threads=1, n_streams=2, ops_per_step=16,
                 launches_per_step=16, max_depth=4, sync_api=0, n_names=64, name_mode=0,
                 k_med1_ns=20000.0, k_sigma1=1.0)
        per_step = 48
        p["n_steps"] = max(1, target_events // per_step)
        p["step_gap_mean_ns"] = 0.75 * SPAN_30S / p["n_steps"]
    elif family == "c1":
        p.update(mode=1, n_pid=8, n_streams=4, layers_per_step=80, ops_per_layer=4,
                 kernels_per_layer=12, colls_per_layer=2, n_names=256, name_mode=2,
                 k_med1_ns=15000.0, k_sigma1=0.8, coll_skew_sigma_ns=30000.0)
        per_step = (2 + 80 * 30) * 8
        p["n_steps"] = max(1, target_events // per_step)
    elif family == "c2":
        p.update(mode=0, n_pid=4, n_threads=2, n_streams=8, ops_per_step=32,
                 launches_per_step=32, max_depth=8, n_names=1024, name_mode=1, zipf_s=1.1,
                 k_med1_ns=10000.0, k_sigma1=0.5, k_frac2=0.3, k_med2_ns=2.0e6, k_sigma2=0.5,
                 stall_prob=0.05, stall_min_ns=0.5e6, stall_max_ns=5.0e6, memcpy_frac=0.02,
                 span_ns=0)
        per_step = 97 * 4 * 2
        p["n_steps"] = max(1, target_events // per_step)
    elif family == "c3":
        p.update(mode=1, n_pid=16, n_streams=4, layers_per_step=48, ops_per_layer=3,
                 kernels_per_layer=10, colls_per_layer=2, n_names=4096, name_mode=1, zipf_s=1.3,
                 k_med1_ns=4000.0, k_sigma1=1.2, delete_launch_frac=0.01,
                 coll_skew_sigma_ns=30000.0)
        per_step = (2 + 48 * 25) * 16
        p["n_steps"] = max(1, target_events // per_step)
    else:
        raise ValueError(f"unknown workload family {family!r}")
    return p


def generate_window(params: dict, t0: int, out=None, truth: bool = True):
    """Runs the simulation once.  Returns (events, t1, truth_dict)."""
    lib = _load()
    cfg = _Config(**params)
    cap = int(lib.tasynth_max_events(ctypes.byref(cfg)))
    if out is None:
        out = np.empty(cap, dtype=EVENT_DTYPE)
    elif len(out) < cap:
        raise ValueError("output buffer too small")
    link = np.empty(cap, dtype=np.int32) if truth else None
    val = np.empty(cap, dtype=np.int64) if truth else None
    wait = np.empty(cap, dtype=np.int64) if truth else None
    n = ctypes.c_int64()
    t1 = ctypes.c_int64()
    ndel = ctypes.c_int64()
    rc = lib.tasynth_generate(
        ctypes.byref(cfg), t0, out.ctypes.data, cap,
        link.ctypes.data if truth else None, val.ctypes.data if truth else None,
        wait.ctypes.data if truth else None,
        ctypes.byref(n), ctypes.byref(t1), ctypes.byref(ndel))
    if rc != 0:
        raise RuntimeError(
            {1: "capacity too small", 2: "simulated activity exceeds the fixed window span",
             3: "bad generator configuration"}.get(rc, f"generator error {rc}"))
    n = n.value
    tr = None
    if truth:
        tr = {"link": link[:n], "val": val[:n], "wait": wait[:n], "n_deleted": ndel.value}
    return out[:n], t1.value, tr


CONFIG_EVENTS = {"c0": 60_000, "c1": 1 << 22, "c2": 1 << 24, "c3": 1 << 26, "c4": 1 << 28}
CONFIG_SEED = {"c0": 0, "c1": 1, "c2": 2, "c3": 3}
C4_WINDOWS = 512


class Workload(dict):
    """events, win_off, win_t0, win_t1 (numpy), truth (list per window or None),
    comm_sizes (list of (comm_id, n_ranks)), name."""

    __getattr__ = dict.__getitem__


def _comm_sizes(params: dict):
    if params["mode"] == 1 and params["colls_per_layer"] > 0:
        ns = min(params["colls_per_layer"], params["n_streams"])
        return [(0x5EED0000 + params["comm_offset"] + s, params["n_pid"]) for s in range(ns)]
    return []


def make_workload(name: str, scale: float = 1.0, shuffle_mode: int = 0, truth: bool = True,
                  n_windows: int | None = None, seed_offset: int = 0, threads: int = 8) -> Workload:
    """Builds benchmark workload c0..c4 (optionally scaled down by `scale`).

    c0..c3 are single windows; c4 concatenates `n_windows` (default 512)
    independent 30 s windows drawn in turn from the c1, c2 and c3 families, all
    using the same pid numbers and correlation ids."""
    if name in ("c0", "c1", "c2", "c3"):
        target = max(48, int(CONFIG_EVENTS[name] * scale))
        params = window_params(name, target, CONFIG_SEED[name] + seed_offset)
        params["shuffle_mode"] = shuffle_mode
        ev, t1, tr = generate_window(params, T0_BASE, truth=truth)
        n = len(ev)
        return Workload(
            name=name, events=ev, win_off=np.array([0, n], dtype=np.int64),
            win_t0=np.array([T0_BASE], dtype=np.int64), win_t1=np.array([t1], dtype=np.int64),
            truth=[tr] if truth else None, comm_sizes=_comm_sizes(params), params=[params])
    if name != "c4":
        raise ValueError(f"unknown workload {name!r}")
    W = n_windows if n_windows is not None else C4_WINDOWS
    per_window = max(48, int(CONFIG_EVENTS["c4"] * scale) // C4_WINDOWS)
    lib = _load()
    plist = []
    caps = []
    for w in range(W):
        fam = ("c1", "c2", "c3")[w % 3]
        p = window_params(fam, per_window, 1000 + w + seed_offset)
        p["shuffle_mode"] = shuffle_mode
        p["pid_base"] = 100
        if fam == "c3":
            p["comm_offset"] = 16  # 16-rank communicators get ids of their own
        if fam == "c2":
            # scaled-down prefill windows fit a 30 s span; keep it fixed like the others
            p["span_ns"] = SPAN_30S
            p["stall_max_ns"] = min(p["stall_max_ns"], 5.0e6)
        plist.append(p)
        caps.append(int(lib.tasynth_max_events(ctypes.byref(_Config(**p)))))
    offs_cap = np.concatenate([[0], np.cumsum(caps)]).astype(np.int64)
    buf = np.empty(int(offs_cap[-1]), dtype=EVENT_DTYPE)
    results = [None] * W

    def run(w):
        t0 = T0_BASE + w * WINDOW_STRIDE_NS
        sl = buf[offs_cap[w]:offs_cap[w + 1]]
        ev, t1, tr = generate_window(plist[w], t0, out=sl, truth=truth)
        results[w] = (len(ev), t0, t1, tr)

    with ThreadPoolExecutor(max_workers=threads) as ex:
        list(ex.map(run, range(W)))
    counts = np.array([r[0] for r in results], dtype=np.int64)
    win_off = np.concatenate([[0], np.cumsum(counts)]).astype(np.int64)
    if not np.array_equal(win_off, offs_cap):
        # compact (deleted launches make windows shorter than their capacity)
        out = np.empty(int(win_off[-1]), dtype=EVENT_DTYPE)
        for w in range(W):
            out[win_off[w]:win_off[w + 1]] = buf[offs_cap[w]:offs_cap[w] + counts[w]]
        buf = out
    sizes = {}
    for p in plist:
        for cid, nr in _comm_sizes(p):
            sizes[cid] = nr
    return Workload(
        name="c4", events=buf, win_off=win_off,
        win_t0=np.array([r[1] for r in results], dtype=np.int64),
        win_t1=np.array([r[2] for r in results], dtype=np.int64),
        truth=[r[3] for r in results] if truth else None,
        comm_sizes=sorted(sizes.items()), params=plist)


# Device peaks used with the synthetic operation counts (nominal dense bf16 and HBM3e figures
# of one B200; inputs of the efficiency step, not measurements).
PEAK_FLOPS = 2.25e15
PEAK_BW = 7.7e12


def op_work(events: np.ndarray, seed: int = 0, unknown_frac: float = 0.03):
    """Synthetic side table for the operator-efficiency step: per INPUT record a theoretical
    operation count (FLOP) and a logical data volume (bytes), float64, the stand-in for what
    an analyzer derives from shapes, data types and sharding.  Only OP records get counts
    (every other record holds -1 = not known); the counts depend on the symbol (a GEMM-like
    or a bandwidth-bound operator per name_id) and vary per invocation like a batch size; a
    fraction `unknown_frac` of the OP records has no counts."""
    n = len(events)
    rng = np.random.default_rng(seed)
    flops = np.full(n, -1.0)
    nbytes = np.full(n, -1.0)
    ops = np.nonzero(events["kind"] == 0)[0]
    name = events["name_id"][ops].astype(np.int64)
    batch = rng.integers(1, 65, size=len(ops)).astype(np.float64)
    hidden = 1024.0 * (1 + name % 8)
    gemm_like = (name % 3) != 0
    f = np.where(gemm_like, 2.0 * batch * hidden * hidden, 4.0 * batch * hidden)
    b = np.where(gemm_like, 2.0 * (hidden * hidden + 2.0 * batch * hidden), 6.0 * batch * hidden)
    known = rng.random(len(ops)) >= unknown_frac
    flops[ops] = np.where(known, f, -1.0)
    nbytes[ops] = np.where(known, b, -1.0)
    return flops, nbytes
