#!/usr/bin/env python
"""Benchmark of the trace-window analyzer hot path.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--workload c0..c4] [--scale S]

One step = the whole hot path (load, sort, correlate, attribute, gaps, two
aggregate calls, collectives, free) over one synthetic window batch.  Default
workload: c3, the 64M-record MoE expert-parallel decode window the headline
metric is quoted on.  Prints ONE JSON line (rank 0).  With N > 1 (launched by
torch.distributed.run) every rank analyses its own copy of the workload on its
own GPU - the path does not shard, so these are independent replicas and no
collective sits on the data path.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "trace events analysed/sec per 30 s window (1 B200) and % of HBM roofline"
UNIT = "events/s"
WORKLOAD_TEXT = {
    "c0": "c0: tiny single-process window (1 pid, 2 streams)",
    "c1": "c1: 8-rank tensor-parallel decode window (8 pids x 4 streams)",
    "c2": "c2: prefill-heavy mixed-batch window (4 pids x 8 streams)",
    "c3": "c3: MoE expert-parallel decode window (16 pids x 4 streams), the 64M-record window",
    "c4": "c4: fleet batch of 512 independent 30 s windows",
}
# ncu: dram__bytes_read.sum + dram__bytes_write.sum of one k_radix_pass launch divided by the
# records it sorted, on the quarter-size case (profiles/radix_pass_c3_quarter.txt)
RADIX_TRAFFIC_BYTES_PER_RECORD = 13.8


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c3", choices=sorted(WORKLOAD_TEXT))
    ap.add_argument("--scale", type=float, default=1.0)
    ap.add_argument("--e2e-steps", type=int, default=4)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--allocator", default="library", choices=["library", "torch"],
                    help="device memory through the library's own stream-ordered pool, or through "
                         "PyTorch's caching allocator (ta_env callbacks into Python)")
    ap.add_argument("--cpu-sample-events", type=int, default=70_000_000,
                    help="records of the workload the CPU oracle is timed on (the whole c0..c3 "
                         "window by default: about 36 s for c3; a sample of c4's windows)")
    return ap.parse_args()


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons (NVML, read-only) while the timed region runs."""

    def __init__(self, device_index):
        self.idx = device_index
        self.sm, self.reasons, self.max_mhz = [], set(), None
        self._stop = False
        self._thread = None

    def _run(self):
        try:
            import pynvml as nv
            nv.nvmlInit()
            # LOCAL_RANK indexes the visible devices; map through CUDA_VISIBLE_DEVICES if it is set
            vis = os.environ.get("CUDA_VISIBLE_DEVICES")
            idx = self.idx
            if vis:
                ids = [x for x in vis.split(",") if x != ""]
                if self.idx < len(ids) and ids[self.idx].isdigit():
                    idx = int(ids[self.idx])
            hnd = nv.nvmlDeviceGetHandleByIndex(idx)
            self.max_mhz = float(nv.nvmlDeviceGetMaxClockInfo(hnd, nv.NVML_CLOCK_SM))
            names = {"hw_slowdown": nv.nvmlClocksThrottleReasonHwSlowdown,
                     "hw_thermal_slowdown": nv.nvmlClocksThrottleReasonHwThermalSlowdown,
                     "sw_thermal_slowdown": nv.nvmlClocksThrottleReasonSwThermalSlowdown,
                     "sw_power_cap": nv.nvmlClocksThrottleReasonSwPowerCap}
            while not self._stop:
                self.sm.append(float(nv.nvmlDeviceGetClockInfo(hnd, nv.NVML_CLOCK_SM)))
                r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(hnd)
                for k, bit in names.items():
                    if r & bit:
                        self.reasons.add(k)
                time.sleep(0.01)
        except Exception as e:  # no NVML: report that no samples were taken
            self.error = str(e)

    def start(self):
        import threading
        self._thread = threading.Thread(target=self._run, daemon=True)
        self._thread.start()

    def stop(self):
        self._stop = True
        if self._thread is not None:
            self._thread.join(timeout=2)
        out = {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons)}
        if self.sm:
            out["sm_mhz"] = statistics.median(self.sm)
            out["samples"] = len(self.sm)
        return out


ALLOCATOR = "library"
SOL_WORK = None  # (flops, bytes) CUDA tensors per input record, for the per-call timing of ta_operator_sol


def run_pipeline(ta, buf, wl, read_back=False, per_call=None, stream=None):
    """The whole hot path once.  Returns (n_valid, bytes read back from the device).
    per_call: dict that collects the wall time of each call (every call ends synchronised).
    stream: the torch stream the window works on (default: the current one)."""
    marks = [time.perf_counter()]

    def mark(name):
        if per_call is not None:
            marks.append(time.perf_counter())
            per_call.setdefault(name, []).append(1e3 * (marks[-1] - marks[-2]))

    with ta.Window(buf, wl.win_off, wl.win_t0, wl.win_t1, stream=stream,
                   use_torch_allocator=(ALLOCATOR == "torch")) as w:
        mark("load_window")
        s = w.sort_timeline()
        mark("sort_timeline")
        j = w.correlate_launches()
        mark("correlate_launches")
        a = w.attribute_operators()
        mark("attribute_operators")
        g = w.stream_gaps(500_000)
        mark("stream_gaps")
        k1 = w.aggregate_ops(ta.DEVICE_KINDS, 0)
        mark("aggregate_ops(device kinds, duration)")
        k2 = w.aggregate_ops(1 << ta.KIND_OP, 1)
        mark("aggregate_ops(OP, T_op)")
        c = w.match_collectives(wl.comm_sizes)
        mark("match_collectives")
        if per_call is not None:  # analyses built on top of the hot path: not part of a step
            w.device_overlap()
            mark("device_overlap (outside the timed step)")
            w.blame_gaps(g)
            w.aggregate_ops(1 << ta.KIND_OP, 2)
            mark("blame_gaps + aggregate_ops(OP, idle charged) (outside the timed step)")
            w.rollup_operators()
            mark("rollup_operators (outside the timed step)")
            if SOL_WORK is not None:
                from paper_2609_40247_b200 import synth as _synth
                w.operator_sol(SOL_WORK[0], SOL_WORK[1], _synth.PEAK_FLOPS, _synth.PEAK_BW)
                mark("operator_sol (outside the timed step)")
            w.critical_path()
            mark("critical_path (outside the timed step)")
        nbytes = w.load_summary.nbytes + j.join_sum.nbytes + a.attr_sum.nbytes
        if read_back:
            for res, names in ((g, ("lane_gaps", "win_hist", "long_gaps")),
                               (k1, ("g_count", "g_sum", "g_min", "g_max", "g_name", "g_pid")),
                               (k2, ("g_count", "g_sum", "g_min", "g_max", "g_name", "g_pid")),
                               (c, ("r_pid", "r_n_coll", "r_sum_wait", "r_max_wait", "r_n_straggler"))):
                for nm in names:
                    nbytes += res.numpy(nm).nbytes
        return s.n_valid, nbytes


def lsd_model_bytes_per_event(wl):
    """Algorithmic bytes per record of the whole path when the sort is modelled as an LSD radix
    sort of (key, index) pairs with one pass per key byte: the numerator of the headline
    roofline fraction, recomputed from the workload's own event mix and key width."""
    ev = wl.events
    n = max(len(ev), 1)
    kinds = np.bincount(np.clip(ev["kind"].astype(np.int64), 0, 6), minlength=7)[:6] / n
    f_o, f_api, f_l, f_k, f_m, f_c = (float(x) for x in kinds)
    f_K = f_k + f_m
    f_h, f_d = f_o + f_api + f_l, f_K + f_c

    def bits(x):
        return int(np.ceil(np.log2(max(int(x), 1)))) if x > 1 else 0

    n_streams = len(np.unique(ev["stream"])) if len(ev) else 1
    span = int(np.max(np.asarray(wl.win_t1) - np.asarray(wl.win_t0))) if len(wl.win_t0) else 1
    key_bits = bits(len(wl.win_t0)) + bits(len(np.unique(ev["pid"]))) + 1 + bits(n_streams) + bits(span)
    passes = (key_bits + 7) // 8
    parts = {
        "load": 52.0,
        "sort": 8.0 + passes * 24.0,
        "gather": 84.0,
        "join": f_l * 44.0 + f_K * 64.0,
        "attribute": f_h * 23.0 + f_K * 40.0 + f_o * 28.0,
        "gaps": f_d * 26.0,
        "aggregate": (2.0 + f_d * 24.0) + (2.0 + f_o * 32.0),
        "collectives": f_c * 100.0,
    }
    return sum(parts.values()), key_bits, passes, parts


def built_path_bytes_per_event(wl, radix_bytes_per_event):
    """Algorithmic bytes per record of the path AS BUILT, kernel by kernel (reads + writes of
    every column or table a kernel touches, fills and read-modify-write atomics included;
    lookups that stay in cache across a tile are counted once per record).  The radix passes
    enter with the bytes the library reports for them (16 B per record and pass for packed
    keys).  f_x = share of the records of kind x."""
    ev = wl.events
    n = max(len(ev), 1)
    kinds = np.bincount(np.clip(ev["kind"].astype(np.int64), 0, 6), minlength=7)[:6] / n
    f_o, f_api, f_l, f_k, f_m, f_c = (float(x) for x in kinds)
    f_K, f_h, f_d = f_k + f_m, f_o + f_api + f_l, f_k + f_m + f_c
    parts = {
        "discover": 40.0 + 8.0,                       # records in, one word per record out
        "radix passes": radix_bytes_per_event,        # keys in, keys out, per pass
        "gather": 8.0 + 40.0 + 44.0,                  # key, record (random), 8 columns + perm
        "join": 4.0 + (2.0 + f_l * 12.0)              # kol fill; build: kind, corr, table slot
                + (2.0 + f_K * 36.0 + 20.0 + f_K * 4.0)   # probe: kind, corr, ts, slot, launch ts/te; 3 outputs; kol
                + (2.0 + f_l * 8.0),                  # launch statistics: kind, slot, kol
        "attribute": 28.0 + (2.0 + f_h * 8.0)         # per-operator fill; tile stacks: kind, ts_end
                     + (2.0 + f_h * 16.0 + 5.0 + f_l * 12.0)   # resolve: kind, ts pair; parent, depth; kernels of the launch, count added to its operator
                     + (2.0 + f_K * (4.0 + 16.0 + 4.0 + 24.0) + 4.0)   # inherit: launch_of, ts pair, parent, 3 atomics; op_of
                     + (4.0 + f_o * 32.0),            # finalize: count; first/last read and rewritten
        "gaps": 2.0 + f_d * 16.0 + 8.0,
        "aggregate": (2.0 + f_d * 20.0) + (2.0 + f_o * 24.0),
        "collectives": 8.0 + 2.0 + f_c * 100.0,       # wait fill, kind, compaction + pair sort + groups
    }
    return sum(parts.values()), parts


def time_oracle(wl):
    """Times the CPU oracle, as it stands, on one workload (single thread)."""
    from oracle.ta_oracle import Oracle
    t = time.perf_counter()
    o = Oracle(wl.events, wl.win_off, wl.win_t0, wl.win_t1)
    o.load()
    o.sort()
    o.correlate()
    o.attribute()
    o.gaps(500_000)
    o.aggregate((1 << 3) | (1 << 4) | (1 << 5), 0)
    o.aggregate(1, 1)
    o.collectives(wl.comm_sizes)
    dt = time.perf_counter() - t
    o.close()
    return dt


def time_oracle_by_window(wl, threads):
    """The oracle as it stands, one window per task on `threads` host threads (windows are
    independent; the library call releases the interpreter lock).  Returns seconds."""
    from concurrent.futures import ThreadPoolExecutor
    import numpy as np
    from types import SimpleNamespace
    off = np.asarray(wl.win_off)
    parts = [SimpleNamespace(events=wl.events[off[w]:off[w + 1]], win_off=[0, int(off[w + 1] - off[w])],
                             win_t0=[wl.win_t0[w]], win_t1=[wl.win_t1[w]], comm_sizes=wl.comm_sizes)
             for w in range(len(off) - 1)]
    t = time.perf_counter()
    with ThreadPoolExecutor(max_workers=threads) as ex:
        list(ex.map(time_oracle, parts))
    return time.perf_counter() - t


def reference_arm(args, rank):
    """--impl reference: the oracle on the host cores, each step a bounded sample."""
    if rank != 0:
        return
    from paper_2609_40247_b200 import synth
    full = synth.CONFIG_EVENTS[args.workload]
    scale = min(1.0, 2_000_000 / full) * args.scale if args.workload != "c0" else 1.0
    wl = synth.make_workload(args.workload, scale, truth=False,
                             n_windows=8 if args.workload == "c4" else None)
    n = len(wl.events)
    for _ in range(args.warmup):
        time_oracle(wl)
    t = [time_oracle(wl) for _ in range(args.steps)]
    total = sum(t)
    value = n * args.steps / total
    sample = f"{n} records of workload {args.workload} (scale {scale:.4g}) per step"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int64",
        "data": "synthetic",
        "config": {"workload": WORKLOAD_TEXT[args.workload], "events_per_step": n, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def reduce_over_ranks(dist, elapsed_ms, e2e_ms, n_records, device):
    """Whole-job numbers: the slowest rank's times, the records of all ranks."""
    import torch
    t = torch.tensor([elapsed_ms, e2e_ms], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    cnt = torch.tensor([n_records], device=device, dtype=torch.int64)
    dist.all_reduce(cnt, op=dist.ReduceOp.SUM)
    return float(t[0]), float(t[1]), int(cnt[0])


def main():
    args = parse_args()
    global ALLOCATOR
    ALLOCATOR = args.allocator
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.impl == "reference":
        reference_arm(args, rank)
        return

    import torch
    import torch.distributed as dist
    from paper_2609_40247_b200 import synth, ta

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the analyzer has no CPU path")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    ta.lib()  # fail loudly now if libta.so is missing

    # ---- synthetic workload (each rank its own replica, different seed) ----
    wl = synth.make_workload(args.workload, args.scale, truth=False, seed_offset=100 * rank)
    n = len(wl.events)
    host = torch.from_numpy(np.ascontiguousarray(wl.events).view(np.uint8).reshape(-1))
    dev_buf = host.to(dev)
    torch.cuda.synchronize()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timing ----
    for _ in range(max(args.warmup, 0)):
        run_pipeline(ta, dev_buf, wl)
    barrier()
    sampler = ClockSampler(local_rank)
    sampler.start()
    time.sleep(0.05)
    launches0 = ta.launch_count()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    barrier()
    ev0.record()
    for k in range(args.steps):
        n_valid, _ = run_pipeline(ta, dev_buf, wl)
        marks[k].record()
    ev1.record()
    torch.cuda.synchronize()
    barrier()
    elapsed_ms = ev0.elapsed_time(ev1)
    per_step = [(ev0 if k == 0 else marks[k - 1]).elapsed_time(marks[k]) for k in range(args.steps)]
    launches = ta.launch_count() - launches0
    clocks = sampler.stop()

    # ---- the dominant kernel, timed live in steps of its own (the library records a CUDA event
    # pair around every radix pass of the timeline sort; nothing of this runs in the timed region)
    ta.profile_enable(True)
    radix_steps = max(1, min(args.steps, 5))
    for _ in range(radix_steps):
        run_pipeline(ta, dev_buf, wl)
    torch.cuda.synchronize()
    n_pass, radix_ms, radix_bytes = ta.profile_radix()
    ta.profile_enable(False)

    # ---- per-call breakdown (outside the timed region) ----
    global SOL_WORK
    fl, nb = synth.op_work(wl.events, seed=1)
    SOL_WORK = (torch.from_numpy(fl).to(dev), torch.from_numpy(nb).to(dev))
    per_call = {}
    for _ in range(3):
        run_pipeline(ta, dev_buf, wl, per_call=per_call)
    per_call_ms = {k: round(min(v), 4) for k, v in per_call.items()}
    SOL_WORK = None

    # ---- end to end: pinned host input, host<->device copies inside the timed region ----
    e2e = None
    if args.e2e_steps > 0:
        pinned = host.pin_memory()
        host_np = pinned.numpy().view(synth.EVENT_DTYPE)
        run_pipeline(ta, host_np, wl, read_back=True)
        barrier()
        # Two windows in flight, as a service that analyses one window after another would run
        # it: two host threads, each with a stream and a handle of its own, take the steps in
        # turn, so that the host->device copy of one window overlaps the analysis of the one
        # before (every step still copies its own 40 bytes per record in and its results out).
        import threading
        streams = [torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)]
        d2h_of = [0, 0]
        errors = []

        def worker(k):
            try:
                torch.cuda.set_device(dev)
                with torch.cuda.stream(streams[k]):
                    for _ in range(k, args.e2e_steps, 2):
                        _, d2h_of[k] = run_pipeline(ta, host_np, wl, read_back=True, stream=streams[k])
                    streams[k].synchronize()
            except Exception as exc:  # surfaces in the main thread
                errors.append(exc)

        for k in range(2):  # one untimed step per stream: its pool blocks and staging buffers
            with torch.cuda.stream(streams[k]):
                run_pipeline(ta, host_np, wl, read_back=True, stream=streams[k])
        torch.cuda.synchronize()
        barrier()
        t0 = time.perf_counter()
        threads = [threading.Thread(target=worker, args=(k,)) for k in range(2)]
        for th in threads:
            th.start()
        for th in threads:
            th.join()
        torch.cuda.synchronize()
        e2e_ms = 1e3 * (time.perf_counter() - t0)
        if errors:
            raise errors[0]
        d2h = max(d2h_of)
        e2e = {"ms": e2e_ms, "d2h": d2h}

    # ---- max over ranks ----
    if world > 1:
        elapsed_ms, e2e_ms, total_events = reduce_over_ranks(
            dist, elapsed_ms, e2e["ms"] if e2e else 0.0, n, dev)
        if e2e:
            e2e["ms"] = e2e_ms
    else:
        total_events = n

    if rank == 0:
        peak, peak_kind = measured_peak()
        value = total_events * args.steps / (elapsed_ms * 1e-3)
        roof = None
        if n_pass > 0 and radix_ms > 0:
            per_launch_bytes = radix_bytes / n_pass  # 8 B read + 8 B written per packed key
            ach = radix_bytes / (radix_ms * 1e-3) / 1e9
            roof = {"bound": "hbm", "kernel": "k_radix_pass", "achieved": ach, "peak": peak,
                    "peak_source": f"of {peak_kind}", "unit": "GB/s", "frac": ach / peak,
                    "launches_timed": n_pass, "avg_launch_ms": radix_ms / n_pass,
                    "algorithmic_bytes_per_launch": per_launch_bytes,
                    "traffic": (RADIX_TRAFFIC_BYTES_PER_RECORD * n
                                if RADIX_TRAFFIC_BYTES_PER_RECORD else None)}
        cpu = None
        if world == 1 and not args.no_cpu_baseline:
            full = synth.CONFIG_EVENTS[args.workload] * args.scale
            sc = min(1.0, args.cpu_sample_events / full) * args.scale
            if args.workload == "c4":  # whole windows of the batch's own size, as many as the sample allows
                per_window = full / synth.C4_WINDOWS
                sc = args.scale
                swl = synth.make_workload("c4", sc, truth=False,
                                          n_windows=max(1, min(synth.C4_WINDOWS,
                                                               int(args.cpu_sample_events / per_window))))
            else:
                swl = wl if sc >= args.scale else synth.make_workload(args.workload, sc, truth=False)
            dt = time_oracle(swl)
            whole = len(swl.events) == n
            cpu = {"value": len(swl.events) / dt, "unit": UNIT, "cores": 1, "kind": "oracle",
                   "sample": (f"the whole workload ({len(swl.events)} records), one pass, {dt:.1f} s" if whole
                              else f"{len(swl.events)} records of workload {args.workload} "
                                   f"(scale {sc:.4g}), one pass, {dt:.1f} s"),
                   "host_cores": os.cpu_count()}
            if args.workload == "c4":  # many independent windows: also all host cores, one window per task
                th = os.cpu_count() or 1
                dta = time_oracle_by_window(swl, th)
                cpu["all_cores"] = {"value": len(swl.events) / dta, "threads": th,
                                    "sample": f"the same {len(swl.win_t0)} windows, one per task, {dta:.1f} s"}
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": elapsed_ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "int64", "data": "synthetic",
            "config": {"workload": WORKLOAD_TEXT[args.workload], "events_per_gpu": n,
                       "n_valid": int(n_valid), "windows": int(len(wl.win_t0)),
                       "parallelism": "replicas only" if world > 1 else "single GPU",
                       "allocator": ("the library's own stream-ordered pool" if args.allocator == "library"
                                     else "PyTorch's caching allocator through ta_env callbacks"),
                       "l2": f"inputs are {n * 40 / 1e6:.0f} MB and every pass streams them; "
                             "no L2 flush needed above 126 MB"},
            "clocks": clocks, "gpu_launches": int(launches),
            "roofline": roof, "cpu_baseline": cpu,
            "per_call_ms": per_call_ms,
            "step_ms": {"median": statistics.median(per_step), "best": min(per_step)} if per_step else None,
        }
        lsd_bytes, key_bits, passes, parts = lsd_model_bytes_per_event(wl)
        per_gpu = value / world
        radix_per_event = (radix_bytes / radix_steps / n) if (n_pass > 0 and n > 0) else 0.0
        built_bytes, built_parts = built_path_bytes_per_event(wl, radix_per_event)
        line["hbm_model"] = {
            # headline: the bytes the path as built touches (kernel by kernel, built_path_bytes_per_event)
            "built_bytes_per_event": round(built_bytes, 2),
            "built_parts": {k: round(v, 2) for k, v in built_parts.items()},
            "radix_passes_per_step": (n_pass / radix_steps) if n_pass else 0,
            "frac_of_measured_peak": per_gpu * built_bytes / (peak * 1e9),
            "frac_of_nominal_8TBs": per_gpu * built_bytes / 8.0e12,
            "target_ms_for_half_of_measured_peak": 2e3 * n * built_bytes / (peak * 1e9),
            # secondary: the byte model of an LSD sort of (key, index) pairs, one pass per key
            # byte - a different algorithm's bytes - and the compulsory bytes alone
            "lsd_bytes_per_event": round(lsd_bytes, 2), "lsd_key_bits": key_bits, "lsd_passes": passes,
            "lsd_parts": {k: round(v, 2) for k, v in parts.items()},
            "frac_of_measured_peak_lsd_model": per_gpu * lsd_bytes / (peak * 1e9),
            "target_ms_for_half_of_measured_peak_lsd_model": 2e3 * n * lsd_bytes / (peak * 1e9),
            "compulsory_bytes_per_event": 108.0,
            "frac_of_measured_peak_compulsory": per_gpu * 108.0 / (peak * 1e9),
        }
        if e2e:
            line["e2e"] = {"value": total_events * args.e2e_steps / (e2e["ms"] * 1e-3), "unit": UNIT,
                           "h2d_bytes_per_step": n * 40, "d2h_bytes_per_step": int(e2e["d2h"]),
                           "steps": args.e2e_steps, "windows_in_flight": 2}
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
