#!/usr/bin/env python
"""Benchmark of the AdaCons aggregation hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload bert64] [--impl ours|reference]

One "step" = one adacons_aggregate call (pass 1 + coefficient step + pass 2) on one N x d matrix
of synthetic worker gradients that is already resident in HBM.  Rank 0 prints ONE JSON line.

--gpus N > 1 (launched by torch.distributed.run): the aggregation of one matrix does not shard
across GPUs in this library, so every rank runs an independent replica of the same workload
(different seed); `value` = elements aggregated by all ranks / max-over-ranks time.

--impl reference times the float64 CPU oracle (oracle/), as it stands, on the host cores on a
bounded column sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "aggregated_grad_elements_per_s"
UNIT = "elements/s"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
ORACLE_SAMPLE_COLUMNS = 2_000_000      # --impl reference: columns per step
CPU_BASELINE_COLUMNS = 4_000_000       # cpu_baseline leg of the CUDA arm: 3 steps of this many columns

# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel, from the ncu
# captures summarised under profiles/ (a scaled-down case of the same recipe, traffic proportional
# to the columns processed), as a multiple of that kernel's algorithmic bytes.  Keyed by
# (workload, coefficient mode, kernel); anything else reports no traffic figure.
NCU_TRAFFIC_RATIO = {
    ("bert64", "model-wise", "pass1"): (1.0016, "profiles/pass1_pass2_bert64_d20M_full_set.md (same kernel, d = 20 M, scaled by d)"),
    ("bert64", "model-wise", "pass2"): (0.9989, "profiles/pass2_wide_bf16_result_larger_than_L2.md (same kernel, N = 16, d = 80 M; "
                                                "reads and writes both scale with the bytes processed)"),
}


def parse_args(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="bert64")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--d", type=int, default=0, help="override the gradient length (debugging)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-overlap-launch", action="store_true", help="plain stream order for the coefficient kernel too")
    ap.add_argument("--per-segment", action="store_true", help="layer-wise coefficients (workloads with segments)")
    ap.add_argument("--no-profile", action="store_true",
                    help="keep the per-kernel CUDA events out of the headline timed region (they are taken in a second loop)")
    ap.add_argument("--no-extra-loops", action="store_true",
                    help="skip the two additional loops (per-step events for the median; the launch sequence without events)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--shape", default="", help="N,d,dtype of an ad-hoc Gaussian workload instead of a named one, e.g. 128,20000000,bf16")
    ap.add_argument("--cluster-pass1", type=int, default=-1, choices=[-1, 0, 1], help="ADACONS_OPT_CLUSTER_PASS1 (64 < N <= 512)")
    ap.add_argument("--tall-tiles", type=int, default=-1, choices=[-1, 0, 1, 2], help="ADACONS_OPT_TALL_TILES (64 < N <= 256)")
    ap.add_argument("--column-sharded", action="store_true",
                    help="each rank holds its own d columns of ONE matrix of world*d columns: pass 1, an all-gather of the "
                         "statistics records, coefficient step and pass 2 (default for --gpus N > 1: independent replicas)")
    ap.add_argument("--gram-pass1", type=int, default=-1, help="ADACONS_OPT_GRAM_PASS1 (bf16, N <= 64): tiles per first-level sum; 0 = off")
    ap.add_argument("--shifted-loads", type=int, default=-1, choices=[-1, 0, 1],
                    help="ADACONS_OPT_SHIFTED_LOADS (rows at arbitrary element offsets, e.g. --shape with an odd d)")
    ap.add_argument("--one-launch", type=int, default=-1, choices=[-1, 0, 1, 2],
                    help="ADACONS_OPT_ONE_LAUNCH (default: the library's own choice by size)")
    return ap.parse_args(argv)


# ------------------------------------------------------------------------------------------------
# multi-process plumbing (replicas only)
# ------------------------------------------------------------------------------------------------
def dist_setup(n_gpus: int, use_cuda: bool):
    """Returns (rank, world, local_rank).  Initialises torch.distributed when world > 1."""
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29511")
        if not dist.is_initialized():
            dist.init_process_group(backend="nccl" if use_cuda else "gloo", rank=rank, world_size=world)
    return rank, world, local


def reduce_over_ranks(ms_local: float, units_local: float, device="cpu"):
    """Whole-job figures for independent replicas: (max over ranks of the time, sum of units)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms_local), float(units_local)
    t = torch.tensor([ms_local], dtype=torch.float64, device=device)
    u = torch.tensor([units_local], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


def barrier():
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


# ------------------------------------------------------------------------------------------------
# clocks during the timed region (read-only NVML queries)
# ------------------------------------------------------------------------------------------------
class ClockSampler(threading.Thread):
    def __init__(self, index: int, period_s: float = 0.005):
        super().__init__(daemon=True)
        self.index, self.period = index, period_s
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop_evt = threading.Event()
        self.ok = False
        self.uuid = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            u = pynvml.nvmlDeviceGetUUID(self.h)
            self.uuid = u.decode() if isinstance(u, bytes) else str(u)
            self.ok = True
        except Exception:
            self.nv = None

    def _reasons(self):
        nv = self.nv
        try:
            get = getattr(nv, "nvmlDeviceGetCurrentClocksEventReasons", None) or nv.nvmlDeviceGetCurrentClocksThrottleReasons
            mask = get(self.h)
        except Exception:
            return
        names = {
            "sw_power_cap": 0x4, "hw_slowdown": 0x8, "sync_boost": 0x10, "sw_thermal_slowdown": 0x20,
            "hw_thermal_slowdown": 0x40, "hw_power_brake_slowdown": 0x80, "applications_clocks_setting": 0x2,
            "display_clock_setting": 0x100,
        }
        for k, bit in names.items():
            if mask & bit:
                self.reasons.add(k)

    def run(self):
        if not self.ok:
            return
        while not self._stop_evt.is_set():
            try:
                self.samples.append(self.nv.nvmlDeviceGetClockInfo(self.h, self.nv.NVML_CLOCK_SM))
                self._reasons()
            except Exception:
                pass
            self._stop_evt.wait(self.period)

    def stop(self):
        self._stop_evt.set()
        if self.is_alive():
            self.join(timeout=2)
        s = sorted(self.samples)
        return {"sm_mhz": (s[len(s) // 2] if s else None), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(s), "gpu_uuid": self.uuid}


def physical_gpu_index(local_index: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_index])
        except Exception:
            return local_index
    return local_index


def measured_peak_gbs():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured (MEASURED_PEAKS.json, copy read+write)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (earlier measurement on this pool)"


# ------------------------------------------------------------------------------------------------
# CPU oracle legs
# ------------------------------------------------------------------------------------------------
def oracle_sample_steps(w, steps: int, warmup: int, columns: int):
    """Time oracle.step on a column sample of workload w; returns (mean seconds/step, elements/step)."""
    import numpy as np  # noqa: F401
    from oracle import adacons_oracle as oc
    from paper_2411_03742_b200 import workloads as wl
    ws = w.scaled(min(columns, w.d))
    orc = oc.AdaConsOracle(ws.N, ws.d)
    times = []
    for t in range(warmup + steps):
        G64 = wl.generate(ws, t, "cpu").to(dtype=__import__("torch").float64).numpy()
        t0 = time.perf_counter()
        orc.step(G64, storage=ws.dtype)
        dt = time.perf_counter() - t0
        if t >= warmup:
            times.append(dt)
    return sum(times) / len(times), ws.N * ws.d, ws


def run_reference(args):
    from paper_2411_03742_b200 import workloads as wl
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    w = pick_workload(args)
    sec, elems, ws = oracle_sample_steps(w, args.steps, min(args.warmup, 1), ORACLE_SAMPLE_COLUMNS)
    value = elems / sec
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": min(args.warmup, 1), "ms_per_step": sec * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": describe(w), "sample": f"first {ws.d} columns of every row, regenerated per step on the CPU"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle",
                         "sample": f"N={ws.N} x {ws.d} columns per step (float64 numpy, one thread; "
                                   f"host has {os.cpu_count()} cores)"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)
    return 0


def pick_workload(args):
    from paper_2411_03742_b200 import workloads as wl
    if args.shape:
        n, d, dt = args.shape.split(",")
        return wl.Workload(f"custom{n}x{d}", int(n), int(d), dt, 10, "gauss", seed=9000, note="signal N(0,1) + noise N(0,0.5^2)")
    w = wl.WORKLOADS[args.workload]
    return w.scaled(args.d) if args.d else w


def describe(w) -> str:
    return (f"{w.name}: N={w.N} workers, d={w.d}, {w.dtype} storage / fp32 accumulate, {w.steps}-step recipe "
            f"({w.note})")


# ------------------------------------------------------------------------------------------------
# the CUDA library
# ------------------------------------------------------------------------------------------------
def run_ours(args):
    import torch
    from paper_2411_03742_b200 import binding as ac, workloads as wl

    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the library has no CPU fallback")
    rank, world, local = dist_setup(args.gpus, use_cuda=True)
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    w = pick_workload(args)
    w_rank = __import__("dataclasses").replace(w, seed=w.seed + 100_000 * rank)

    # One matrix when it dwarfs the 126 MB L2; otherwise enough distinct matrices, used in turn, that
    # a step never finds its input in L2 from the step before.
    gbytes = w.N * w.d * w.elem_bytes
    nbuf = 1 if gbytes >= 8e9 else max(2, min(8, int(1.0e9 // max(gbytes, 1)) + 1))
    if nbuf == 1 and torch.cuda.mem_get_info(dev)[0] > 3 * gbytes + 8e9:
        nbuf = 2     # room for a second matrix beside the end-to-end staging buffer: the timed steps alternate between two seeds
    Gs = [wl.generate(w_rank, t, dev) for t in range(nbuf)]
    G = Gs[0]
    out = torch.empty(w.d, dtype=w.torch_dtype, device=dev)
    h = ac.AdaCons(w.N, w.d, w.dtype, seg_offsets=wl.segment_offsets(w))
    if args.per_segment:
        h.set_option(ac.OPT_PER_SEGMENT, 1)
    if args.no_overlap_launch:
        h.set_option(ac.OPT_OVERLAP_LAUNCH, 0)
    if args.one_launch >= 0:
        h.set_option(ac.OPT_ONE_LAUNCH, args.one_launch)
    if args.cluster_pass1 >= 0:
        h.set_option(ac.OPT_CLUSTER_PASS1, args.cluster_pass1)
    if args.gram_pass1 >= 0:
        h.set_option(ac.OPT_GRAM_PASS1, args.gram_pass1)
    if args.shifted_loads >= 0:
        h.set_option(ac.OPT_SHIFTED_LOADS, args.shifted_loads)
    if args.tall_tiles >= 0:
        h.set_option(ac.OPT_TALL_TILES, args.tall_tiles)
    stream = torch.cuda.current_stream()
    if args.column_sharded:
        from paper_2411_03742_b200.sharded import ColumnSharded
        sh = ColumnSharded(h, rank, world, device=dev)
        args.no_profile = True        # the two halves are separate calls: only the whole step is timed

        def step_fn(Gt):
            sh.aggregate(Gt, out)
    else:
        def step_fn(Gt):
            h.aggregate(Gt, out)

    for t in range(max(args.warmup, 3)):
        step_fn(Gs[t % nbuf])
    torch.cuda.synchronize()
    # A timed region that saw a thermal or hardware slowdown is measured once more.
    for attempt in range(2):
        if not args.no_profile:
            h.set_option(ac.OPT_PROFILE, 1)          # also clears the recorded samples
        launches0 = h.info(ac.INFO_TOTAL_LAUNCHES)
        sampler = ClockSampler(physical_gpu_index(local))
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        torch.cuda.synchronize()
        sampler.start()
        ev0.record(stream)
        for t in range(args.steps):
            step_fn(Gs[t % nbuf])
        ev1.record(stream)
        torch.cuda.synchronize()
        clocks = sampler.stop()
        barrier()
        ms_local = ev0.elapsed_time(ev1)
        launches = h.info(ac.INFO_TOTAL_LAUNCHES) - launches0
        slowed = any(r in clocks["reasons"] for r in ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown"))
        slowed_anywhere = reduce_over_ranks(1.0 if slowed else 0.0, 0.0, device=dev)[0] > 0.0
        clocks["remeasured"] = attempt > 0
        if not slowed_anywhere:
            break
    if args.no_profile and not args.column_sharded:
        h.set_option(ac.OPT_PROFILE, 1)
        for t in range(args.steps):
            step_fn(Gs[t % nbuf])
        torch.cuda.synchronize()
    kernel_ms, kcalls = ([0.0, 0.0, 0.0], args.steps) if args.column_sharded else h.profile()
    extra = {}
    if not args.no_extra_loops:
        # (a) the launch sequence a user gets: no events between the kernels, so the coefficient
        # kernel's launch overlaps pass 1; (b) one event per step, for the median step time
        h.set_option(ac.OPT_PROFILE, 0)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record(stream)
        for t in range(args.steps):
            step_fn(Gs[t % nbuf])
        e1.record(stream)
        torch.cuda.synchronize()
        extra["ms_per_step_no_kernel_events"] = e0.elapsed_time(e1) / args.steps
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
        evs[0].record(stream)
        for t in range(args.steps):
            step_fn(Gs[t % nbuf])
            evs[t + 1].record(stream)
        torch.cuda.synchronize()
        per = sorted(evs[t].elapsed_time(evs[t + 1]) for t in range(args.steps))
        extra["ms_per_step_median"] = per[len(per) // 2] if len(per) % 2 else 0.5 * (per[len(per) // 2 - 1] + per[len(per) // 2])
        extra["ms_per_step_min_max"] = [per[0], per[-1]]
    status = h.status()
    assert status == 0, f"library raised status flags {status:#x}"
    path = h.info(ac.INFO_LAST_PATH)
    assert path in (1, 3, 4, 5, 6, 7, 9, 10) or (path == 2 and args.shape), "a named workload must run a vectorised path"

    units_local = float(w.N) * w.d * args.steps
    ms, units = reduce_over_ranks(ms_local, units_local, device=dev)
    value = units / (ms * 1e-3)
    b = w.elem_bytes
    step_bytes = 2.0 * w.N * w.d * b + w.d * b
    hbm_gbs = step_bytes * args.steps / (ms_local * 1e-3) / 1e9

    # roofline of the dominant kernel, from CUDA events recorded around it inside the timed region
    peak, peak_src = measured_peak_gbs()
    if args.column_sharded:   # the step as a whole (two calls and, with several ranks, the exchange between them)
        alg = {"step": step_bytes}
        kms = {"step": ms_local / args.steps}
        dom = "step"
    elif path == 3:     # single-pass kernel: the matrix is read from HBM once
        alg = {"fused": float(w.N) * w.d * b + w.d * b}
        kms = {"fused": kernel_ms[0]}
        dom = "fused"
        step_bytes = alg["fused"]
        hbm_gbs = step_bytes * args.steps / (ms_local * 1e-3) / 1e9
    elif path == 5:   # one launch, two reads: only the whole kernel can be timed
        alg = {"one_launch": step_bytes}
        kms = {"one_launch": kernel_ms[0]}
        dom = "one_launch"
    else:
        alg = {"pass1": float(w.N) * w.d * b, "pass2": float(w.N) * w.d * b + w.d * b}
        kms = {"pass1": kernel_ms[0], "coeff": kernel_ms[1], "pass2": kernel_ms[2]}
        dom = "pass1" if kms["pass1"] >= kms["pass2"] else "pass2"
    achieved = alg[dom] / (kms[dom] * 1e-3) / 1e9
    ratio, ratio_src = NCU_TRAFFIC_RATIO.get((w.name, "per segment" if args.per_segment else "model-wise", dom), (None, None))
    roofline = {
        "bound": "hbm", "kernel": dom, "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
        "frac_of_nominal_8tbs": achieved / NOMINAL_HBM_GBS,
        "peak_source": peak_src, "traffic": (ratio * alg[dom] if ratio else None), "traffic_source": ratio_src,
        "algorithmic_bytes_per_launch": alg[dom], "kernel_ms": kms, "timed_calls": kcalls,
        "events_in_timed_region": not args.no_profile,
        "other_kernel_gbs": {k: alg[k] / (kms[k] * 1e-3) / 1e9 for k in alg if k != dom},
    }

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "storage_dtype": w.dtype, "data": "synthetic",
        "config": {"workload": describe(w), "N": w.N, "d": w.d, "storage_dtype": w.dtype,
                   "parallelism": (("column-sharded: every GPU holds all N rows of its own d columns; per step one all-gather "
                                    f"of {h.stats_doubles} doubles per GPU, summed in rank order inside the coefficient kernel")
                                   if args.column_sharded and world > 1 else
                                   "single GPU, the step in two halves (adacons_pass1, adacons_finish)" if args.column_sharded else
                                   "replicas only" if world > 1 else "single GPU"),
                   "coefficients": "per segment" if args.per_segment else "model-wise",
                   "library_options": {k: v for k, v in (("one_launch", args.one_launch), ("cluster_pass1", args.cluster_pass1),
                                                         ("tall_tiles", args.tall_tiles), ("gram_pass1", args.gram_pass1),
                                                         ("shifted_loads", args.shifted_loads)) if v >= 0},
                   "path": {1: "three kernels (TMA-staged pass 1)", 3: "single-pass kernel (matrix in shared memory)",
                            4: "N > 64: column sums, dot products per 64 rows, pass 2 (three reads)",
                            6: "N > 64: cluster pass 1 (one read), coefficient step, pass 2",
                            7: "64 < N <= 256: pass 1 on 128- or 256-row tiles (one read), coefficient step, pass 2",
                            9: "pass 1 from the Gram matrix on the tensor cores, coefficient step, pass 2",
                            2: "scalar kernels (rows at arbitrary offsets, shifted loads switched off or not applicable)",
                            10: "rows at arbitrary offsets: pass 1 with a tensor map per row class, coefficient step, pass 2 with shifted loads",
                            5: "one launch, two reads (pass 1, coefficient step, pass 2 in one cooperative kernel)"}[path],
                   "l2": (f"inputs ({gbytes / 1e9:.2f} GB) larger than the 126 MB L2; no flush between steps" if nbuf == 1 else
                          f"two distinct input matrices of {gbytes / 1e9:.2f} GB used in turn, each larger than the 126 MB L2; no flush"
                          if gbytes >= 8e9 else
                          f"{nbuf} distinct input matrices of {gbytes / 1e9:.3f} GB used in turn ({nbuf * gbytes / 1e9:.2f} GB "
                          "between two uses of one matrix, larger than the 126 MB L2); no flush")},
        "hbm_gbs": hbm_gbs, "hbm_frac_of_measured_copy": hbm_gbs / peak, "hbm_frac_of_nominal_8tbs": hbm_gbs / NOMINAL_HBM_GBS,
        "minimal_bytes_per_step": step_bytes,
        "roofline": roofline, "clocks": clocks, "gpu_launches": int(launches),
    }
    line.update(extra)

    # ---- end to end through the host-buffer entry point -----------------------------------------
    if not args.no_e2e:
        line["e2e"] = run_e2e(h, w, G, dev, args, world)
    del G, Gs
    # ---- CPU oracle on a bounded sample (rank 0, single GPU run only) ---------------------------
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        sec, elems, ws = oracle_sample_steps(w, 3, 1, CPU_BASELINE_COLUMNS)
        line["cpu_baseline"] = {"value": elems / sec, "unit": UNIT, "cores": 1, "kind": "oracle",
                                "sample": f"3 steps of N={ws.N} x {ws.d} columns (float64 numpy, one thread; "
                                          f"host has {os.cpu_count()} cores); {sec:.2f} s per step"}
    if rank == 0:
        print(json.dumps(line), flush=True)
    h.close()
    return 0


def run_e2e(h, w, G, dev, args, world):
    """adacons_aggregate_host: host -> device copy of the whole matrix, the three kernels, device ->
    host copy of the result, every step, timed with the wall clock around the (synchronous) calls."""
    import torch
    b = w.elem_bytes
    need = w.N * w.d * b
    pinned = True
    try:
        with open("/proc/meminfo") as fh:
            avail = next(int(l.split()[1]) * 1024 for l in fh if l.startswith("MemAvailable"))
    except Exception:
        avail = None
    if avail is not None and avail < 1.5 * need * max(1, world):
        return {"value": None, "unit": UNIT, "h2d_bytes_per_step": need, "d2h_bytes_per_step": w.d * b,
                "note": f"skipped: host has {avail / 1e9:.0f} GB available, needs {1.5 * need * world / 1e9:.0f} GB"}
    try:
        Gh = torch.empty((w.N, w.d), dtype=w.torch_dtype, pin_memory=True)
        oh = torch.empty(w.d, dtype=w.torch_dtype, pin_memory=True)
    except RuntimeError:
        pinned = False
        Gh = torch.empty((w.N, w.d), dtype=w.torch_dtype)
        oh = torch.empty(w.d, dtype=w.torch_dtype)
    Gh.copy_(G)
    torch.cuda.synchronize()
    steps = max(1, min(args.steps, 3))
    h.aggregate_host(Gh, oh)          # warm-up: allocates the staging buffer
    barrier()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(steps):
        h.aggregate_host(Gh, oh)
    torch.cuda.synchronize()
    sec_local = time.perf_counter() - t0
    barrier()
    ms, units = reduce_over_ranks(sec_local * 1e3, float(w.N) * w.d * steps, device=dev)
    return {"value": units / (ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": need, "d2h_bytes_per_step": w.d * b,
            "steps": steps, "ms_per_step": ms / steps, "pinned_host_memory": pinned,
            "call": "adacons_aggregate_host (C ABI, host buffers)"}


def main(argv=None):
    args = parse_args(argv)
    if args.impl == "reference":
        return run_reference(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
