#!/usr/bin/env python
"""Benchmark of the DeepSqueeze node update on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg3]
    python bench.py --impl reference ...        # times the CPU checker instead

One "step" is one whole iteration of Algorithm 1 for all n nodes (gradient,
error-compensated compression, residual, gossip mix) on synthetic data of the
workload's shape.  Metric: node-element updates per second (n * N per step).

With N > 1 GPUs the path does not shard (one GPU simulates all nodes), so every
rank runs an independent replica of the workload; the reported value is the sum
of the replicas' updates divided by the slowest rank's time.

Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

from paper_1907_07346_b200 import inputs as I  # noqa: E402

METRIC = "node-element updates/sec per DeepSqueeze step"
UNIT = "updates/s"
FALLBACK_HBM_GBS = 6650.0


def algorithmic_bytes_per_update(w: I.Workload, given_gradient: bool = False) -> float:
    """Read x, delta, a, c (16 B; x, delta, g = 12 B when the gradient is given),
    write x, delta (8 B), write the codes (b/8 B) and one binary32 scale per
    chunk (4/chunk B)."""
    bits = 32 if w.comp_kind == I.COMP_IDENTITY else (1 if w.comp_kind == I.COMP_SIGN1_L1 else w.bits)
    chunk = w.chunk if w.chunk > 0 else w.N
    return (20.0 if given_gradient else 24.0) + bits / 8.0 + 4.0 / chunk


# DRAM bytes per update of the dominant kernel from one ncu capture of a small case
# (dram__bytes_read.sum + dram__bytes_write.sum over one launch of 67,108,864 updates,
# scaled per update), valid for the kernel sources whose digest is recorded beside it.
NCU_TRAFFIC = {"kernel": "ds_fused_tma_kernel", "workload": "cfg3", "bytes_per_update": 1.59492e9 / 67108864,
               "sources_sha256": "4cdbfdb9daee43c8ce108f76b785a0449b103167ccdcf77e02b0c4b9457180cc"}
KERNEL_SOURCES = ["ds_fused_tma_kernel.cuh", "ds_column_kernel.cuh", "ds_device.cuh", "ds_internal.h"]


def kernel_sources_digest() -> str:
    import hashlib
    h = hashlib.sha256()
    for name in KERNEL_SOURCES:
        with open(os.path.join(ROOT, "paper_1907_07346_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons of one GPU with nvidia-smi while
    the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.proc = None
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), [t.strip() for t in line.split(",")]))

    def stop(self, t0: float, t1: float):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        rows = [r for ts, r in self.rows if t0 - 0.05 <= ts <= t1 + 0.15 and len(r) >= 8]
        if not rows:
            rows = [r for _, r in self.rows if len(r) >= 8]
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            try:
                sm.append(float(r[0]))
                smax.append(float(r[1]))
            except ValueError:
                continue
            for name, val in zip(names, r[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(smax) if smax else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def max_over_ranks(ms: float, dist, device) -> float:
    """Slowest rank's device time (every rank gets the same number back)."""
    if dist is None:
        return ms
    import torch
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(world: int, updates_per_step: int, steps: int, total_ms: float) -> float:
    """Updates of all replicas per second of the slowest replica."""
    return world * updates_per_step * steps / (total_ms * 1e-3)


def cpu_baseline(w: I.Workload, a: np.ndarray, c: np.ndarray, sample_cols: int, steps: int = 1,
                 full_N: int | None = None):
    """Time the CPU checker, as it stands, on the first `sample_cols` columns
    of every node of the workload."""
    from oracle import oracle as orc
    g = w.build_graph()
    cols = min(sample_cols, w.N)
    if w.chunk > 0 and cols < w.N:
        cols = max(w.chunk, cols // w.chunk * w.chunk)
    ld = I.round_up(cols, 4)
    aa = np.zeros((w.n, ld), np.float32)
    cc = np.zeros((w.n, ld), np.float32)
    aa[:, :cols] = a[:, :cols]
    cc[:, :cols] = c[:, :cols]
    x = np.zeros((w.n, ld), np.float32)
    d = np.zeros((w.n, ld), np.float32)
    times = []
    for t in range(steps):
        t0 = time.perf_counter()
        orc.step(g, w.comp_kind, w.bits, w.chunk, x, d, aa, cc, cols, w.sigma, w.noise_kind,
                 w.gamma, w.eta, w.seed, t)
        times.append(time.perf_counter() - t0)
    return {"value": w.n * cols * steps / sum(times), "unit": UNIT, "cores": orc.num_threads(),
            "kind": "oracle",
            "sample": f"{steps} step(s) on the first {cols} of {full_N or w.N} parameters of all {w.n} nodes "
                      f"({w.n * cols} updates per step)"}, times


def device_objective(torch, w: I.Workload, ld: int, dev):
    """a, c drawn ON THE DEVICE from the workload's distributions (a ~ U[0.5, 2] or
    10^U[-1, 1], c ~ N(0, 1)), padding columns zero.  For the secondary timing lines
    only: the values do not come from inputs.objective(), which the headline run and
    every parity test use."""
    gen = torch.Generator(device=dev)
    gen.manual_seed(w.seed)
    a = torch.zeros((w.n, ld), dtype=torch.float32, device=dev)
    c = torch.zeros((w.n, ld), dtype=torch.float32, device=dev)
    u = torch.rand((w.n, w.N), generator=gen, dtype=torch.float32, device=dev)
    a[:, :w.N] = 0.5 + 1.5 * u if w.a_dist == "uniform" else torch.pow(10.0, 2.0 * u - 1.0)
    del u
    c[:, :w.N] = torch.randn((w.n, w.N), generator=gen, dtype=torch.float32, device=dev)
    return a, c


def timed_steps(torch, step_fn, first_step: int, steps: int, stream, dev, local_rank: int):
    """Run step_fn(k) for k = first_step .. first_step+steps-1 with a CUDA event after
    every call (on the launching stream) and the clock sampler running; returns
    (per-step ms, total ms, clocks)."""
    sampler = ClockSampler(local_rank)
    sampler.start()
    time.sleep(0.3)
    events = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
    torch.cuda.synchronize(dev)
    t0 = time.time()
    events[0].record(stream)
    for k in range(steps):
        step_fn(first_step + k)
        events[k + 1].record(stream)
    torch.cuda.synchronize(dev)
    t1 = time.time()
    clocks = sampler.stop(t0, t1)
    per_step = [events[k].elapsed_time(events[k + 1]) for k in range(steps)]
    return per_step, events[0].elapsed_time(events[-1]), clocks


KERNEL_OF = {"cfg1": "ds_column_kernel (reduce) + ds_finalize_scales_kernel + ds_fused_tma_kernel",
             "cfg2": "ds_wide_tma_kernel", "cfg3": "ds_fused_tma_kernel", "cfg3_l2": "ds_fused_tma_kernel",
             "cfg4": "ds_fused_tma_pair_kernel", "cfg5": "ds_wide_tma_kernel"}


def other_workload_line(torch, B, name: str, steps: int, dev, local_rank: int, peak: float,
                        algorithm: str = "deepsqueeze", shared=None, noise_kind=None):
    """One secondary timing line: `steps` device-timed steps of another workload (or of
    centralized error-compensated SGD on the headline shape) on its default path.
    noise_kind: the workload with another gradient-noise kind."""
    w = I.WORKLOADS[name]
    if noise_kind is not None:
        w = w.with_size(w.N)
        w.noise_kind = noise_kind
    ld = I.row_pitch(w.N)
    g = w.build_graph()
    stream = torch.cuda.current_stream(dev)
    if shared is not None:
        a, c, x, delta = shared
        x.zero_()
        delta.zero_()
        data = "a, c of the headline run (same shape and distributions)"
    else:
        a, c = device_objective(torch, w, ld, dev)
        x = torch.zeros((w.n, ld), dtype=torch.float32, device=dev)
        delta = torch.zeros_like(x)
        data = "a, c drawn on the device from the workload's distributions (timing only)"
    ds = B.DeepSqueeze(g, w.N, ld, w.comp_kind, w.bits, w.chunk, device=dev)
    info = ds.ds_get_info()

    def step_fn(k):
        if algorithm == "ecsgd":
            ds.ds_ecsgd_step(x, delta, a, c, w.sigma, w.noise_kind, w.gamma, w.seed, k, stream)
        else:
            ds.ds_step(x, delta, a, c, w.sigma, w.noise_kind, w.gamma, w.eta, w.seed, k, stream)

    for k in range(5):
        step_fn(k)
    per_step, total_ms, clocks = timed_steps(torch, step_fn, 5, steps, stream, dev, local_rank)
    ds.ds_sync(stream)
    ok = bool(torch.isfinite(x).all()) and bool(torch.isfinite(delta).all())
    b_alg = algorithmic_bytes_per_update(w)
    ms = total_ms / steps
    achieved = b_alg * w.n * w.N / (ms * 1e-3) / 1e9
    desc = w.describe()
    if w.noise_kind == I.NOISE_STUDENT_T3:
        desc += " [elements 2m, 2m+1 of the t3 noise share one radius: each is t3, the pair is uncorrelated, not independent]"
    if algorithm == "ecsgd":
        desc += " [centralized error-compensated SGD: ds_ecsgd_step]"
    fused = info.path == B.DS_PATH_FUSED
    kernel = (KERNEL_OF.get(name, "?") if fused else "not the TMA-staged path")
    if algorithm == "ecsgd":
        kernel = "ds_fused_tma_kernel (error-compensated SGD instantiation)"
    if noise_kind == I.NOISE_STUDENT_T3_IID and name == "cfg4":
        kernel = "ds_fused_tma_kernel (one node per warp, 1024 threads: the two-nodes-per-warp kernel does not take this noise)"
    line = {"workload": desc, "kernel": kernel, "steps": steps, "ms_per_step": ms,
            "updates_per_s": w.n * w.N / (ms * 1e-3), "algorithmic_bytes_per_update": b_alg,
            "achieved": achieved, "frac": achieved / peak,
            "ms_first_last_10": [statistics.mean(per_step[:10]), statistics.mean(per_step[-10:])],
            "block_threads": info.block_threads, "grid_blocks": info.grid_blocks, "node_batches": info.node_batches,
            "clocks": clocks, "finite": ok, "data": data,
            "l2": "inputs larger than L2" if 16 * w.n * w.N > 4 * 126e6 else "inputs fit in L2: not a roofline point"}
    ds.close()
    return line


def guarded_line(what: str, fn, *a, **kw):
    """A secondary line must never cost the headline: a failure becomes an entry that says so."""
    try:
        return fn(*a, **kw)
    except Exception as err:            # noqa: BLE001 (reported, not swallowed)
        return {"workload": what, "error": f"{type(err).__name__}: {err}"}


def run_reference(args, w: I.Workload):
    """The reference arm: the CPU checker on a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    sample = w.with_size(min(w.N, args.ref_cols) if args.ref_cols > 0 else w.N)
    a, c = I.objective(sample, I.row_pitch(sample.N))
    total = args.warmup + args.steps
    base, times = cpu_baseline(sample, a, c, sample.N, steps=total, full_N=w.N)
    timed = times[args.warmup:]
    value = sample.n * sample.N * len(timed) / sum(timed)
    base["value"] = value
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": 1e3 * sum(timed) / len(timed),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic", "impl": "reference",
            "config": {"workload": w.describe(), "timed_sample": base["sample"]},
            "cpu_baseline": base,
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="cfg3", choices=sorted(I.WORKLOADS))
    ap.add_argument("--size", type=int, default=0, help="override N (parameters per node)")
    ap.add_argument("--path", default="auto", choices=["auto", "fused", "fused_ldg", "split"])
    ap.add_argument("--algorithm", default="deepsqueeze", choices=["deepsqueeze", "ecsgd"],
                    help="deepsqueeze: Algorithm 1 (the default, the headline metric); ecsgd: centralized "
                         "error-compensated SGD of Section 1 (ds_ecsgd_step, two kernels per step)")
    ap.add_argument("--runner", default="step", choices=["step", "graph", "resident"],
                    help="step: one ds_step call per iteration (the default); graph: all iterations as one ds_run "
                         "call (a replayed CUDA graph); resident: all iterations as one ds_run_resident launch "
                         "(small shapes only)")
    ap.add_argument("--elems-per-lane", type=int, default=0, help="tuning knob (0 = library default)")
    ap.add_argument("--given-gradient", action="store_true",
                    help="time ds_step_g (gradient read from memory) instead of the synthetic objective")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--cpu-steps", type=int, default=3, help="steps of the CPU-baseline sample")
    ap.add_argument("--cpu-cols", type=int, default=1 << 25,
                    help="columns per node of the CPU-baseline sample")
    ap.add_argument("--ref-cols", type=int, default=0,
                    help="columns per node of each step of --impl reference (0 = the whole workload)")
    ap.add_argument("--sustained-steps", type=int, default=1000,
                    help="steps of the sustained leg run after the headline region (0 = skip; 1 GPU only)")
    ap.add_argument("--other-steps", type=int, default=50,
                    help="timed steps of each secondary workload line (0 = skip; 1 GPU only)")
    ap.add_argument("--cpu-single-cols", type=int, default=1 << 20,
                    help="columns per node of the one-thread CPU-baseline sample (0 = skip)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3

    w = I.WORKLOADS[args.workload]
    if args.size:
        w = w.with_size(args.size)
    if args.impl == "reference":
        run_reference(args, w)
        return

    import torch
    from paper_1907_07346_b200 import binding as B

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1 or "TORCHELASTIC_RUN_ID" in os.environ:      # launched by torch.distributed.run
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    g = w.build_graph()
    ld = I.row_pitch(w.N)
    a_h, c_h = I.objective(w, ld)
    ds = B.DeepSqueeze(g, w.N, ld, w.comp_kind, w.bits, w.chunk, device=dev)
    ds.ds_set_path({"auto": B.DS_PATH_AUTO, "fused": B.DS_PATH_FUSED, "fused_ldg": B.DS_PATH_FUSED_LDG,
                    "split": B.DS_PATH_SPLIT}[args.path])
    if args.elems_per_lane:
        ds.ds_tune(args.elems_per_lane)
    info = ds.ds_get_info()
    a = torch.from_numpy(a_h).to(dev)
    c = torch.from_numpy(c_h).to(dev)
    x = torch.zeros((w.n, ld), dtype=torch.float32, device=dev)
    delta = torch.zeros_like(x)
    stream = torch.cuda.current_stream(dev)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize(dev)

    def one_step(k):
        if args.algorithm == "ecsgd":
            ds.ds_ecsgd_step(x, delta, a, c, w.sigma, w.noise_kind, w.gamma, w.seed, k, stream)
        elif args.given_gradient:       # a stands in for the caller's gradient array
            ds.ds_step_g(x, delta, a, w.gamma, w.eta, w.seed, k, stream)
        else:
            ds.ds_step(x, delta, a, c, w.sigma, w.noise_kind, w.gamma, w.eta, w.seed, k, stream)

    def many_steps(k, count):
        """count iterations from step k as ONE call: a replayed CUDA graph or the resident kernel."""
        run = ds.ds_run if args.runner == "graph" else ds.ds_run_resident
        run(x, delta, a, c, w.sigma, w.noise_kind, [w.gamma] * count, [w.eta] * count, w.seed, k, stream)

    step_index = 0
    if args.runner == "step":
        for _ in range(args.warmup):
            one_step(step_index)
            step_index += 1
    else:
        for _ in range(3):                       # same count as the timed call, so the graph is instantiated once
            many_steps(step_index, args.steps)
            step_index += args.steps
    barrier()

    sampler = ClockSampler(local_rank)
    sampler.start()
    time.sleep(0.3)
    events = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    barrier()
    t_wall0 = time.time()
    events[0].record(stream)
    if args.runner == "step":
        for k in range(args.steps):
            one_step(step_index)
            step_index += 1
            events[k + 1].record(stream)
    else:
        many_steps(step_index, args.steps)
        step_index += args.steps
        events[-1].record(stream)
    barrier()
    t_wall1 = time.time()
    clocks = sampler.stop(t_wall0, t_wall1)
    total_ms = events[0].elapsed_time(events[-1])
    if args.runner == "step":
        per_step = [events[k].elapsed_time(events[k + 1]) for k in range(args.steps)]
    else:
        per_step = [total_ms / args.steps] * args.steps
    total_ms = max_over_ranks(total_ms, dist, dev)
    updates_per_step = w.n * w.N
    value = whole_job_value(world, updates_per_step, args.steps, total_ms)
    ds.ds_sync(stream)
    assert torch.isfinite(x).all() and torch.isfinite(delta).all()

    # Roofline of the dominant kernel.  On the fused path a step IS one launch
    # of the column kernel, so its average duration is the event time per step.
    b_alg = algorithmic_bytes_per_update(w, args.given_gradient)
    # ds_ecsgd_step runs as one fused launch where the persistent kernel takes the shape with 16 elements per lane
    ecsgd_fused = (args.algorithm == "ecsgd" and args.path == "auto" and info.path == B.DS_PATH_FUSED
                   and info.elems_per_lane == 16 and info.block_threads <= 512 and info.node_batches == 1)
    peak, peak_kind = measured_peak()
    kernel_ms = statistics.mean(per_step)
    traffic = None      # per launch; null once the kernel sources differ from the profiled ones
    if (not args.given_gradient and info.path == B.DS_PATH_FUSED and args.workload == NCU_TRAFFIC["workload"] and not args.elems_per_lane
            and args.runner == "step" and args.algorithm == "deepsqueeze" and kernel_sources_digest() == NCU_TRAFFIC["sources_sha256"]):
        traffic = NCU_TRAFFIC["bytes_per_update"] * updates_per_step
    # `achieved` counts ALGORITHMIC bytes (what the step must move); `achieved_dram` counts the
    # DRAM bytes the profiler saw for this kernel (less than algorithmic when the last written
    # lines are still dirty in L2 at the end of the one captured launch).
    achieved = b_alg * updates_per_step / (kernel_ms * 1e-3) / 1e9
    achieved_dram = None if traffic is None else traffic / (kernel_ms * 1e-3) / 1e9
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "traffic": traffic, "peak_source": f"of {peak_kind}",
                "achieved_alg": achieved, "achieved_dram": achieved_dram,
                "frac_dram": None if achieved_dram is None else achieved_dram / peak,
                "kernel": "ds_resident_kernel" if args.runner == "resident" else
                          "ds_fused_tma_kernel (error-compensated SGD instantiation)" if ecsgd_fused else
                          "ds_column_kernel (compress, g + delta) + ds_mix_kernel (server update)" if args.algorithm == "ecsgd" else
                          {B.DS_PATH_FUSED: "ds_fused_tma_kernel", B.DS_PATH_FUSED_LDG: "ds_column_kernel (fused)",
                           B.DS_PATH_SPLIT: "ds_column_kernel (compress) + ds_mix_kernel"}[info.path],
                "algorithmic_bytes_per_update": b_alg,
                "algorithmic_bytes_per_launch": b_alg * updates_per_step,
                "kernel_ms_mean": kernel_ms, "kernel_ms_min": min(per_step),
                "kernel_ms_median": statistics.median(per_step),
                "kernel_ms_first_last_10": [statistics.mean(per_step[:10]), statistics.mean(per_step[-10:])],
                "frac_of_nominal_8TBs": achieved / 8000.0}

    # Sustained leg: the same kernel for long enough (>= 1.5 s) that the board's power
    # management has settled; the headline region above is a short burst.
    if world == 1 and args.sustained_steps > 0 and args.runner == "step":
        sus_ms, sus_total, sus_clocks = timed_steps(torch, one_step, step_index, args.sustained_steps, stream, dev,
                                                    local_rank)
        step_index += args.sustained_steps
        sus = sus_total / args.sustained_steps
        sus_ach = b_alg * updates_per_step / (sus * 1e-3) / 1e9
        roofline["sustained"] = {"steps": args.sustained_steps, "timed_region_s": sus_total * 1e-3, "ms_per_step": sus,
                                 "updates_per_s": updates_per_step / (sus * 1e-3),
                                 "achieved": sus_ach, "frac": sus_ach / peak,
                                 "ms_first_last_10": [statistics.mean(sus_ms[:10]), statistics.mean(sus_ms[-10:])],
                                 "sm_mhz": sus_clocks.get("sm_mhz"), "sm_max_mhz": sus_clocks.get("sm_max_mhz"),
                                 "reasons": sus_clocks.get("reasons"), "samples": sus_clocks.get("samples")}
        ds.ds_sync(stream)

    # End to end through the host-buffer entry point: pinned host arrays in,
    # x and delta back out, every step.
    e2e = None
    if not args.no_e2e and not args.given_gradient and args.algorithm == "deepsqueeze":
        hx = torch.zeros((w.n, ld), dtype=torch.float32).pin_memory()
        hd = torch.zeros((w.n, ld), dtype=torch.float32).pin_memory()
        ha = torch.from_numpy(a_h).pin_memory()
        hc = torch.from_numpy(c_h).pin_memory()
        for t in range(2):
            ds.ds_step_host(hx, hd, ha, hc, w.sigma, w.noise_kind, w.gamma, w.eta, w.seed, t,
                            x, delta, a, c, stream)
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for t in range(args.e2e_steps):
            ds.ds_step_host(hx, hd, ha, hc, w.sigma, w.noise_kind, w.gamma, w.eta, w.seed, 2 + t,
                            x, delta, a, c, stream)
        e1.record(stream)
        barrier()
        e2e_ms = max_over_ranks(e0.elapsed_time(e1), dist, dev)
        arr_bytes = w.n * ld * 4
        e2e = {"value": whole_job_value(world, updates_per_step, args.e2e_steps, e2e_ms), "unit": UNIT,
               "h2d_bytes_per_step": 4 * arr_bytes, "d2h_bytes_per_step": 2 * arr_bytes,
               "steps": args.e2e_steps, "ms_per_step": e2e_ms / args.e2e_steps,
               "entry_point": "ds_step_host (pinned host x, delta, a, c in; x, delta out; slabs of column tiles "
                              "pipelined: copy in / compute / copy out overlap)"}
        del hx, hd, ha, hc

    # Secondary lines: the other workloads (and the headline shape's other modes), each on its
    # default path, device-timed; context for the headline, not part of `value`.
    others = None
    if world == 1 and args.other_steps > 0 and args.workload == "cfg3" and not args.size and args.path == "auto" \
            and args.algorithm == "deepsqueeze" and not args.given_gradient and not args.elems_per_lane:
        others = []
        shared = (a, c, x, delta)
        others.append(guarded_line("cfg3 ecsgd", other_workload_line, torch, B, "cfg3", args.other_steps, dev, local_rank, peak, "ecsgd", shared))
        others.append(guarded_line("cfg3_l2", other_workload_line, torch, B, "cfg3_l2", args.other_steps, dev, local_rank, peak, shared=shared))
        ds.close()
        del shared, a, c, x, delta
        torch.cuda.empty_cache()
        for name in ("cfg2", "cfg4", "cfg5"):
            others.append(guarded_line(name, other_workload_line, torch, B, name, args.other_steps, dev, local_rank, peak))
            torch.cuda.empty_cache()
        # cfg4 with independent Student-t(3) coordinates (four normals per element): the reading of
        # "Student-t(3) gradient noise" that is bound by the instruction stream instead of memory
        others.append(guarded_line("cfg4 independent t3", other_workload_line, torch, B, "cfg4",
                                   max(10, args.other_steps // 5), dev, local_rank, peak, noise_kind=I.NOISE_STUDENT_T3_IID))
        torch.cuda.empty_cache()

    base = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        base, _ = cpu_baseline(w, a_h, c_h, args.cpu_cols, steps=args.cpu_steps)
        if args.cpu_single_cols > 0:
            from oracle import oracle as orc
            threads = orc.num_threads()
            orc.set_num_threads(1)
            try:
                single, _ = cpu_baseline(w, a_h, c_h, args.cpu_single_cols, steps=1)
            finally:
                orc.set_num_threads(threads)
            base["single_thread"] = {"value": single["value"], "unit": UNIT, "cores": 1, "sample": single["sample"]}

    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": total_ms / args.steps, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                "config": {"workload": w.describe() + (" [gradient given: ds_step_g]" if args.given_gradient else "")
                           + (" [centralized error-compensated SGD: ds_ecsgd_step]" if args.algorithm == "ecsgd" else ""),
                           "row_pitch": ld,
                           "path": {B.DS_PATH_FUSED: "fused (persistent, TMA-staged)",
                                    B.DS_PATH_FUSED_LDG: "fused (direct loads)", B.DS_PATH_SPLIT: "split"}[info.path],
                           "elems_per_lane": info.elems_per_lane, "warps_per_chunk": info.warps_per_chunk,
                           "block_threads": info.block_threads, "grid_blocks": info.grid_blocks,
                           "l2": "inputs larger than L2 (no flush needed)"
                                 if 16 * updates_per_step > 4 * 126e6 else "inputs fit in L2: not a roofline point",
                           "replicas": world},
                "clocks": clocks, "e2e": e2e, "gpu_launches": 1 if args.runner == "resident" else args.steps * (((1 if ecsgd_fused else 2) + (2 if w.chunk == 0 and w.comp_kind != I.COMP_IDENTITY else 0)) if args.algorithm == "ecsgd" else info.launches_per_step),
                "runner": args.runner, "roofline": roofline, "cpu_baseline": base, "other_workloads": others}
        print(json.dumps(line))
    ds.close()
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
