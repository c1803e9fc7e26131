#!/usr/bin/env python
"""Benchmark of the fused GEMM + epilogue + row-reduce operator on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config all|c1..c5|...] [--impl ours|reference]

One step = one pass of the whole hot path (GEMM mainloop, fused epilogue, per-tile row reduction,
split-N merge / softmax normalisation) over one seeded synthetic problem of the named workload.
Rank 0 prints ONE JSON line.  The default (--config all) times the five named workloads one after
the other, W warm-up and K timed steps each: the top-level keys describe the largest one (c3) and
"per_config" carries the record of every workload, "targets_met" the whole-step roofline fractions
against the stated targets.  --config NAME times that workload alone.

With N > 1 every rank runs its own problems on its own GPU (rows / batches are independent: no
collective on the data path; weak scaling).  `python bench.py --gpus N` without a launcher starts
the N ranks itself (torch.distributed.run on 127.0.0.1); under torchrun it uses the ranks it is given.

Timing: W warm-up steps, then K steps between two CUDA events on the launching stream, bracketed
by a barrier and a device synchronise; max over ranks.  Consecutive steps use different input and
output buffers (a rotation larger than the 126 MB L2), so no step finds its operands in L2.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

L2_BYTES = 126e6
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
METRIC = "fused GEMM+epilogue+rowreduce TFLOP/s (or GB/s) and % of roofline, 1 B200"
HBM_BOUND = {"c4", "g2"}
# extra workloads of the fused operator beside the five named ones: the skinny CUDA-core GEMV path
EXTRA_CONFIGS = {"g2": ("c4", dict(M=2)),     # c4's shapes and epilogue with M = 2
                 "f2": ("c2", dict(dtype=0)),  # c2's shapes and epilogue with fp32 inputs and outputs: the 3xTF32 path
                 # 1-D convolution with c2's epilogue: 8 signals of 2051 x 512 channels, 4096 filters of 4 taps (shared)
                 "v2": ("c2", dict(batch=8, M=2048, N=4096, K=2048, conv_taps=4, w_shared=1)),
                 # 2-D convolution with c2's epilogue: 16 images of 66 x 66 x 64 channels, 1024 shared filters of 3 x 3
                 # (64 x 64 outputs per image at the image's row pitch: M = 63 * 66 + 64 rows, 3 % of them unused)
                 "v3": ("c2", dict(batch=16, M=63 * 66 + 64, N=1024, K=3 * 3 * 64, conv_rows=3, conv_taps=3, conv_width=66, w_shared=1))}


def make_cfg(name, **kw):
    import fgr_inputs as gi
    if name in EXTRA_CONFIGS:
        base, over = EXTRA_CONFIGS[name]
        p = gi.make_config(base, **dict(over, **kw))
        p.name = name
        return p
    return gi.make_config(name, **kw)


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            d = json.load(f)
        return {k: float(d[k]) for k in FALLBACK_PEAKS}, "measured"
    except Exception:
        return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the GPU works."""

    def __init__(self, index: int, period_s: float = 0.001):
        self.index, self.period = index, period_s
        self.samples = []          # (host time, sm MHz, reasons bitmask)
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        self.ok = False
        try:
            import pynvml
            self.nv = pynvml
            pynvml.nvmlInit()
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception:
            self.ok = False

    def _run(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                mhz = nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)
                try:
                    reasons = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    reasons = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                self.samples.append((time.perf_counter(), float(mhz), int(reasons)))
            except Exception:
                pass
            self._stop.wait(self.period)

    def start(self):
        if self.ok:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def stop(self):
        if self._thread:
            self._stop.set()
            self._thread.join()

    def summary(self, t0: float, t1: float):
        if not self.ok or not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": ["unavailable"], "samples": 0}
        inside = [s for s in self.samples if t0 <= s[0] <= t1]
        window = "timed region"
        if len(inside) < 3:        # a very short region: fall back to everything sampled under load
            inside, window = self.samples, "warm-up + timed region"
        mhz = sorted(s[1] for s in inside)
        bits = 0
        for s in inside:
            bits |= s[2]
        names = {0x1: "gpu_idle", 0x2: "applications_clocks_setting", 0x4: "sw_power_cap", 0x8: "hw_slowdown",
                 0x10: "sync_boost", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
                 0x80: "hw_power_brake_slowdown", 0x100: "display_clock_setting"}
        reasons = [n for b, n in names.items() if bits & b and n != "gpu_idle"]
        return {"sm_mhz": mhz[len(mhz) // 2], "sm_max_mhz": self.max_mhz, "reasons": reasons,
                "samples": len(inside), "window": window}


def max_over_ranks(x: float, world: int, device=None) -> float:
    """Maximum of a per-rank scalar over all ranks (the slowest rank defines the step time)."""
    if world <= 1:
        return float(x)
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(x)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def rank_seeds(rank: int, rotation: int):
    """Seeds of the `rotation` distinct problems rank `rank` cycles through: no two ranks share one."""
    return [1000 * rank + r for r in range(rotation)]


def dist_env():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


class Ctx:
    """What every leg of the benchmark shares: the rank layout, the device, the process group, the peaks."""

    def __init__(self, backend: str = "nccl", use_gpu: bool = True):
        self.rank, self.local_rank, self.world = dist_env()
        self.peaks, self.peak_src = load_peaks()
        self.dev = None
        if use_gpu:
            import torch
            if not torch.cuda.is_available():
                raise SystemExit("bench.py needs a CUDA device: the operator has no CPU path")
            torch.cuda.set_device(self.local_rank)
            self.dev = torch.device("cuda", self.local_rank)
        if self.world > 1:
            import torch.distributed as dist
            if backend == "nccl":
                dist.init_process_group("nccl", device_id=self.dev)
            else:
                dist.init_process_group(backend)

    def barrier(self):
        if self.world > 1:
            import torch.distributed as dist
            dist.barrier()
        if self.dev is not None:
            import torch
            torch.cuda.synchronize(self.dev)

    def close(self):
        if self.world > 1:
            import torch.distributed as dist
            dist.destroy_process_group()


def launch_ranks(n: int) -> int:
    """`python bench.py --gpus N` without a launcher: start N local ranks of this same command line
    (one per GPU, rendezvous on 127.0.0.1) and pass their output through."""
    import socket
    import subprocess
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(n),
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def oracle_sample(p, seconds: float):
    """Times the CPU oracle, as it stands, on a leading block of rows sized for about `seconds`."""
    import numpy as np
    import oracle
    total = p.batch * p.M
    probe = min(total, 16)
    t = time.perf_counter()
    _, _, threads = oracle.run_problem(p, rows=np.arange(probe), want_y=False)
    dt = max(time.perf_counter() - t, 1e-4)
    rows = int(max(probe, min(total, probe * seconds / dt)))
    stride = max(1, total // rows)
    idx = (np.arange(rows) * stride) % total
    t = time.perf_counter()
    oracle.run_problem(p, rows=idx, want_y=False)
    dt = time.perf_counter() - t
    flop = 2.0 * rows * p.N * p.K
    return flop, dt, threads, rows


def unit_and_value(cfg, p, seconds_per_step, n_problems=1):
    if cfg in HBM_BOUND:
        return "GB/s", n_problems * p.min_bytes() / seconds_per_step / 1e9
    return "TFLOP/s", n_problems * p.flop / seconds_per_step / 1e12


ACT_NAMES = ["none", "relu", "gelu_tanh", "sigmoid", "tanh", "silu"]
SCALE_NAMES = ["none", "scalar", "per_column"]
REDUCE_NAMES = {0: "lse", 1: "softmax", 2: "maxsum", 3: "max_sumexp", 6: "meanvar"}


def shape_keys(cfg, p):
    """The keys of `config` that name the workload itself (both arms print exactly these)."""
    import fgr_inputs as gi
    return {"workload": cfg, "batch": p.batch, "M": p.M, "N": p.N, "K": p.K, "act": ACT_NAMES[p.act],
            "scale": SCALE_NAMES[p.scale_kind], "reduce": REDUCE_NAMES[p.reduce],
            "write_y": int(bool(p.write_y) or p.reduce == gi.RED_SOFTMAX), "conv_taps": p.conv_taps, "w_shared": p.w_shared,
            "conv_rows": p.conv_rows, "conv_width": p.conv_width}


def run_reference(args):
    rank, _, world = dist_env()
    if rank != 0:
        return
    cfg = HEADLINE if args.config == "all" else args.config
    p = make_cfg(cfg, seed=0)
    per_step = min(2.0, 60.0 / max(args.steps, 1))   # the whole run stays near a minute of CPU time
    threads = rows = 0
    for _ in range(max(args.warmup, 0)):
        oracle_sample(p, 0.2)
    f_sum = t_sum = 0.0
    for _ in range(args.steps):
        flop, dt, threads, rows = oracle_sample(p, per_step)
        f_sum += flop
        t_sum += dt
    if cfg in HBM_BOUND:
        unit, value = "GB/s", (f_sum / p.flop) * p.min_bytes() / t_sum / 1e9
    else:
        unit, value = "TFLOP/s", f_sum / t_sum / 1e12
    sample = "%d of %d rows per step (every %d-th row), all N and K" % (rows, p.batch * p.M, max(1, p.batch * p.M // rows))
    config = shape_keys(cfg, p)
    config["note"] = "CPU fp64 oracle on a bounded row sample"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": unit, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * t_sum / max(args.steps, 1), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config,
        "cpu_baseline": {"value": value, "unit": unit, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": unit, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


HEADLINE = "c3"                                     # the largest of the five named workloads
NAMED = ["c1", "c2", "c3", "c4", "c5"]
TARGETS = {"c2": 0.60, "c3": 0.60, "c5": 0.60, "c4": 0.70}   # whole-step fraction of the measured peak


def empty_launch_us(ctx, n: int = 200) -> float:
    """Mean time of one launch of an empty kernel in a back-to-back stream of n: the floor under any
    step that is bound by launch latency (c1)."""
    import torch
    import paper_2511_06345_b200 as fgr
    stream = torch.cuda.current_stream(ctx.dev).cuda_stream
    fgr.fgr_profile_empty_launches(16, ctx.local_rank, stream)
    torch.cuda.synchronize(ctx.dev)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    fgr.fgr_profile_empty_launches(n, ctx.local_rank, stream)
    e1.record()
    torch.cuda.synchronize(ctx.dev)
    return e0.elapsed_time(e1) * 1e3 / n


def measure_fused(cfg, args, ctx, with_e2e=True, with_cpu=True):
    """Times one workload of the fused operator; returns the record rank 0 prints (None elsewhere)."""
    import numpy as np
    import torch
    import fgr_inputs as gi
    import paper_2511_06345_b200 as fgr

    rank, local_rank, world, dev = ctx.rank, ctx.local_rank, ctx.world, ctx.dev
    peaks, peak_src = ctx.peaks, ctx.peak_src
    warmup = max(args.warmup, 3)

    sampler = ClockSampler(local_rank)
    # ---- inputs: a rotation of distinct problems so that no step finds its operands in L2
    shape = make_cfg(cfg, materialize=False)
    set_bytes = shape.min_bytes()
    rot = max(2, int(math.ceil(2.4 * L2_BYTES / set_bytes)) + 1)
    rot = min(rot, 8)
    b16 = shape.dtype == gi.DTYPE_BF16
    tdt = torch.bfloat16 if b16 else torch.float32

    def up(a, bits16):
        t = torch.from_numpy(np.ascontiguousarray(a))
        if bits16:
            t = t.view(torch.int16).view(torch.bfloat16)
        return t.to(dev)

    sets = []
    host0 = None
    for r, seed in enumerate(rank_seeds(rank, rot)):
        p = make_cfg(cfg, seed=seed)
        if r == 0:
            host0 = p
        sets.append(dict(X=up(p.X, b16), W=up(p.W, b16),
                         bias=None if p.bias is None else up(p.bias, False),
                         scale=None if p.scale_vec is None else up(p.scale_vec, False)))
    p = host0
    need_y = bool(p.write_y) or p.reduce == gi.RED_SOFTMAX
    rows = p.batch * p.M
    for s in sets:
        s["Y"] = torch.empty((p.batch, p.M, p.N), dtype=tdt, device=dev) if need_y else None
        s["out"] = torch.empty((rows, p.out_width), dtype=torch.float32, device=dev) if p.out_width else None

    desc = fgr.make_desc(p.batch, p.M, p.N, p.K, p.dtype, p.act, p.scale_kind, p.reduce, scale=p.scale,
                         write_y=p.write_y, bias_per_batch=p.bias_per_batch, device=local_rank,
                         conv_taps=p.conv_taps, w_shared=p.w_shared, conv_rows=p.conv_rows, conv_width=p.conv_width)
    h = fgr.fgr_create(desc)
    plan = fgr.fgr_get_plan(h)
    ws_bytes = fgr.fgr_workspace_bytes(h)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream(dev).cuda_stream

    def step(i):
        s = sets[i % rot]
        fgr.fgr_run(h, s["X"], s["W"], s["bias"], s["scale"], s["Y"], s["out"], ws, ws_bytes, stream)

    sampler.start()
    for i in range(warmup):
        step(i)
    ctx.barrier()
    # ---- the timed region: K steps, nothing else on the stream
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_host0 = time.perf_counter()
    e0.record()
    for i in range(args.steps):
        step(i)
    e1.record()
    ctx.barrier()
    status = fgr.fgr_get_status(h)
    if status != fgr.FGR_OK:
        raise SystemExit("device status after the timed region: " + fgr.fgr_status_string(status))
    ms_total = max_over_ranks(e0.elapsed_time(e1), world, dev)
    # ---- the same K steps again with a CUDA event before and after every main-kernel launch
    # (recorded inside fgr_run): the duration of the dominant kernel for the roofline.  Kept out of
    # the region above because an event between two launches undoes their overlap.
    fgr.fgr_profile_enable(h, True)
    for i in range(args.steps):
        step(i)
    ctx.barrier()
    t_host2 = time.perf_counter()
    sampler.stop()
    fgr.fgr_profile_enable(h, False)
    kern_ms, kern_runs = fgr.fgr_profile_read(h)
    ms_step = ms_total / args.steps
    unit, value = unit_and_value(cfg, p, ms_step * 1e-3, n_problems=world)
    clocks = sampler.summary(t_host0, t_host2)

    # ---- roofline of the dominant kernel (the main GEMM + epilogue launch)
    kern_s = (kern_ms / max(kern_runs, 1)) * 1e-3
    if cfg in HBM_BOUND:
        roof = {"bound": "hbm", "achieved": p.min_bytes() / kern_s / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s"}
    else:
        roof = {"bound": "tensor", "achieved": p.flop / kern_s / 1e12, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                "frac_of_sustained_peak": p.flop / kern_s / 1e12 / peaks["bf16_tflops_sustained"]}
        if plan.path == fgr.FGR_PATH_UMMA_TF32X3:
            # fp32 result from three tf32 products: the peak for algorithmic (fp32) flop is the tf32 rate / 3;
            # the tf32 rate is the measured bf16 rate times the nominal tf32 : bf16 ratio (1.1 : 2.25 PFLOP/s)
            roof["peak"] = peaks["bf16_tflops"] * (1.1 / 2.25) / 3.0
            roof["frac_of_sustained_peak"] = roof["achieved"] / (peaks["bf16_tflops_sustained"] * (1.1 / 2.25) / 3.0)
            roof["peak_note"] = "measured bf16 rate x 1.1/2.25 (nominal tf32 : bf16) / 3 products per fp32 product"
    roof["frac"] = roof["achieved"] / roof["peak"]
    # the whole step (every launch of fgr_run, one GPU's share of the job) against the same peak
    roof["step_frac"] = value / world / roof["peak"]
    roof["peak_source"] = peak_src + (" (burst)" if roof["bound"] == "tensor" else "")
    roof["kernel"] = {fgr.FGR_PATH_UMMA_TILED: "umma_kernel", fgr.FGR_PATH_UMMA_STREAM_W: "umma_kernel",
                      fgr.FGR_PATH_SIMT_GEMV: "gemv_kernel", fgr.FGR_PATH_UMMA_TF32X3: "umma_kernel (tf32)"}.get(plan.path, "simt_gemm_kernel")
    roof["kernel_us"] = kern_s * 1e6
    roof["timing"] = "CUDA events around each of %d launches of the kernel, in a second pass of the same steps" % kern_runs
    roof["traffic"] = TRAFFIC.get(cfg)
    if cfg == "c1":
        # launch-latency bound: the fractions above mean little; the floor is the cost of a launch
        roof["note"] = "launch-latency bound (33.6 Mflop): compare the step with empty_launch_us x launches per step"
        roof["empty_launch_us"] = empty_launch_us(ctx)
        roof["launches_per_step"] = plan.launches

    # ---- end to end: host buffers through fgr_run_host, copies inside the timed region
    e2e = None
    if with_e2e:
        hp = {k: (None if v is None else v.cpu().pin_memory()) for k, v in sets[0].items()}
        e2e_steps = max(3, min(args.steps, 20))
        for _ in range(2):
            fgr.fgr_run_host(h, hp["X"], hp["W"], hp["bias"], hp["scale"], hp["Y"], hp["out"])
        ctx.barrier()
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            fgr.fgr_run_host(h, hp["X"], hp["W"], hp["bias"], hp["scale"], hp["Y"], hp["out"])
        torch.cuda.synchronize(dev)
        dt = (time.perf_counter() - t0) / e2e_steps
        dt = max_over_ranks(dt, world, dev)
        eu, ev = unit_and_value(cfg, p, dt, n_problems=world)
        h2d = sum(hp[k].numel() * hp[k].element_size() for k in ("X", "W", "bias", "scale") if hp[k] is not None)
        d2h = sum(hp[k].numel() * hp[k].element_size() for k in ("Y", "out") if hp[k] is not None)
        e2e = {"value": ev, "unit": eu, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps,
               "ms_per_step": dt * 1e3}
        del hp
    fgr.fgr_destroy(h)
    del sets, ws
    torch.cuda.empty_cache()

    # ---- the CPU oracle timed beside it (rank 0, single-GPU runs only)
    cpu = None
    if rank == 0 and world == 1 and with_cpu:
        flop, dt, threads, nrows = oracle_sample(p, 12.0)
        if cfg in HBM_BOUND:
            cu, cv = "GB/s", (flop / p.flop) * p.min_bytes() / dt / 1e9
        else:
            cu, cv = "TFLOP/s", flop / dt / 1e12
        cpu = {"value": cv, "unit": cu, "cores": threads, "kind": "oracle", "seconds": dt,
               "sample": "%d of %d rows (evenly spaced), all N and K, fp64 triple loop" % (nrows, rows)}

    if rank != 0:
        return None
    config = shape_keys(cfg, p)
    config.update({"path": fgr.fgr_path_name(plan.path), "tile": [plan.tile_m, plan.tile_n], "stages": plan.stages,
                   "grid": plan.grid, "l2": "rotating %d distinct input/output sets (%.0f MB > 126 MB L2)" % (rot, rot * set_bytes / 1e6),
                   "parallelism": "independent problems per GPU, no collective" if world > 1 else "1 GPU"})
    line = {
        "metric": METRIC, "value": value, "unit": unit, "n_gpus": world, "steps": args.steps, "warmup": warmup,
        "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if b16 else ("tf32x3" if plan.path == fgr.FGR_PATH_UMMA_TF32X3 else "f32"), "data": "synthetic",
        "config": config, "clocks": clocks, "gpu_launches": args.steps * plan.launches, "roofline": roof,
    }
    if e2e is not None:
        line["e2e"] = e2e
    if cpu is not None:
        line["cpu_baseline"] = cpu
    return line


def run_ours(args, ctx):
    line = measure_fused(args.config, args, ctx, with_e2e=not args.no_e2e, with_cpu=not args.no_cpu_baseline)
    if line is not None:
        print(json.dumps(line))


def run_all(args, ctx):
    """The default: every named workload, W warm-up + K timed steps each.  The top level of the line is
    the record of the largest workload; per_config holds all five, trimmed to what differs."""
    records = {}
    for cfg in NAMED:
        head = cfg == HEADLINE
        records[cfg] = measure_fused(cfg, args, ctx, with_e2e=head and not args.no_e2e,
                                     with_cpu=head and not args.no_cpu_baseline)
    if ctx.rank != 0:
        return
    line = dict(records[HEADLINE])
    per, met = {}, {}
    for cfg in NAMED:
        r = records[cfg]
        per[cfg] = {k: r[k] for k in ("value", "unit", "ms_per_step", "dtype", "config", "clocks", "gpu_launches", "roofline")}
        if cfg in TARGETS:
            f = r["roofline"]["step_frac"]
            met[cfg] = {"bound": r["roofline"]["bound"], "step_frac": f, "kernel_frac": r["roofline"]["frac"],
                        "target": TARGETS[cfg], "met": bool(f >= TARGETS[cfg])}
    line["per_config"] = per
    line["targets_met"] = met
    line["gpu_launches"] = sum(r["gpu_launches"] for r in records.values())
    line["gpu_launches_note"] = "kernels launched inside the five timed regions together (the top-level workload alone: %d)" % records[HEADLINE]["gpu_launches"]
    print(json.dumps(line))


def run_plumbing(args, ctx):
    """Rendezvous, barrier, the max over ranks and rank 0's line, with no GPU work: what the CPU tests of
    the launcher run (gloo).  It measures nothing and says so."""
    ms = max_over_ranks(1.0 + ctx.rank, ctx.world)
    ctx.barrier()
    if ctx.rank == 0:
        print(json.dumps({"metric": METRIC, "value": None, "unit": None, "n_gpus": ctx.world, "steps": 0, "warmup": 0,
                          "plumbing_only": True, "max_over_ranks_check": ms}))


REDUCE_CONFIGS = {   # stand-alone row reduction of a bf16 matrix, the paper's GPU case-study category (Section 4.4.1)
    "r_max": dict(M=8192, N=8192, kind=4, name="max"),
    "r_lse": dict(M=8192, N=8192, kind=0, name="lse"),
    "r_softmax": dict(M=8192, N=8192, kind=1, name="softmax"),
    "r_meanvar": dict(M=8192, N=8192, kind=6, name="meanvar"),
    # few, long rows (the shape of a reduction over a flattened dimension): clusters of 8 CTAs share a row
    "r_lse_long": dict(M=16, N=4194304, kind=0, name="lse"),
    "r_max_long": dict(M=16, N=4194304, kind=4, name="max"),
}


def run_reduce(args, ctx):
    """Bench leg of fgr_reduce_rows: same JSON contract; one step = one launch over one matrix."""
    import numpy as np
    import torch
    import torch.distributed as dist
    import fgr_inputs as gi
    import paper_2511_06345_b200 as fgr
    rank, local_rank, world, dev = ctx.rank, ctx.local_rank, ctx.world, ctx.dev
    c = REDUCE_CONFIGS[args.config]
    M, N, kind = c["M"], c["N"], c["kind"]
    peaks, peak_src = ctx.peaks, ctx.peak_src
    rot = 3                                                    # 3 x 134 MB > 126 MB L2
    hosts = [gi.f32_to_bf16_bits(gi.normal(1000 * rank + r, 9, M * N, 2.0)).reshape(M, N) for r in range(rot)]
    mats = [torch.from_numpy(h).view(torch.int16).view(torch.bfloat16).to(dev) for h in hosts]
    P = torch.empty((M, N), dtype=torch.bfloat16, device=dev) if kind == 1 else None
    out = None if kind == 1 else torch.empty((M, 2), dtype=torch.float32, device=dev)
    stream = torch.cuda.current_stream(dev).cuda_stream
    step = lambda i: fgr.fgr_reduce_rows(M, N, fgr.FGR_BF16, kind, mats[i % rot], P, out, device=local_rank, stream=stream)
    sampler = ClockSampler(local_rank)
    sampler.start()
    for i in range(max(args.warmup, 3)):
        step(i)
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize(dev)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0 = time.perf_counter()
    e0.record()
    for i in range(args.steps):
        step(i)
    e1.record()
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize(dev)
    t1 = time.perf_counter()
    sampler.stop()
    ms_step = max_over_ranks(e0.elapsed_time(e1), world, dev) / args.steps
    nbytes = M * N * 2 * (2 if kind == 1 else 1) + (0 if kind == 1 else M * 4)
    value = world * nbytes / (ms_step * 1e-3) / 1e9
    # end to end: pinned host matrix in, result out, around the same C-ABI call
    hp = torch.from_numpy(hosts[0]).pin_memory()
    res_h = torch.empty((M, N), dtype=torch.int16).pin_memory() if kind == 1 else torch.empty((M, 2), dtype=torch.float32).pin_memory()
    stage = mats[0]
    e2e_steps = max(3, min(args.steps, 20))
    def e2e_step():
        stage.view(torch.int16).copy_(hp.view(torch.int16), non_blocking=True)
        fgr.fgr_reduce_rows(M, N, fgr.FGR_BF16, kind, stage, P, out, device=local_rank, stream=stream)
        (res_h.copy_(P.view(torch.int16), non_blocking=True) if kind == 1 else res_h.copy_(out, non_blocking=True))
        torch.cuda.synchronize(dev)
    e2e_step()
    te = time.perf_counter()
    for _ in range(e2e_steps):
        e2e_step()
    dt = max_over_ranks((time.perf_counter() - te) / e2e_steps, world, dev)
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle
        rows = 512
        tc = time.perf_counter()
        oracle.reduce_rows(hosts[0][:rows], dtype=oracle.BF16, kind=kind)
        dtc = time.perf_counter() - tc
        cpu = {"value": nbytes * rows / M / dtc / 1e9, "unit": "GB/s", "cores": 1, "kind": "oracle", "seconds": dtc,
               "sample": "the first %d of %d rows, fp64 loops, one thread" % (rows, M)}
    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
                "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
                "data": "synthetic", "config": {"workload": args.config, "M": M, "N": N, "reduce": c["name"],
                "l2": "rotating %d distinct matrices (%.0f MB > 126 MB L2)" % (rot, rot * M * N * 2 / 1e6)},
                "clocks": sampler.summary(t0, t1), "gpu_launches": args.steps,
                "roofline": {"bound": "hbm", "achieved": value / world, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                             "frac": value / world / peaks["hbm_gbs"], "peak_source": peak_src, "kernel": "reduce_rows_kernel",
                             "kernel_us": ms_step * 1e3, "timing": "the step is this one kernel",
                             "traffic": TRAFFIC.get(args.config)},
                "e2e": {"value": world * nbytes / dt / 1e9, "unit": "GB/s", "h2d_bytes_per_step": M * N * 2,
                        "d2h_bytes_per_step": res_h.numel() * res_h.element_size(), "steps": e2e_steps, "ms_per_step": dt * 1e3}}
        if cpu:
            line["cpu_baseline"] = cpu
        print(json.dumps(line))


NSHARD_CONFIGS = {"c4n": "c4"}   # the skinny workload with W's rows (N) sharded over the ranks: strong scaling


def run_nshard(args, ctx):
    """Bench leg of the N-sharded operator: every rank streams its slice of W, one all-gather of the
    per-row statistics (rows x 8 bytes per rank, NCCL), then fgr_combine_shards.  The problem is fixed
    as ranks are added (strong scaling); value = the whole problem's algorithmic bytes / step time."""
    import numpy as np
    import torch
    import torch.distributed as dist
    import fgr_inputs as gi
    import paper_2511_06345_b200 as fgr
    rank, local_rank, world, dev = ctx.rank, ctx.local_rank, ctx.world, ctx.dev
    base = NSHARD_CONFIGS[args.config]
    peaks, peak_src = ctx.peaks, ctx.peak_src
    shape = make_cfg(base, materialize=False)
    op = fgr.NShardedFusedGemmReduce(shape.batch, shape.M, shape.N, shape.K, shape.dtype, shape.act, shape.scale_kind,
                                     shape.reduce, scale=shape.scale, device=local_rank)
    n0, n1 = op.n0, op.n1
    slice_bytes = (n1 - n0) * shape.K * 2 + shape.M * shape.K * 2
    rot = min(8, max(2, int(math.ceil(2.4 * L2_BYTES / slice_bytes)) + 1))
    up16 = lambda a: torch.from_numpy(np.ascontiguousarray(a)).view(torch.int16).view(torch.bfloat16).to(dev)
    sets, host0 = [], None
    for seed in range(rot):                       # all ranks draw the same problems and keep their slice
        p = make_cfg(base, seed=seed)
        sets.append((up16(p.X), up16(p.W[:, n0:n1, :]), torch.from_numpy(p.bias[n0:n1].copy()).to(dev)))
        host0 = host0 or p
    p = host0
    step = lambda i: op(*sets[i % rot])

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(dev)
    sampler = ClockSampler(local_rank)
    sampler.start()
    for i in range(max(args.warmup, 3)):
        step(i)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0 = time.perf_counter()
    e0.record()
    for i in range(args.steps):
        _, out = step(i)
    e1.record()
    barrier()
    t1 = time.perf_counter()
    if op.status() != fgr.FGR_OK:
        raise SystemExit("device status after the timed region: " + fgr.fgr_status_string(op.status()))
    ms_step = max_over_ranks(e0.elapsed_time(e1), world, dev) / args.steps
    h = op.local.handle
    fgr.fgr_profile_enable(h, True)
    for i in range(args.steps):
        step(i)
    barrier()
    sampler.stop()
    kern_ms, kern_runs = fgr.fgr_profile_read(h)
    kern_s = kern_ms / max(kern_runs, 1) * 1e-3
    value = p.min_bytes() / (ms_step * 1e-3) / 1e9
    local_bytes = slice_bytes + (n1 - n0) * 4 + p.M * 8
    roof = {"bound": "hbm", "achieved": local_bytes / kern_s / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s",
            "peak_source": peak_src, "kernel": "umma_kernel", "kernel_us": kern_s * 1e6, "traffic": None,
            "timing": "CUDA events around each of %d launches of the rank-local main kernel (its slice: %d columns)" % (kern_runs, n1 - n0)}
    roof["frac"] = roof["achieved"] / roof["peak"]
    # end to end: this rank's host slice in, the result out
    hp = [t.cpu().pin_memory() for t in sets[0]]
    res = torch.empty(out.shape, dtype=out.dtype).pin_memory()
    e2e_steps = max(3, min(args.steps, 20))

    def e2e_step():
        for d, s_ in zip(sets[0], hp):
            d.copy_(s_, non_blocking=True)
        res.copy_(op(*sets[0])[1], non_blocking=True)
        torch.cuda.synchronize(dev)
    e2e_step()
    barrier()
    te = time.perf_counter()
    for _ in range(e2e_steps):
        e2e_step()
    dt = max_over_ranks((time.perf_counter() - te) / e2e_steps, world, dev)
    if rank == 0:
        plan = op.local.plan
        print(json.dumps({
            "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
            "ms_per_step": ms_step, "higher_is_better": True, "scaling": "strong", "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic",
            "config": {"workload": args.config, "batch": p.batch, "M": p.M, "N": p.N, "K": p.K, "act": "gelu_tanh",
                       "reduce": "lse", "path": fgr.fgr_path_name(plan.path), "tile": [plan.tile_m, plan.tile_n],
                       "columns_per_rank": n1 - n0,
                       "l2": "rotating %d distinct input sets per rank (%.0f MB > 126 MB L2)" % (rot, rot * slice_bytes / 1e6),
                       "parallelism": "N sharded over %d rank(s); all-gather of [rows, 2] fp32 + combine kernel" % world},
            "clocks": sampler.summary(t0, t1), "gpu_launches": args.steps * (plan.launches + 1), "roofline": roof,
            "e2e": {"value": p.min_bytes() / dt / 1e9, "unit": "GB/s", "h2d_bytes_per_step": sum(t.numel() * t.element_size() for t in hp),
                    "d2h_bytes_per_step": res.numel() * 4, "steps": e2e_steps, "ms_per_step": dt * 1e3}}))
    op.close()


# DRAM bytes per launch of the main kernel from ncu (dram__bytes_read.sum + dram__bytes_write.sum), one
# capture per workload of the kernel as it stands; a workload without a capture of the current kernel
# reports null.
TRAFFIC = {"c2": 90.43e6, "c3": 183.49e6, "c4": 274.99e6, "c5": 70.69e6, "g2": 271.83e6,
           "r_max": 138.23e6, "r_lse": 139.97e6, "r_softmax": 224.41e6, "r_meanvar": 138.14e6,
           "r_max_long": 138.70e6, "r_lse_long": 140.99e6, "f2": 769.50e6, "v2": 124.35e6}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="all", choices=["all"] + NAMED + sorted(EXTRA_CONFIGS) + sorted(REDUCE_CONFIGS) + sorted(NSHARD_CONFIGS))
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--backend", default="nccl", choices=["nccl", "gloo"], help="process-group backend of a multi-rank run")
    ap.add_argument("--plumbing-only", action="store_true",
                    help="start the ranks, meet, print rank 0's line and stop: no GPU work, no measurement")
    args = ap.parse_args()
    if args.impl == "reference":
        # the CPU oracle, on rank 0 alone; the other ranks of a multi-rank launch exit at once
        if args.config in NSHARD_CONFIGS:
            args.config = NSHARD_CONFIGS[args.config]     # the oracle has no shards: the same workload, whole
        if args.config in REDUCE_CONFIGS:
            raise SystemExit("the reference arm covers the fused operator's workloads c1..c5")
        run_reference(args)
        return
    if "WORLD_SIZE" not in os.environ and args.gpus > 1:
        sys.exit(launch_ranks(args.gpus))
    ctx = Ctx(backend=args.backend, use_gpu=not args.plumbing_only)
    try:
        if args.plumbing_only:
            run_plumbing(args, ctx)
        elif args.config == "all":
            run_all(args, ctx)
        elif args.config in NSHARD_CONFIGS:
            run_nshard(args, ctx)
        elif args.config in REDUCE_CONFIGS:
            run_reduce(args, ctx)
        else:
            run_ours(args, ctx)
    finally:
        ctx.close()


if __name__ == "__main__":
    main()
