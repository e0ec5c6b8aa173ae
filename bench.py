#!/usr/bin/env python
"""Benchmark of the Moonwalk gradient step on B200.

One "step" = one pass of the whole hot path over one batch: per-step preparation (W^-1 of every
layer), Phase I + Phase II (mw_input_cotangent) and the forward sweep (mw_forward_sweep).
Default workload: config 5 of the baseline at depth 32 (dense leaky-ReLU MLP, width 4096, batch
1024, bf16 storage / fp32 accumulate, MSE), the largest single-GPU configuration; synthetic seeded
data.  Prints ONE JSON line (rank 0).  On one GPU the default run adds, in the same line, short
measurements of the other configurations (`per_config`) and the peak-memory / throughput study
over depth (`depth_sweep`); --quick leaves them out.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--workload NAME]

Workloads: sweep_mlp --depth D (default, config 5), deep_mlp (config 2), lu_mlp (config 2's sizes, LU-parameterised layers), deep_mlp_small, mixed_mlp
(config 4), submersive_cnn (config 3), tiny_mlp (config 1); the paper's own convolutional experiments
strided_cnn [--depth D] (stride-2 submersive layers) and fragmental_cnn1d [--depth D --frag-block B]
(1-D, fragmental checkpoints), their bf16 forms strided_cnn_bf16 / fragmental_cnn1d_bf16, and
strided_cnn_small.  --with-backprop adds the time of the library's own Backprop; --depth-sweep and
--memory-table print the memory studies instead of the benchmark line.

The roofline object prices the product kernel inside the forward sweep at the flops of the
products the method defines (recompute, vijp, weight vjp); `whole_step` prices a step at
10 B n^2 + 2 n^3 per layer.  The iterations of the per-step inverse never count as algorithmic work.

N > 1 (under torchrun): independent replicas of the same step on every GPU, no data-path
collective ("replicas only"); NCCL is used only for the barrier and the max over ranks.
--impl reference times the CPU oracle (fp64, numpy) on the host cores instead, on the same bounded
sample of the workload that the GPU arm's cpu_baseline uses.
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
sys.path.insert(0, ROOT)

DEFAULT_WORKLOAD = "sweep_mlp"     # config 5 at depth 32: the largest single-GPU configuration
METRIC = "moonwalk_grad_samples_per_s"
UNIT = "samples/s"
NOMINAL_TF32_OVER_BF16 = 1.1 / 2.25      # dense tensor peaks, nominal ratio
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def workload(name: str, seed: int = 0, depth: int = 0, block: int = 0):
    from paper_2402_14212_b200 import synth as S
    if name == "deep_mlp":
        return S.deep_mlp(seed=seed)
    if name == "deep_mlp_small":
        return S.deep_mlp(seed=seed, depth=8, n=256, batch=128)
    if name == "mixed_mlp":
        return S.mixed_mlp(seed=seed)
    if name == "lu_mlp":
        # config 2's sizes with every layer parameterised by the triangular factors of its weight
        return S.lu_mlp(seed=seed, depth=depth or 64)
    if name == "sweep_mlp":
        return S.sweep_mlp(seed=seed, depth=depth or 32, pool=4)
    if name == "submersive_cnn":
        return S.submersive_cnn(seed=seed)
    if name == "strided_cnn":
        # the paper's own convolutional experiment: 256 x 256 x 128 inputs, batch 128, 3x3 stride-2
        # submersive layers (`depth` of them, 8 by default: down to 1 x 1)
        return S.strided_cnn(seed=seed, depth=depth or 8)
    if name == "strided_cnn_bf16":
        return S.strided_cnn(seed=seed, depth=depth or 8, prec=S.BF16)
    if name == "strided_cnn_small":
        return S.strided_cnn(seed=seed, depth=depth or 4, H=64, W=64, batch=16)
    if name == "fragmental_cnn1d":
        # the paper's 1-D experiment: 2048 x 256 sequences, batch 128, k = 3 stride-1 convolutions,
        # output cotangents checkpointed at 2 of every `block` positions
        return S.fragmental_cnn1d(seed=seed, depth=depth or 16, block=block or 4)
    if name == "fragmental_cnn1d_bf16":
        return S.fragmental_cnn1d(seed=seed, depth=depth or 16, block=block or 4, prec=S.BF16)
    if name == "tiny_mlp":
        return S.tiny_mlp(seed=seed)
    raise SystemExit(f"unknown workload {name}")


def describe(p):
    if p.layers[0].kind == "conv1d":
        l0 = p.layers[0]
        return {"workload": p.name, "layers": len(p.layers), "conv": f"{l0.k}x{l0.C_in}x{l0.C_out}",
                "sequence": f"{l0.W}x{l0.C_in}", "stride": 1, "batch": p.batch, "prec": p.prec,
                "loss": p.loss, "reseed_every": p.reseed_every, "frag_block": p.frag_block, "seed": p.seed}
    if p.layers[0].kind == "conv2d":
        l0 = p.layers[0]
        return {"workload": p.name, "layers": len(p.layers), "conv": f"{l0.k}x{l0.k}x{l0.C_in}x{l0.C_out}",
                "image": f"{l0.H}x{l0.W}", "stride": l0.stride, "batch": p.batch, "prec": p.prec, "loss": p.loss,
                "reseed_every": p.reseed_every, "conv_vijp_iters": p.conv_vijp_iters, "seed": p.seed}
    return {"workload": p.name, "layers": len(p.layers), "width": p.layers[0].n_in,
            "batch": p.batch, "prec": p.prec, "loss": p.loss, "reseed_every": p.reseed_every,
            "seed": p.seed}


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        d["_source"] = "measured"
        return d
    d = dict(FALLBACK_PEAKS)
    d["_source"] = "fallback"
    return d


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                mx = float(f[1])
            except ValueError:
                continue
            for nme, val in zip(names, f[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(nme)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": mx,
                "reasons": sorted(reasons), "samples": len(sm)}


# The oracle is a plain fp64 numpy program: a step of the large dense workloads would take minutes
# (an LU solve of every n x n weight per layer).  Both arms therefore time it on the SAME bounded
# sample of the workload -- the first `batch` samples through the first `layers` layers -- and
# scale the result to the full depth (cost is linear in depth); (0, 0) = the whole workload.
ORACLE_SAMPLE = {
    "sweep_mlp": (32, 1), "mixed_mlp": (32, 4), "deep_mlp": (32, 0), "lu_mlp": (32, 0), "submersive_cnn": (2, 8),
    "strided_cnn": (1, 0), "strided_cnn_bf16": (1, 0), "fragmental_cnn1d": (1, 0),
    "fragmental_cnn1d_bf16": (1, 0),
}


def oracle_sample(p):
    """(layers, params, x, target, samples, layers used, description) of the bounded oracle sample."""
    import numpy as np
    b, ls = ORACLE_SAMPLE.get(p.name, (0, 0))
    b = min(b or p.batch, p.batch)
    L = len(p.layers)
    ls = min(ls or L, L)
    layers, params = p.layers[:ls], p.params[:ls]
    x = np.asarray(p.x[:b], dtype=np.float64)
    if ls == L:
        t = p.target[:b]
    else:   # a target of the shape of the last kept layer's output (timing only)
        rng = np.random.default_rng(p.seed + 17)
        t = rng.standard_normal((b, layers[-1].n_out))
    what = (f"{b} of {p.batch} samples through {'all' if ls == L else 'the first ' + str(ls) + ' of'} "
            f"{L} layers, fp64 numpy, Algorithm 1")
    if ls != L:
        what += f"; value scaled by {ls}/{L} to the full depth"
    return layers, params, x, t, b, ls, what


def oracle_step_fn(p):
    from oracle import moonwalk_oracle as O
    layers, params, x, t, b, ls, what = oracle_sample(p)
    loss = p.loss if ls == len(p.layers) else "mse_mean"

    def step():
        O.moonwalk(layers, params, x, t, loss, reseed_every=p.reseed_every, frag_block=p.frag_block)

    return step, b, ls, what


def time_oracle(p, seconds_target: float, max_reps: int = 50):
    """Oracle (as it stands) on the host cores, on the bounded sample both arms use."""
    step, b, ls, what = oracle_step_fn(p)
    reps, t0 = 0, time.perf_counter()
    while True:
        step()
        reps += 1
        dt = time.perf_counter() - t0
        if dt >= seconds_target or reps >= max_reps:
            break
    value = b * reps / dt * ls / len(p.layers)
    return value, reps, dt, what


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [d.get("num_threads", 0) for d in threadpool_info() if d.get("user_api") == "blas"]
        return max(n) if n else os.cpu_count()
    except Exception:
        return os.cpu_count()


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    p = workload(args.workload, depth=args.depth, block=args.frag_block)
    step, b, ls, what = oracle_step_fn(p)
    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = time.perf_counter() - t0
    value = b * args.steps / dt * ls / len(p.layers)
    cores = blas_threads()
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT,
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": 1e3 * dt / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": describe(p),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                             "sample": what},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def aggregate_replicas(ms_local: float, batch: int, steps: int, world: int, device=None):
    """Whole-job throughput of `world` independent replicas: all samples over the slowest rank's
    time (max over ranks through torch.distributed when world > 1)."""
    import torch
    ms_max = float(ms_local)
    if world > 1:
        import torch.distributed as dist
        t = torch.tensor([ms_local], dtype=torch.float64, device=device)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms_max = float(t.item())
    return batch * steps * world / (ms_max * 1e-3), ms_max


def kernel_source_hash():
    import hashlib
    path = os.path.join(ROOT, "paper_2402_14212_b200", "csrc", "mw_tc_gemm.cu")
    return hashlib.sha256(open(path, "rb").read()).hexdigest()[:16]


def recorded_traffic(workload_name: str):
    """DRAM bytes per launch of the product kernel inside the forward sweep, from the committed ncu
    summary -- only while the kernel source is still the one that was profiled (else None)."""
    path = os.path.join(ROOT, "profiles", f"tc_group_kernel_sweep_traffic_{workload_name}.md")
    if not os.path.exists(path):
        return None
    vals = {}
    for ln in open(path):
        if ln.startswith("    ") and "=" in ln:
            k, v = ln.strip().split("=", 1)
            vals[k.strip()] = v.strip()
    if vals.get("kernel_source_sha256_16") != kernel_source_hash():
        return None
    try:
        return float(vals["dram_bytes_per_launch"])
    except (KeyError, ValueError):
        return None


def algorithmic_flops(p):
    """Flops the method itself prices (dense nets): per layer the sweep's three products 6 B n^2,
    the whole step 10 B n^2 (Phase I, Phase II, recompute, vijp, weight vjp) plus one inverse 2 n^3."""
    if p.layers[0].kind != "dense":
        return None
    n, B, L = p.layers[0].n_in, p.batch, len(p.layers)
    return {"sweep": 6.0 * B * n * n * L, "whole_step": (10.0 * B * n * n + 2.0 * n ** 3) * L}


class Bench:
    """One workload on the current device: buffers, the step, and its measurements."""

    def __init__(self, p, args, dev, warm_inverse=False):
        import torch
        from paper_2402_14212_b200 import binding as mwb
        self.torch, self.mwb, self.p, self.dev = torch, mwb, p, dev
        self.net = mwb.net_for(p, backend=args.backend, warm_inverse=warm_inverse)
        self.params, self.x, self.target = mwb.to_device(p, dev)
        self.ws = self.net.alloc_workspace("moonwalk", dev)
        # nets of strided submersive convolutions keep the part of g0 that the sweep reads inside
        # the workspace (mw_input_cotangent with g0_out = NULL); the others hand g0 over in full
        self.lean = p.layers[0].kind == "conv2d" and p.layers[0].stride != 1 and not args.full_g0
        self.g0 = None if self.lean else torch.empty(self.x.shape, dtype=self.net.grad_dtype(), device=dev)
        self.dW = [torch.empty(w.shape, dtype=self.net.grad_dtype(), device=dev) for w in self.params]
        self.loss = torch.zeros(1, dtype=torch.float64, device=dev)
        self.stream = torch.cuda.current_stream()
        self.dp = None

    def cotangent(self):
        self.net.input_cotangent(self.params, self.x, self.target, self.ws, g0_out=self.g0,
                                 loss_out=self.loss, keep_seed=self.lean)

    def sweep(self):
        self.net.forward_sweep(self.params, self.x, self.g0, self.ws, dW_out=self.dW)

    def step(self):
        if self.dp is not None:
            self.dp.step(self.params, self.x, self.target, self.ws, self.g0, self.dW, loss_out=self.loss)
            return
        self.cotangent()
        self.sweep()

    def enable_data_parallel(self, world, layers_per_bucket=8):
        """--parallel dp: this rank's net holds one shard of the batch; the step all-reduces the
        gradients bucket by bucket on a side stream while the sweep runs (data_parallel.py)."""
        from paper_2402_14212_b200 import data_parallel
        self.dp = data_parallel.DataParallelStep(self.net, self.p.loss, world, layers_per_bucket, device=self.dev)

    def warm(self, n):
        for _ in range(n):
            self.step()
        code, detail = self.net.last_device_status(self.ws)
        if code != 0:
            raise SystemExit(f"device status {code} {detail} during warm-up of {self.p.name}")

    def timed_block(self, steps):
        torch = self.torch
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(self.stream)
        for _ in range(steps):
            self.step()
        e1.record(self.stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1)

    def phases(self, reps):
        torch = self.torch
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
        t_cot = t_sweep = 0.0
        for _ in range(reps):
            ev[0].record(self.stream)
            self.cotangent()
            ev[1].record(self.stream)
            self.sweep()
            ev[2].record(self.stream)
            torch.cuda.synchronize()
            t_cot += ev[0].elapsed_time(ev[1])
            t_sweep += ev[1].elapsed_time(ev[2])
        return t_cot / reps, t_sweep / reps

    def backprop_ms(self, reps):
        torch = self.torch
        ws_bp = self.net.alloc_workspace("backprop", self.dev)
        for _ in range(2):
            self.net.backprop_reference(self.params, self.x, self.target, ws_bp, dW_out=self.dW)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(self.stream)
        for _ in range(reps):
            self.net.backprop_reference(self.params, self.x, self.target, ws_bp, dW_out=self.dW)
        e1.record(self.stream)
        torch.cuda.synchronize()
        del ws_bp
        return e0.elapsed_time(e1) / reps

    def sweep_kernel_profile(self, reps):
        """Product-kernel launches of the forward sweep alone (Algorithm 1's loop), each bracketed by
        CUDA events on its stream; the input-cotangent call is left outside the events."""
        sw = {"total_ms": 0.0, "launches": 0, "flops": 0.0, "mma_flops": 0.0}
        for _ in range(reps):
            self.cotangent()        # no host synchronisation here: the sweep runs as it does inside a step
            self.mwb.profile_begin()
            self.sweep()
            one = self.mwb.profile_end()
            for k in sw:
                sw[k] += one[k]
        return sw

    def step_kernel_profile(self, steps):
        self.mwb.profile_begin()
        for _ in range(steps):
            self.step()
        return self.mwb.profile_end()


def tensor_peak(p, pk):
    bf16_peak = float(pk.get("bf16_tflops_sustained", pk["bf16_tflops"]))
    src = pk["_source"]
    if p.prec == "f32":
        return bf16_peak * NOMINAL_TF32_OVER_BF16, bf16_peak, f"{src} sustained bf16 x nominal tf32/bf16 ratio (fp32 products), of {src}"
    return bf16_peak, bf16_peak, f"{src} sustained bf16 (kernel timed inside a long step), of {src}"


def roofline_of(b: "Bench", reps: int, step_ms: float):
    """Roofline object of the dominant kernel: the tcgen05 product kernel inside the forward sweep,
    priced at the flops of the products the method defines (2MNK each: recompute, vijp, weight vjp);
    whole_step beside it: 10 B n^2 + 2 n^3 per layer over the kernel time of a whole step (the
    iterations of the per-step inverse are NOT counted as algorithmic work)."""
    p = b.p
    if b.net.prec == "f64":
        return None
    pk = peaks()
    peak, bf16_peak, note = tensor_peak(p, pk)
    sw = b.sweep_kernel_profile(reps)
    if not sw["launches"]:
        return None
    a_sw = sw["flops"] / (sw["total_ms"] * 1e-3) / 1e12
    e_sw = sw["mma_flops"] / (sw["total_ms"] * 1e-3) / 1e12
    roof = {"bound": "tensor", "kernel": "tc_group_kernel inside mw_forward_sweep (tcgen05 products: recompute, vijp, weight vjp)",
            "achieved": a_sw, "peak": peak, "unit": "TFLOP/s", "frac": a_sw / peak,
            "traffic": recorded_traffic(p.name), "peak_source": note,
            "launches_per_sweep": sw["launches"] / reps,
            "avg_launch_us": 1e3 * sw["total_ms"] / sw["launches"],
            "algorithmic_flops_per_launch": sw["flops"] / sw["launches"],
            "executed_bf16_tflops": e_sw, "executed_frac_of_bf16_peak": e_sw / bf16_peak,
            "kernel_source_sha256_16": kernel_source_hash()}
    alg = algorithmic_flops(p)
    st = b.step_kernel_profile(reps)
    if st["launches"]:
        kms = st["total_ms"] / reps
        ws = {"kernel_ms_per_step": kms, "kernel_time_share_of_step": kms / step_ms,
              "launched_2mnk_tflops": st["flops"] / (st["total_ms"] * 1e-3) / 1e12,
              "executed_bf16_tflops": st["mma_flops"] / (st["total_ms"] * 1e-3) / 1e12}
        if alg:
            a = alg["whole_step"] / (kms * 1e-3) / 1e12
            ws.update({"algorithmic_flops": alg["whole_step"], "achieved": a, "frac": a / peak,
                       "priced_as": "per layer 10 B n^2 (Phase I, Phase II, recompute, vijp, weight vjp) + 2 n^3 (one inverse)"})
        roof["whole_step"] = ws
    return roof


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2402_14212_b200 import binding as mwb

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (no CPU fallback)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    if args.no_coop:
        mwb.set_cooperative_launch(False)
    p = workload(args.workload, depth=args.depth, block=args.frag_block)
    global_batch = p.batch
    if args.parallel == "dp":
        # the batch of the workload is the GLOBAL batch: this rank keeps its shard (strong scaling)
        from paper_2402_14212_b200 import data_parallel
        lo, hi = data_parallel.shard_bounds(p.batch, rank, world)
        p.x, p.target, p.batch = p.x[lo:hi], p.target[lo:hi], hi - lo
    b = Bench(p, args, dev)
    if args.parallel == "dp":
        b.enable_data_parallel(world)
    net = b.net
    mw_bytes, bp_bytes, (mw_res, bp_res) = net.workspace_bytes()
    warm = max(args.warmup, 3)
    b.warm(warm)

    # ---- device-resident timing: blocks of K steps, CUDA events on the launching stream ---------
    # The contract's K steps are one block; the block is repeated so that the clock sampler sees
    # the GPU under load for seconds, and the median block is reported.
    sampler = ClockSampler(local)
    barrier()
    sampler.start()
    launches0 = mwb.launch_count()
    blocks = []
    for _ in range(max(1, args.blocks)):
        barrier()
        blocks.append(b.timed_block(args.steps))
    barrier()
    launches = (mwb.launch_count() - launches0) // max(1, args.blocks)
    clocks = sampler.stop()
    ms = statistics.median(blocks)
    value, ms_max = aggregate_replicas(ms, p.batch, args.steps, world, dev)   # shards or replicas: all samples
    step_ms = ms_max / args.steps

    reps = min(args.steps, 5)
    t_cot, t_sweep = b.phases(reps)
    t_bp = b.backprop_ms(reps) if (args.with_backprop or args.workload == DEFAULT_WORKLOAD) else None

    # ---- end to end through the C ABI with host buffers --------------------------------------
    x, target = b.x, b.target
    xh = x.cpu().pin_memory()
    th = target.cpu().pin_memory()
    lh = torch.zeros(1, dtype=torch.float64).pin_memory()
    xd, td = torch.empty_like(x), torch.empty_like(target)
    for _ in range(2):
        net.gradient_step_host(b.params, xh, th, xd, td, b.g0, b.dW, b.loss, lh, b.ws)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    w0 = time.perf_counter()
    e0.record(b.stream)
    for _ in range(args.steps):
        net.gradient_step_host(b.params, xh, th, xd, td, b.g0, b.dW, b.loss, lh, b.ws)
    e1.record(b.stream)
    barrier()
    wall = time.perf_counter() - w0
    ms_e2e = max(e0.elapsed_time(e1), 0.0)
    e2e_value, _ = aggregate_replicas(max(ms_e2e, wall * 1e3), p.batch, args.steps, world, dev)
    h2d = xh.numel() * xh.element_size() + th.numel() * th.element_size()

    roof = roofline_of(b, reps, step_ms) if net.prec != "f64" else None

    # ---- the other configurations and the depth study (single GPU, rank 0; the default run only) --
    per_config = depth_rows = steady = None
    full = rank == 0 and world == 1 and args.workload == DEFAULT_WORKLOAD and not args.quick
    if full:
        del xh, th, xd, td
        main_ws = b.ws
        b.ws = None
        del main_ws
        torch.cuda.empty_cache()
        # the same step inside a training loop: the workspace keeps every W^-1 and each step
        # refreshes it with one Newton-Schulz step (mw_net_opts.warm_inverse).  The weights do not
        # move here; a step that moves them by a training-sized amount costs the same.
        if p.layers[0].kind == "dense":
            bw = Bench(p, args, dev, warm_inverse=True)
            bw.warm(3)
            ms_w = statistics.median([bw.timed_block(args.steps) for _ in range(3)]) / args.steps
            tc_w, ts_w = bw.phases(reps)
            steady = {"ms_per_step": ms_w, "samples_per_s": p.batch / (ms_w * 1e-3),
                      "phases_ms": {"prep_phase1_phase2": tc_w, "forward_sweep": ts_w},
                      "what": "warm_inverse = 1: kept inverses refreshed by the last Newton-Schulz step, residual-gated per layer"}
            del bw
            torch.cuda.empty_cache()
        per_config = {}
        for name in PER_CONFIG:
            try:
                per_config[name] = measure_config(name, args, dev)
            except SystemExit as e:
                per_config[name] = {"error": str(e)}
            torch.cuda.empty_cache()
        depth_rows = depth_sweep_rows(args, dev, max_depth=args.max_depth)

    # ---- the oracle on the host cores (rank 0, single GPU only) -----------------------------
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        v, reps_o, dt, what = time_oracle(p, 12.0)
        cpu = {"value": v, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
               "sample": f"{reps_o} steps in {dt:.1f} s of: {what}"}

    if rank == 0:
        sm = clocks.get("sm_mhz")
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": warm, "ms_per_step": step_ms,
                "higher_is_better": True, "scaling": "strong" if args.parallel == "dp" else "weak",
                "vs_baseline": None,
                "dtype": {"f64": "f64", "f32": "f32 (bf16x3 split on tensor cores, fp32 accumulate)",
                          "bf16_f32acc": "bf16 (fp32 accumulate)"}[p.prec]
                if net_backend_is_tensor(net) else ("f64" if p.prec == "f64" else "f32"),
                "data": "synthetic", "config": describe(p),
                "parallelism": (f"data parallel x{world}: global batch {global_batch} in equal shards, bucketed all-reduce of dW"
                                if args.parallel == "dp" else (f"replicas x{world}" if world > 1 else "single GPU")),
                "l2_policy": "working set (weights, inverses, gradients: GBs) far above the 126 MB L2; no flush between steps",
                "timed_blocks": {"count": len(blocks), "steps_each": args.steps, "ms": blocks, "reported": "median"},
                "clocks": clocks, "ms_per_step_x_sm_mhz": (step_ms * sm) if sm else None,
                "gpu_launches": launches,
                "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": 8,
                        "returns": "the loss (8 bytes) per step; the gradients stay on the device for the update"},
                "roofline": roof, "cpu_baseline": cpu,
                "phases_ms": {"prep_phase1_phase2": t_cot, "forward_sweep": t_sweep, "backprop": t_bp},
                "memory_bytes": {"moonwalk_workspace": mw_bytes, "backprop_workspace": bp_bytes,
                                 "moonwalk_residual": mw_res, "backprop_residual": bp_res,
                                 "params": sum(w.numel() * w.element_size() for w in b.params),
                                 "grads": sum(g.numel() * g.element_size() for g in b.dW)},
                "steady_state_training_step": steady,
                "per_config": per_config, "depth_sweep": depth_rows}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


# the other baseline configurations and the paper's two experiments, reported beside the main line
PER_CONFIG = ["deep_mlp", "lu_mlp", "submersive_cnn", "mixed_mlp", "strided_cnn", "fragmental_cnn1d"]


def measure_config(name, args, dev):
    """Short measurement of one more workload: step time, phases, sweep-only roofline."""
    import torch
    p = workload(name, depth=0, block=0)
    b = Bench(p, args, dev)
    b.warm(3)
    steps = 5
    ms = b.timed_block(steps) / steps
    t_cot, t_sweep = b.phases(3)
    out = {"config": describe(p), "ms_per_step": ms, "samples_per_s": p.batch / (ms * 1e-3),
           "phases_ms": {"prep_phase1_phase2": t_cot, "forward_sweep": t_sweep},
           "parity": "full-size parity against the oracle: tests/ (-m gpu)"}
    if b.net.prec != "f64":
        pk = peaks()
        peak, bf16_peak, note = tensor_peak(p, pk)
        sw = b.sweep_kernel_profile(2)
        if sw["launches"]:
            a = sw["flops"] / (sw["total_ms"] * 1e-3) / 1e12
            e = sw["mma_flops"] / (sw["total_ms"] * 1e-3) / 1e12
            out["forward_sweep_roofline"] = {"achieved": a, "peak": peak, "frac": a / peak, "unit": "TFLOP/s",
                                             "executed_bf16_tflops": e, "executed_frac_of_bf16_peak": e / bf16_peak,
                                             "peak_source": note, "launches_per_sweep": sw["launches"] / 2,
                                             "avg_launch_us": 1e3 * sw["total_ms"] / sw["launches"]}
    mw_b, bp_b, (mw_res, bp_res) = b.net.workspace_bytes()
    out["memory_bytes"] = {"moonwalk_workspace": mw_b, "backprop_workspace": bp_b,
                           "moonwalk_residual": mw_res, "backprop_residual": bp_res}
    del b
    torch.cuda.empty_cache()
    return out


def depth_sweep_rows(args, dev, max_depth: int):
    """Config 5: dense leaky-ReLU MLP, width 4096, batch 1024, bf16 / fp32 accumulate, depth
    doubling from 32.  Per depth: workspace and residual bytes of both methods (from the library's
    own accounting), peak device bytes seen by the allocator, samples/s; and the largest depth whose
    total (parameters + gradients + workspace) fits 64 GB, from the same accounting.  Moonwalk runs
    in its lean-memory mode (one transient inverse slot: resident_inverse = 0) and, where the
    workspace fits the device, also with every layer's inverse resident (the benchmark's mode)."""
    import torch
    from paper_2402_14212_b200 import binding as mwb
    from paper_2402_14212_b200 import synth as S
    n, batch, budget = 4096, 1024, 64e9
    base = S.sweep_mlp(seed=0, depth=4, pool=4)
    pool_dev = [torch.from_numpy(w).to(torch.bfloat16).to(dev) for w in base.params[:4]]
    x = torch.from_numpy(base.x).to(torch.bfloat16).to(dev)
    target = torch.from_numpy(base.target).to(torch.float32).to(dev)
    free_bytes = torch.cuda.mem_get_info(dev)[0]

    def accounting(depth, resident):
        layers = [base.layers[0]] * depth
        net = mwb.Net(layers, batch, base.prec, base.loss, reseed_every=base.reseed_every,
                      backend="tensor", resident_inverse=resident)
        mw_b, bp_b, (mw_res, bp_res) = net.workspace_bytes()
        return net, mw_b, bp_b, mw_res, bp_res

    pbytes, gbytes = n * n * 2, n * n * 4
    rows = []
    depth = 32
    while depth <= max_depth:
        net, mw_b, bp_b, mw_res, bp_res = accounting(depth, False)
        net_r, mw_r, _, mw_res_r, _ = accounting(depth, True)
        row = {"depth": depth, "params_bytes": depth * pbytes,
               "moonwalk": {"workspace_bytes": mw_b, "residual_bytes": mw_res},
               "moonwalk_resident_inverses": {"workspace_bytes": mw_r, "residual_bytes": mw_res_r},
               "backprop": {"workspace_bytes": bp_b, "residual_bytes": bp_res}}
        # gradients streamed: layer l's dW lands in one of two rotating buffers (applied and
        # dropped, Algorithm 1's last line), so the totals below exclude a full set of gradients
        params = [pool_dev[l % 4].clone() for l in range(depth)]
        dW2 = [torch.empty((n, n), dtype=torch.float32, device=dev) for _ in range(2)]
        dW = [dW2[l & 1] for l in range(depth)]
        g0 = torch.empty((batch, n), dtype=torch.float32, device=dev)
        for which, the_net, need in (("moonwalk", net, mw_b), ("moonwalk_resident_inverses", net_r, mw_r),
                                     ("backprop", net, bp_b)):
            if need + depth * pbytes > 0.85 * free_bytes:
                row[which]["skipped"] = "workspace does not fit this device"
                continue
            torch.cuda.synchronize()
            torch.cuda.reset_peak_memory_stats(dev)
            before = torch.cuda.memory_allocated(dev)
            ws = the_net.alloc_workspace("backprop" if which == "backprop" else "moonwalk", dev)
            ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]

            def step():
                if which == "backprop":
                    the_net.backprop_reference(params, x, target, ws, dW_out=dW)
                else:
                    the_net.input_cotangent(params, x, target, ws, g0_out=g0)
                    the_net.forward_sweep(params, x, g0, ws, dW_out=dW)

            step()
            code, detail = the_net.last_device_status(ws)
            if code != 0:
                raise SystemExit(f"device status {code} {detail} at depth {depth} ({which})")
            reps = 2
            ev[0].record()
            for _ in range(reps):
                step()
            ev[1].record()
            torch.cuda.synchronize()
            ms = ev[0].elapsed_time(ev[1]) / reps
            row[which].update({"ms_per_step": ms, "samples_per_s": batch / (ms * 1e-3),
                               "peak_device_bytes": torch.cuda.max_memory_allocated(dev),
                               "extra_over_params_and_inputs": torch.cuda.max_memory_allocated(dev) - before})
            del ws
            torch.cuda.empty_cache()
        rows.append(row)
        del params, dW, dW2, net, net_r
        torch.cuda.empty_cache()
        depth *= 2

    def max_depth_under(which, keep_grads):
        lo, hi = 1, 1 << 14
        while lo < hi:
            mid = (lo + hi + 1) // 2
            _, mw_b, bp_b, _, _ = accounting(mid, False)
            ws = mw_b if which == "moonwalk" else bp_b
            total = mid * pbytes + ws + (mid * gbytes if keep_grads else 2 * gbytes)
            if total <= budget:
                lo = mid
            else:
                hi = mid - 1
        return lo

    return {"workload": "depth sweep: dense leaky-ReLU MLP, width 4096, batch 1024, bf16 storage / fp32 accumulate",
            "per_layer_bytes": {"params_bf16": pbytes, "grad_fp32": gbytes,
                                "backprop_stored_activation_bf16": batch * n * 2,
                                "moonwalk_sign_bits": batch * n // 8,
                                "moonwalk_cotangent_checkpoint_fp32_every_K": batch * n * 4,
                                "K": base.reseed_every},
            "rows": rows,
            "max_depth_under_64GB": {
                "moonwalk_grads_streamed": max_depth_under("moonwalk", False),
                "backprop_grads_streamed": max_depth_under("backprop", False),
                "moonwalk_grads_kept": max_depth_under("moonwalk", True),
                "backprop_grads_kept": max_depth_under("backprop", True)}}


def run_depth_sweep(args):
    import torch
    torch.cuda.set_device(0)
    print(json.dumps(depth_sweep_rows(args, torch.device("cuda", 0), args.max_depth)), flush=True)


def net_backend_is_tensor(net):
    return net.prec != "f64" and all(l.kind == "dense" and l.n_in % 64 == 0 for l in net.layers)


def memory_table(budget_bytes: float = 24e9):
    """The paper's memory experiments from the library's own accounting (mw_workspace_bytes; no GPU
    work): workspace and between-phase residual bytes of Moonwalk and of the in-library Backprop for
    the 2-D submersive CNN over its depth and for the 1-D CNN with fragmental checkpoints over depth
    and block size, and the largest 1-D depth whose total (workspace + parameters + gradients + input
    and target) stays under `budget_bytes` (the paper's GPU has 24 GB)."""
    from paper_2402_14212_b200 import binding as mwb
    from paper_2402_14212_b200 import synth as S

    def strided_layers(depth, C=128, H=256):
        out, h = [], H
        for _ in range(depth):
            lay = S.Layer(S.CONV2D, S.ACT_LEAKY, 0.1, h * h * C, 0, H=h, W=h, C_in=C, C_out=C, k=3, stride=2, pad=1)
            ho, wo = lay.out_hw()
            lay.n_out = ho * wo * C
            out.append(lay)
            h = ho
        return out

    def conv1d_layers(depth, C=256, N=2048):
        return [S.Layer(S.CONV1D, S.ACT_LEAKY, 0.1, N * C, N * C, H=1, W=N, C_in=C, C_out=C, k=3, stride=1, pad=1)
                for _ in range(depth)]

    def row(layers, batch, **kw):
        net = mwb.Net(layers, batch, S.F32, S.LOSS_MSE_MEAN, backend="tensor", reseed_every=4, **kw)
        mw_b, bp_b, (mw_res, bp_res) = net.workspace_bytes()
        w = sum(4 * l.k * l.k * l.C_in * l.C_out if l.kind == S.CONV2D else 4 * l.k * l.C_in * l.C_out
                for l in layers)
        io = 4 * batch * (layers[0].n_in + layers[-1].n_out)
        net.close()
        return {"depth": len(layers), "moonwalk_workspace": mw_b, "backprop_workspace": bp_b,
                "moonwalk_residual": mw_res, "backprop_residual": bp_res, "params": w, "grads": w,
                "inputs": io, "moonwalk_total": mw_b + 2 * w + io, "backprop_total": bp_b + 2 * w + io}

    table = {"budget_bytes": budget_bytes, "strided_cnn": [row(strided_layers(d), 128) for d in range(1, 9)],
             "fragmental_cnn1d": {}}
    for blk in (4, 16):
        rows = [row(conv1d_layers(d), 128, frag_block=blk) for d in (2, 4, 8, 16, 22, 32)]
        # totals grow linearly in depth: walk up to the budget
        fit = {}
        for which in ("moonwalk_total", "backprop_total"):
            d = 1
            while d < 4096 and row(conv1d_layers(d + 1), 128, frag_block=blk)[which] <= budget_bytes:
                d += 1 if d < 64 else 16
            fit[which.replace("_total", "_max_depth")] = d
        table["fragmental_cnn1d"][f"block_{blk}"] = {"rows": rows, **fit}
    return table


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD)
    ap.add_argument("--blocks", type=int, default=5,
                    help="repetitions of the timed block of --steps steps (the median block is reported)")
    ap.add_argument("--parallel", default="replicas", choices=["replicas", "dp"],
                    help="N > 1: independent replicas (default), or dp = the batch sharded over the ranks with a "
                         "bucketed all-reduce of the gradients overlapped with the sweep (not measured on hardware here)")
    ap.add_argument("--no-coop", action="store_true",
                    help="program launches without the cooperative attribute (for launch lists under a profiler)")
    ap.add_argument("--quick", action="store_true",
                    help="the main line only: no per_config / depth_sweep sections")
    ap.add_argument("--backend", default="auto", choices=["auto", "simt", "tensor"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--full-g0", action="store_true",
                    help="strided CNN workloads: have mw_input_cotangent return g0 in full")
    ap.add_argument("--with-backprop", action="store_true",
                    help="also time mw_backprop_reference on the same inputs (phases_ms.backprop)")
    ap.add_argument("--depth", type=int, default=0, help="depth of the sweep_mlp / CNN workloads")
    ap.add_argument("--frag-block", type=int, default=0, help="block size of the fragmental_cnn1d workload")
    ap.add_argument("--depth-sweep", action="store_true",
                    help="config 5: peak memory and samples/s versus depth, Moonwalk against the "
                         "in-library Backprop (prints one JSON object, not the benchmark line)")
    ap.add_argument("--max-depth", type=int, default=0,
                    help="largest depth of the depth study (default: 256 inside the benchmark line, 512 for --depth-sweep)")
    ap.add_argument("--memory-table", action="store_true",
                    help="the paper's CNN memory experiments from the library's byte accounting "
                         "(prints one JSON object; runs without a GPU)")
    args = ap.parse_args()
    if not args.max_depth:
        args.max_depth = 512 if args.depth_sweep else 256
    if args.memory_table:
        print(json.dumps(memory_table()), flush=True)
    elif args.depth_sweep:
        run_depth_sweep(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
