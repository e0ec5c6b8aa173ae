#!/usr/bin/env python
"""Benchmark of the Moonwalk gradient step on B200.

One "step" = one pass of the whole hot path over one batch: per-step preparation (W^-1 of every
layer), Phase I + Phase II (mw_input_cotangent) and the forward sweep (mw_forward_sweep).
Workload: config 2 of the baseline (64 square dense layers, width 1024, leaky-ReLU 0.1, batch 256,
fp32, MSE), synthetic seeded data.  Prints ONE JSON line (rank 0).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--workload NAME]

Workloads: deep_mlp (default, config 2), deep_mlp_small, mixed_mlp (config 4), sweep_mlp --depth D
(config 5), submersive_cnn (config 3), tiny_mlp (config 1); the paper's own convolutional experiments
strided_cnn [--depth D] (stride-2 submersive layers) and fragmental_cnn1d [--depth D --frag-block B]
(1-D, fragmental checkpoints), their bf16 forms strided_cnn_bf16 / fragmental_cnn1d_bf16, and
strided_cnn_small.  --with-backprop adds the time of the library's own Backprop; --depth-sweep and
--memory-table print the memory studies instead of the benchmark line.

N > 1 (under torchrun): independent replicas of the same step on every GPU, no data-path
collective ("replicas only"); NCCL is used only for the barrier and the max over ranks.
--impl reference times the CPU oracle (fp64, numpy) on the host cores instead.
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

METRIC = "moonwalk_grad_samples_per_s"
UNIT = "samples/s"
NOMINAL_TF32_OVER_BF16 = 1.1 / 2.25      # dense tensor peaks, nominal ratio
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# DRAM bytes (read + written) per launch of the product kernel, averaged over the launches of this
# benchmark's default workload (670 captured launches; profiles/tc_group_kernel_traffic_deep_mlp.md).
# Other workloads have no capture: their `traffic` is null.
NCU_TRAFFIC_BYTES_PER_LAUNCH = {"deep_mlp": 115.4e6}


def workload(name: str, seed: int = 0, depth: int = 0, block: int = 0):
    from paper_2402_14212_b200 import synth as S
    if name == "deep_mlp":
        return S.deep_mlp(seed=seed)
    if name == "deep_mlp_small":
        return S.deep_mlp(seed=seed, depth=8, n=256, batch=128)
    if name == "mixed_mlp":
        return S.mixed_mlp(seed=seed)
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


def time_oracle(p, seconds_target: float, max_reps: int = 50, samples: int = 0):
    """Oracle (as it stands) on the host cores: Algorithm 1 with the same re-seed interval, on the
    first `samples` rows of the batch (0 = the whole batch)."""
    import numpy as np
    from oracle import moonwalk_oracle as O
    b = samples or p.batch
    x, t = np.asarray(p.x[:b], dtype=np.float64), p.target[:b]
    reps, t0 = 0, time.perf_counter()
    while True:
        O.moonwalk(p.layers, p.params, x, t, p.loss, reseed_every=p.reseed_every, frag_block=p.frag_block)
        reps += 1
        dt = time.perf_counter() - t0
        if dt >= seconds_target or reps >= max_reps:
            break
    return b * reps / dt, reps, dt, b


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
    import numpy as np
    from oracle import moonwalk_oracle as O
    from paper_2402_14212_b200 import synth as S
    p = workload(args.workload, depth=args.depth, block=args.frag_block)
    total = args.steps + args.warmup
    # cost of one sample, then as many rows of the batch as the time budget allows
    probe = 1 if p.layers[0].kind in ("conv2d", "conv1d") else min(8, p.batch)
    t0 = time.perf_counter()
    O.moonwalk(p.layers, p.params, np.asarray(p.x[:probe], dtype=np.float64), p.target[:probe], p.loss,
               reseed_every=p.reseed_every, frag_block=p.frag_block)
    t_one = (time.perf_counter() - t0) / probe
    budget = 150.0
    b = int(budget / (t_one * total))
    b = max(1, min(b, p.batch))
    x, t = np.asarray(p.x[:b], dtype=np.float64), p.target[:b]

    def step():
        O.moonwalk(p.layers, p.params, x, t, p.loss, reseed_every=p.reseed_every, frag_block=p.frag_block)

    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = time.perf_counter() - t0
    value = b * args.steps / dt
    cores = blas_threads()
    sample = f"{b} of {p.batch} samples per step, all {len(p.layers)} layers, fp64 numpy"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT,
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": 1e3 * dt / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": describe(p),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                             "sample": sample},
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

    p = workload(args.workload, depth=args.depth, block=args.frag_block)
    net = mwb.net_for(p, backend=args.backend)
    params, x, target = mwb.to_device(p, dev)
    ws = net.alloc_workspace("moonwalk", dev)
    mw_bytes, bp_bytes, (mw_res, bp_res) = net.workspace_bytes()
    # nets of strided submersive convolutions keep the part of g0 that the sweep reads inside the
    # workspace (mw_input_cotangent with g0_out = NULL); the others hand g0 over in full
    lean = p.layers[0].kind == "conv2d" and p.layers[0].stride != 1 and not args.full_g0
    g0 = None if lean else torch.empty(x.shape, dtype=net.grad_dtype(), device=dev)
    dW = [torch.empty(w.shape, dtype=net.grad_dtype(), device=dev) for w in params]
    loss = torch.zeros(1, dtype=torch.float64, device=dev)
    stream = torch.cuda.current_stream()

    def step():
        net.input_cotangent(params, x, target, ws, g0_out=g0, loss_out=loss, keep_seed=lean)
        net.forward_sweep(params, x, g0, ws, dW_out=dW)

    for _ in range(max(args.warmup, 3)):
        step()
    code, detail = net.last_device_status(ws)
    if code != 0:
        raise SystemExit(f"device status {code} {detail} during warm-up")

    # ---- device-resident timing: K steps, events on the launching stream --------------------
    sampler = ClockSampler(local)
    barrier()
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches0 = mwb.launch_count()
    e0.record(stream)
    for _ in range(args.steps):
        step()
    e1.record(stream)
    barrier()
    launches = mwb.launch_count() - launches0
    clocks = sampler.stop()
    ms = e0.elapsed_time(e1)
    value, ms_max = aggregate_replicas(ms, p.batch, args.steps, world, dev)

    # ---- phase split (device timed, a few extra steps) --------------------------------------
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
    reps = min(args.steps, 5)
    t_cot = t_sweep = 0.0
    for _ in range(reps):
        ev[0].record(stream)
        net.input_cotangent(params, x, target, ws, g0_out=g0, loss_out=loss, keep_seed=lean)
        ev[1].record(stream)
        net.forward_sweep(params, x, g0, ws, dW_out=dW)
        ev[2].record(stream)
        torch.cuda.synchronize()
        t_cot += ev[0].elapsed_time(ev[1])
        t_sweep += ev[1].elapsed_time(ev[2])
    t_cot /= reps
    t_sweep /= reps

    # ---- the library's own backprop on the same inputs (optional: needs its workspace too) ----
    t_bp = None
    if args.with_backprop:
        ws_bp = net.alloc_workspace("backprop", dev)
        for _ in range(2):
            net.backprop_reference(params, x, target, ws_bp, dW_out=dW)
        ev[0].record(stream)
        for _ in range(reps):
            net.backprop_reference(params, x, target, ws_bp, dW_out=dW)
        ev[1].record(stream)
        torch.cuda.synchronize()
        t_bp = ev[0].elapsed_time(ev[1]) / reps
        del ws_bp

    # ---- end to end through the C ABI with host buffers --------------------------------------
    xh = x.cpu().pin_memory()
    th = target.cpu().pin_memory()
    lh = torch.zeros(1, dtype=torch.float64).pin_memory()
    xd, td = torch.empty_like(x), torch.empty_like(target)
    for _ in range(2):
        net.gradient_step_host(params, xh, th, xd, td, g0, dW, loss, lh, ws)
    barrier()
    w0 = time.perf_counter()
    e0.record(stream)
    for _ in range(args.steps):
        net.gradient_step_host(params, xh, th, xd, td, g0, dW, loss, lh, ws)
    e1.record(stream)
    barrier()
    wall = time.perf_counter() - w0
    ms_e2e = max(e0.elapsed_time(e1), 0.0)
    e2e_value, _ = aggregate_replicas(max(ms_e2e, wall * 1e3), p.batch, args.steps, world, dev)
    h2d = xh.numel() * xh.element_size() + th.numel() * th.element_size()

    # ---- roofline of the dominant kernel: per-launch events over the same K steps ------------
    roof = None
    if net.prec != "f64":
        barrier()
        mwb.profile_begin()
        for _ in range(args.steps):
            step()
        prof = mwb.profile_end()
        pk = peaks()
        src = pk["_source"]
        bf16_peak = float(pk.get("bf16_tflops_sustained", pk["bf16_tflops"]))
        if p.prec == "f32":
            peak = bf16_peak * NOMINAL_TF32_OVER_BF16
            peak_note = f"{src} sustained bf16 x nominal tf32/bf16 ratio (fp32 products)"
        else:
            peak = bf16_peak
            peak_note = f"{src} sustained bf16"
        if prof["launches"]:
            achieved = prof["flops"] / (prof["total_ms"] * 1e-3) / 1e12
            executed = prof["mma_flops"] / (prof["total_ms"] * 1e-3) / 1e12
            roof = {"bound": "tensor", "kernel": "tc_group_kernel (tcgen05 products: programs and grouped launches)",
                    "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
                    "traffic": NCU_TRAFFIC_BYTES_PER_LAUNCH.get(p.name), "peak_source": peak_note,
                    "launches_per_step": prof["launches"] / args.steps,
                    "avg_launch_us": 1e3 * prof["total_ms"] / prof["launches"],
                    "algorithmic_flops_per_launch": prof["flops"] / prof["launches"],
                    "executed_bf16_tflops": executed, "executed_frac_of_bf16_peak": executed / bf16_peak,
                    "kernel_time_share_of_step": prof["total_ms"] / (ms_max if world == 1 else ms)}
            # the same kernel inside the forward sweep alone (Algorithm 1's loop: the part the paper
            # prices; the input-cotangent call with its per-step inverses is left outside the events)
            sw = {"total_ms": 0.0, "launches": 0, "flops": 0.0, "mma_flops": 0.0}
            for _ in range(min(args.steps, 5)):
                net.input_cotangent(params, x, target, ws, g0_out=g0, loss_out=loss, keep_seed=lean)
                torch.cuda.synchronize()
                mwb.profile_begin()
                net.forward_sweep(params, x, g0, ws, dW_out=dW)
                one = mwb.profile_end()
                for k in sw:
                    sw[k] += one[k]
            if sw["launches"]:
                a_sw = sw["flops"] / (sw["total_ms"] * 1e-3) / 1e12
                e_sw = sw["mma_flops"] / (sw["total_ms"] * 1e-3) / 1e12
                roof["forward_sweep_only"] = {
                    "achieved": a_sw, "frac": a_sw / peak, "executed_bf16_tflops": e_sw,
                    "executed_frac_of_bf16_peak": e_sw / bf16_peak,
                    "avg_launch_us": 1e3 * sw["total_ms"] / sw["launches"]}

    # ---- the oracle on the host cores (rank 0, single GPU only) -----------------------------
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        # the large convolutional workload is sampled: one image of the batch through all layers
        v, reps_o, dt, b_o = time_oracle(p, 10.0, samples=1 if p.name in ("strided_cnn", "fragmental_cnn1d") else 0)
        cpu = {"value": v, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
               "sample": f"{reps_o} steps of {b_o} of {p.batch} samples, all {len(p.layers)} layers, in {dt:.1f} s, "
                         "Algorithm 1 in fp64 numpy"}

    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": max(args.warmup, 3), "ms_per_step": ms_max / args.steps,
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                "dtype": {"f64": "f64", "f32": "f32 (bf16x3 split on tensor cores, fp32 accumulate)",
                          "bf16_f32acc": "bf16 (fp32 accumulate)"}[p.prec]
                if net_backend_is_tensor(net) else ("f64" if p.prec == "f64" else "f32"),
                "data": "synthetic",
                "config": dict(describe(p), parallelism=f"replicas x{world}" if world > 1 else "single GPU",
                               l2="working set (weights, term planes, inverses, gradients) "
                                  "far above the 126 MB L2; no flush between steps"),
                "clocks": clocks, "gpu_launches": launches,
                "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d,
                        "d2h_bytes_per_step": 8},
                "roofline": roof, "cpu_baseline": cpu,
                "phases_ms": {"prep_phase1_phase2": t_cot, "forward_sweep": t_sweep, "backprop": t_bp},
                "memory_bytes": {"moonwalk_workspace": mw_bytes, "backprop_workspace": bp_bytes,
                                 "moonwalk_residual": mw_res, "backprop_residual": bp_res,
                                 "params": sum(w.numel() * w.element_size() for w in params),
                                 "grads": sum(g.numel() * g.element_size() for g in dW)}}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def run_depth_sweep(args):
    """Config 5: dense leaky-ReLU MLP, width 4096, batch 1024, bf16 / fp32 accumulate, depth
    doubling from 32.  Per depth: workspace and residual bytes of both methods (from the library's
    own accounting), peak device bytes seen by the allocator, samples/s; and the largest depth whose
    total (parameters + gradients + workspace) fits 64 GB, from the same accounting."""
    import torch
    from paper_2402_14212_b200 import binding as mwb
    from paper_2402_14212_b200 import synth as S
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    n, batch, budget = 4096, 1024, 64e9
    base = S.sweep_mlp(seed=0, depth=4, pool=4)
    pool_dev = [torch.from_numpy(w).to(torch.bfloat16).to(dev) for w in base.params[:4]]
    x = torch.from_numpy(base.x).to(torch.bfloat16).to(dev)
    target = torch.from_numpy(base.target).to(torch.float32).to(dev)

    def accounting(depth, resident):
        layers = [base.layers[0]] * depth
        net = mwb.Net(layers, batch, base.prec, base.loss, reseed_every=base.reseed_every,
                      backend="tensor", resident_inverse=resident)
        mw_b, bp_b, (mw_res, bp_res) = net.workspace_bytes()
        return net, mw_b, bp_b, mw_res, bp_res

    pbytes, gbytes = n * n * 2, n * n * 4
    rows = []
    depth = 32
    while depth <= args.max_depth:
        net, mw_b, bp_b, mw_res, bp_res = accounting(depth, False)
        row = {"depth": depth, "params_bytes": depth * pbytes,
               "moonwalk": {"workspace_bytes": mw_b, "residual_bytes": mw_res},
               "backprop": {"workspace_bytes": bp_b, "residual_bytes": bp_res}}
        # gradients streamed: layer l's dW lands in one of two rotating buffers (applied and
        # dropped, Algorithm 1's last line), so the totals below exclude a full set of gradients
        params = [pool_dev[l % 4].clone() for l in range(depth)]
        dW2 = [torch.empty((n, n), dtype=torch.float32, device=dev) for _ in range(2)]
        dW = [dW2[l & 1] for l in range(depth)]
        g0 = torch.empty((batch, n), dtype=torch.float32, device=dev)
        for which in ("moonwalk", "backprop"):
            torch.cuda.synchronize()
            torch.cuda.reset_peak_memory_stats(dev)
            before = torch.cuda.memory_allocated(dev)
            ws = net.alloc_workspace(which, dev)
            ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]

            def step():
                if which == "moonwalk":
                    net.input_cotangent(params, x, target, ws, g0_out=g0)
                    net.forward_sweep(params, x, g0, ws, dW_out=dW)
                else:
                    net.backprop_reference(params, x, target, ws, dW_out=dW)

            step()
            code, detail = net.last_device_status(ws)
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
        rows.append(row)
        del params, dW, dW2, net
        torch.cuda.empty_cache()
        depth *= 2

    def max_depth(which, keep_grads):
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

    out = {"workload": "depth sweep: dense leaky-ReLU MLP, width 4096, batch 1024, bf16 storage / fp32 accumulate",
           "per_layer_bytes": {"params_bf16": pbytes, "grad_fp32": gbytes,
                               "backprop_stored_activation_bf16": batch * n * 2,
                               "moonwalk_sign_bits": batch * n // 8,
                               "moonwalk_cotangent_checkpoint_fp32_every_K": batch * n * 4,
                               "K": base.reseed_every},
           "rows": rows,
           "max_depth_under_64GB": {
               "moonwalk_grads_streamed": max_depth("moonwalk", False),
               "backprop_grads_streamed": max_depth("backprop", False),
               "moonwalk_grads_kept": max_depth("moonwalk", True),
               "backprop_grads_kept": max_depth("backprop", True)}}
    print(json.dumps(out), flush=True)


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
    ap.add_argument("--workload", default="deep_mlp")
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
    ap.add_argument("--max-depth", type=int, default=512)
    ap.add_argument("--memory-table", action="store_true",
                    help="the paper's CNN memory experiments from the library's byte accounting "
                         "(prints one JSON object; runs without a GPU)")
    args = ap.parse_args()
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
