"""Small, self-ending cases of single kernels for profiler captures.

  python -m paper_2402_14212_b200.profile_cases gemm --M 256 --N 1024 --K 1024 --terms 3 --b-mn
  python -m paper_2402_14212_b200.profile_cases pack --rows 65536 --cols 2048
  python -m paper_2402_14212_b200.profile_cases fragments --rows 65536 --cols 2048
  python -m paper_2402_14212_b200.profile_cases conv --images 512 --op 1 --terms 2
  python -m paper_2402_14212_b200.profile_cases sconv --images 16 --op 0 --terms 3
  python -m paper_2402_14212_b200.profile_cases step --workload sweep_mlp --depth 4 --no-coop

Each case allocates its seeded inputs, runs the kernel `--reps` times and exits.
"""
from __future__ import annotations

import argparse

import numpy as np


def main():
    import torch
    from . import binding as mwb
    ap = argparse.ArgumentParser()
    ap.add_argument("case", choices=["gemm", "pack", "fragments", "vijp", "conv", "sconv", "step"])
    ap.add_argument("--workload", default="sweep_mlp", help="step: a workload of paper_2402_14212_b200.synth")
    ap.add_argument("--depth", type=int, default=4)
    ap.add_argument("--no-coop", action="store_true",
                    help="step: program launches without the cooperative attribute (for profilers)")
    ap.add_argument("--no-pair", action="store_true", help="one CTA per tile everywhere")
    ap.add_argument("--M", type=int, default=256)
    ap.add_argument("--N", type=int, default=1024)
    ap.add_argument("--K", type=int, default=1024)
    ap.add_argument("--terms", type=int, default=3)
    ap.add_argument("--a-mn", action="store_true")
    ap.add_argument("--b-mn", action="store_true")
    ap.add_argument("--rows", type=int, default=65536)
    ap.add_argument("--cols", type=int, default=2048)
    ap.add_argument("--reps", type=int, default=3)
    ap.add_argument("--images", type=int, default=512)
    ap.add_argument("--op", type=int, default=0, help="0 conv, 1 TransposeConv, 2 weight vjp")
    a = ap.parse_args()
    g = torch.Generator(device="cuda").manual_seed(0)
    if a.no_pair:
        mwb.set_pair_mode(False)
    if a.case == "step":
        # warm steps, then `reps` whole Moonwalk steps of a synthetic workload (launch lists)
        from . import synth as S
        make = {"sweep_mlp": lambda: S.sweep_mlp(seed=0, depth=a.depth, pool=4),
                "mixed_mlp": lambda: S.mixed_mlp(seed=0, depth=a.depth),
                "deep_mlp": lambda: S.deep_mlp(seed=0, depth=a.depth)}[a.workload]
        p = make()
        if a.no_coop:
            mwb.set_cooperative_launch(False)
        net = mwb.net_for(p, backend="tensor")
        params, x, target = mwb.to_device(p)
        ws = net.alloc_workspace("moonwalk")
        g0 = torch.empty(x.shape, dtype=torch.float32, device="cuda")
        dW = [torch.empty(w.shape, dtype=torch.float32, device="cuda") for w in params]
        for _ in range(2 + a.reps):
            net.input_cotangent(params, x, target, ws, g0_out=g0)
            net.forward_sweep(params, x, g0, ws, dW_out=dW)
        torch.cuda.synchronize()
        code, detail = net.last_device_status(ws)
        assert code == 0, (code, detail)
    elif a.case == "gemm":
        A = torch.randn((a.K, a.M) if a.a_mn else (a.M, a.K), device="cuda", generator=g)
        B = torch.randn((a.K, a.N) if a.b_mn else (a.N, a.K), device="cuda", generator=g)
        for _ in range(a.reps):
            mwb.gemm_split_bf16(A, B, a.a_mn, a.b_mn, a.terms)
    elif a.case == "sconv":
        # 3x3, stride 2, padding 1, 128 channels on 256 x 256 images: the first layer of the paper's CNN
        x = torch.randn((a.images, 256, 256, 128), device="cuda", generator=g)
        if a.op == 1:
            x = torch.randn((a.images, 128, 128, 128), device="cuda", generator=g)
        if a.op == 2:
            b = torch.randn((a.images, 128, 128, 128), device="cuda", generator=g)
        else:
            b = torch.randn((3, 3, 128, 128), device="cuda", generator=g)
        for _ in range(a.reps):
            mwb.conv2d_strided_split_bf16(a.op, x, b, 3, 2, 1, a.terms, in_hw=(256, 256))
    elif a.case == "conv":
        # 3x3, 64 channels, 32 x 32 images, channel-last: the convolutional configuration's layer
        x = torch.randn((a.images, 32, 32, 64), device="cuda", generator=g)
        if a.op == 2:
            b = torch.randn((a.images, 32, 32, 64), device="cuda", generator=g)
        else:
            b = torch.randn((3, 3, 64, 64), device="cuda", generator=g)
        for _ in range(a.reps):
            mwb.conv2d_split_bf16(a.op, x, b, 3, a.terms)
    else:
        z = torch.randn((a.rows, a.cols), device="cuda", generator=g)
        h = torch.randn((a.rows, a.cols), device="cuda", generator=g)
        for _ in range(a.reps):
            words = mwb.pack_sign_bits(z)
            if a.case == "fragments":
                cnt, off, vals, total = mwb.relu_fragment_compact(h, words)
                mwb.activation_vijp(h, words, "relu", 0.0, off, vals)
            elif a.case == "vijp":
                mwb.activation_vijp(h, words, "leaky_relu", 0.1)
    torch.cuda.synchronize()
    print("done", a.case)


if __name__ == "__main__":
    main()
