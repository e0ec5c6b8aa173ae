"""GPU parity of the tensor-core (tcgen05) pipelines against the CPU oracle.

fp32 nets: max relative error 1e-4; bf16-input / fp32-accumulate nets: 2e-2 (per layer, normwise).
Sign bits are compared with the oracle's own; where they differ, the oracle's |z| there must be
within tau of zero (a rounding-level sign flip) and gradients are compared against the oracle
evaluated on the GPU's exported masks.
"""
import numpy as np
import pytest

from paper_2402_14212_b200 import synth as S
from parity_util import check_problem

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("n,depth,batch,K", [(128, 8, 64, 4), (256, 6, 100, 2), (192, 5, 13, 0)])
def test_fp32_dense_small(n, depth, batch, K):
    p = S.deep_mlp(seed=1, depth=depth, n=n, batch=batch, reseed_every=K, prec=S.F32)
    check_problem(p, 1e-4, backend="tensor", exact_masks=False, tau=1e-4)


def test_fp32_dense_transient_inverse_slot():
    p = S.deep_mlp(seed=2, depth=6, n=128, batch=64, reseed_every=3, prec=S.F32)
    check_problem(p, 1e-4, backend="tensor", resident=False, exact_masks=False, tau=1e-4)


@pytest.mark.parametrize("n,depth,batch,K", [(128, 8, 64, 4), (256, 12, 96, 4), (320, 6, 40, 2)])
def test_bf16_mixed_small(n, depth, batch, K):
    p = S.mixed_mlp(seed=1, depth=depth, n=n, batch=batch, reseed_every=K, prec=S.BF16)
    check_problem(p, 2e-2, backend="tensor", exact_masks=False, tau=2e-2)


def test_bf16_leaky_only_small():
    p = S.sweep_mlp(seed=3, depth=8, n=256, batch=128, reseed_every=4, prec=S.BF16)
    check_problem(p, 2e-2, backend="tensor", exact_masks=False, tau=2e-2)


def test_config2_deep_mlp_full_size():
    # 64 layers, width 1024, batch 256, fp32: the benchmark's workload and launch configuration
    p = S.deep_mlp(seed=0)
    check_problem(p, 1e-4, backend="tensor", exact_masks=False, tau=1e-4)


def test_config4_mixed_mlp_full_size():
    # 128 layers, width 2048, batch 512, bf16 storage, alternating leaky-ReLU / ReLU with the
    # fragment stream written and read back inside the product kernel's epilogues
    p = S.mixed_mlp(seed=0)
    out, ref, errs = check_problem(p, 2e-2, backend="tensor", exact_masks=False, tau=2e-2)
    assert len(errs) == 128


def test_config5_depth32_full_width():
    # width 4096, batch 1024, bf16, depth 32 (the first point of the depth sweep); four distinct
    # weight matrices cycled over the depth
    p = S.sweep_mlp(seed=0, depth=32, pool=4)
    check_problem(p, 2e-2, backend="tensor", exact_masks=False, tau=2e-2)
