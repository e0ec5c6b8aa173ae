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


@pytest.mark.parametrize("depth,resident", [(32, True), (32, False), (64, True)])
def test_config5_full_width(depth, resident):
    # width 4096, batch 1024, bf16; four distinct weight matrices cycled over the depth.  Depth 32
    # is the benchmark's workload (every inverse resident: the chained sweep) and, with one
    # transient inverse slot, the first point of the depth study; depth 64 is its second point.
    p = S.sweep_mlp(seed=0, depth=depth, pool=4)
    out, ref, errs = check_problem(p, 2e-2, backend="tensor", resident=resident, exact_masks=False, tau=2e-2)
    assert len(errs) == depth


@pytest.mark.parametrize("form", ["pair_chains", "default", "single", "launch_per_layer"])
@pytest.mark.parametrize("n,depth,batch,K", [(256, 8, 256, 4), (512, 10, 512, 4), (256, 9, 768, 3)])
def test_bf16_mixed_pair_sizes(n, depth, batch, K, form):
    """Sizes at which every product qualifies for the CTA-pair form (batch and width multiples of
    256).  The sweep runs as chains of row blocks inside program launches: on CTA pairs
    (forced here, since so few tiles would choose single CTAs), in the form the tile count
    chooses (Phases I-II on pairs, the sweep on single CTAs), with the pair form switched off
    everywhere, and as one launch per layer; each against the oracle."""
    from paper_2402_14212_b200 import binding as mwb
    old_pair = mwb.set_pair_mode(form != "single")
    old_chains = mwb.set_sweep_chains({"pair_chains": 2, "launch_per_layer": 0}.get(form, 1))
    try:
        p = S.mixed_mlp(seed=4, depth=depth, n=n, batch=batch, reseed_every=K, prec=S.BF16)
        check_problem(p, 2e-2, backend="tensor", exact_masks=False, tau=2e-2)
    finally:
        mwb.set_pair_mode(old_pair)
        mwb.set_sweep_chains(old_chains)


@pytest.mark.parametrize("chains", [1, 2])
def test_bf16_pair_sizes_gradients_skipped(chains):
    """dW_out entries left out (gradients need not coexist): the chained sweep (on single CTAs and
    on CTA pairs) drops the weight vjp of those layers and still carries the cotangent through."""
    import torch
    from paper_2402_14212_b200 import binding as mwb
    from oracle import moonwalk_oracle as O
    from parity_util import oracle_masks_from_words
    p = S.sweep_mlp(seed=5, depth=7, n=256, batch=256, reseed_every=3, prec=S.BF16)
    old_chains = mwb.set_sweep_chains(chains)
    net = mwb.net_for(p, backend="tensor")
    params, x, target = mwb.to_device(p)
    ws = net.alloc_workspace("moonwalk")
    g0 = net.input_cotangent(params, x, target, ws)
    keep = [0, 2, 3, 6]
    dW = [torch.zeros(w.shape, dtype=torch.float32, device="cuda") if l in keep else None
          for l, w in enumerate(params)]
    try:
        net.forward_sweep(params, x, g0, ws, dW_out=dW)
    finally:
        mwb.set_sweep_chains(old_chains)
    code, detail = net.last_device_status(ws)
    assert code == 0, detail
    masks = oracle_masks_from_words(p, [net.export_masks(ws, l) for l in range(len(p.layers))])
    ref = O.backprop(p.layers, p.params, p.x, p.target, p.loss, masks=masks)
    for l in keep:
        assert O.normwise_error(dW[l].double().cpu().numpy(), ref["dW"][l]) <= 2e-2, l


@pytest.mark.parametrize("kind", ["pair", "fp32_small"])
def test_bucket_events_and_single_rank_data_parallel_step(kind):
    """mw_sweep_bucket_events: the sweep records one event per bucket of layers (a launch per bucket
    where the sweep runs as chains); the data-parallel step built on it, with one rank, returns the
    gradients of the plain step bit for bit."""
    import torch
    from paper_2402_14212_b200 import binding as mwb
    from paper_2402_14212_b200 import data_parallel as dp
    if kind == "pair":
        p = S.sweep_mlp(seed=6, depth=7, n=256, batch=256, reseed_every=3, prec=S.BF16)
    else:
        p = S.deep_mlp(seed=6, depth=5, n=128, batch=40, reseed_every=2, prec=S.F32)
    net = mwb.net_for(p, backend="tensor")
    params, x, target = mwb.to_device(p)
    ws = net.alloc_workspace("moonwalk")
    g0 = net.input_cotangent(params, x, target, ws)
    plain = [d.clone() for d in net.forward_sweep(params, x, g0, ws)]
    step = dp.DataParallelStep(net, p.loss, world=1, layers_per_bucket=3)
    assert len(step.events) == (len(p.layers) + 2) // 3
    dW = [torch.zeros_like(d) for d in plain]
    step.step(params, x, target, ws, g0, dW)
    torch.cuda.synchronize()
    assert net.last_device_status(ws)[0] == 0
    assert all(e.query() for e in step.events)
    for a, b in zip(plain, dW):
        assert torch.equal(a, b)
    net.set_bucket_events(0)
    again = net.forward_sweep(params, x, g0, ws)
    for a, b in zip(plain, again):
        assert torch.equal(a, b)


@pytest.mark.parametrize("prec,n,batch,iters,tol", [(S.BF16, 512, 256, 3, 2e-2), (S.F32, 256, 64, 4, 1e-4),
                                                   (S.BF16, 512, 256, 1, 6e-2)])
def test_inverse_iters_changes_the_newton_schulz_schedule(prec, n, batch, iters, tol):
    """More steps than the default repeat the most accurate one (their residuals are computed in
    full: only the second step's is symmetric); a single step leaves the start's squared residual
    (about 4e-3 for these weights), which the looser bar allows for."""
    p = S.sweep_mlp(seed=8, depth=4, n=n, batch=batch, reseed_every=2, prec=prec)
    check_problem(p, tol, backend="tensor", inverse_iters=iters, exact_masks=False, tau=tol)


@pytest.mark.parametrize("n,batch", [(256, 256), (512, 96), (768, 512)])
def test_bf16_transient_inverse_slot(n, batch):
    """resident_inverse = 0 on bf16 nets: one inverse slot, each layer's W^-1 rebuilt in the sweep by
    single launches of the same products the program path uses (implicit start, symmetric W W^T
    and second residual), on CTA pairs or single CTAs as the sizes allow."""
    p = S.mixed_mlp(seed=9, depth=6, n=n, batch=batch, reseed_every=3, prec=S.BF16)
    check_problem(p, 2e-2, backend="tensor", resident=False, exact_masks=False, tau=2e-2)


def test_bf16_net_deeper_than_the_product_tables():
    """154 layers of width 2048 do not fit the tables of the program launches: every phase runs as a
    launch per layer, and the resident inverses are built one layer at a time."""
    p = S.mixed_mlp(seed=10, depth=154, n=2048, batch=256, reseed_every=4, prec=S.BF16)
    out, ref, errs = check_problem(p, 2e-2, backend="tensor", exact_masks=False, tau=2e-2)
    assert len(errs) == 154
