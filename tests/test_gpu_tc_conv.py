"""Convolution steps on the tensor cores against the oracle's plain definitions (Lemma 1,
Eq. "conv-vjp", Eq. "g_i"), on the same seeded arrays."""
import numpy as np
import pytest

from oracle import moonwalk_oracle as O
from paper_2402_14212_b200 import binding as mwb

pytestmark = pytest.mark.gpu

TOL = {1: 2e-2, 2: 2e-4, 3: 2e-6}


@pytest.mark.parametrize("terms", [1, 2, 3])
@pytest.mark.parametrize("images,H,W,k", [(1, 4, 32, 3), (3, 8, 16, 3), (2, 16, 64, 3), (4, 32, 32, 3),
                                          (2, 8, 32, 5), (1, 4, 32, 1)])
def test_conv_products(images, H, W, k, terms):
    import torch
    assert torch.cuda.is_available()
    rng = np.random.default_rng(images * 100 + H + W + k + terms)
    x = rng.standard_normal((images, H, W, 64)).astype(np.float32)
    g = rng.standard_normal((images, H, W, 64)).astype(np.float32)
    w = (rng.standard_normal((k, k, 64, 64)) / np.sqrt(64 * k * k)).astype(np.float32)
    # marks that a wrong shift, a transposed tap or a swapped channel pair would move
    x[0, 0, 0, :] = 0.0; x[0, 0, 0, 1] = 3.0
    w[0, k - 1, 1, 2] = 1.5
    p = k // 2
    xt, gt, wt = (torch.from_numpy(a).cuda() for a in (x, g, w))
    x64, g64, w64 = x.astype(np.float64), g.astype(np.float64), w.astype(np.float64)
    cases = [(0, xt, wt, O.conv_forward(x64, w64, 1, p)),
             (1, gt, wt, O.transpose_conv(g64, w64, (H, W), 1, p)),
             (2, xt, gt, O.conv_weight_vjp(x64, g64, k, 1, p))]
    for op, a, b, ref in cases:
        got = mwb.conv2d_split_bf16(op, a, b, k, terms).double().cpu().numpy()
        err = np.abs(got - ref).max() / np.abs(ref).max()
        assert err <= TOL[terms], (op, err)


# ---------------------------------------------------------------------------------------
# whole path on the tensor-core convolution pipeline (fp32, 64 channels)
# ---------------------------------------------------------------------------------------
@pytest.mark.parametrize("depth,H,W,batch,K,iters,resident", [(3, 8, 16, 2, 2, 10, True), (4, 4, 32, 3, 0, 12, True), (6, 4, 32, 2, 3, 10, True),
                                                              (4, 16, 64, 1, 3, 10, False)])
def test_small_cnn_fp32_tensor_path(depth, H, W, batch, K, iters, resident):
    from paper_2402_14212_b200 import synth as S
    from parity_util import check_problem
    p = S.submersive_cnn(seed=depth, depth=depth, C=64, H=H, W=W, batch=batch, gamma=0.05, classes=10,
                         reseed_every=K, conv_vijp_iters=iters, prec=S.F32)
    out, ref, errs = check_problem(p, 1e-4, backend="tensor", resident=resident, exact_masks=False,
                                   tau=1e-4)


@pytest.mark.gpu
@pytest.mark.parametrize("terms", [1, 3])
@pytest.mark.parametrize("images,H,W,C", [(2, 16, 16, 128), (1, 64, 64, 128), (4, 8, 8, 64), (16, 4, 4, 128),
                                          (64, 2, 2, 128), (1, 256, 256, 64), (3, 32, 16, 128)])
def test_strided_conv_products(images, H, W, C, terms):
    """3x3, stride 2, padding 1 (the paper's submersive layer): forward, TransposeConv through its
    four parity classes, weight vjp; tiles that are part of a row, rows of an image, whole images."""
    import torch
    from paper_2402_14212_b200 import binding as mwb
    rng = np.random.default_rng(images * 1000 + H)
    k, s, p = 3, 2, 1
    Ho, Wo = (H + 2 * p - k) // s + 1, (W + 2 * p - k) // s + 1
    x = rng.standard_normal((images, H, W, C)).astype(np.float32)
    w = (rng.standard_normal((k, k, C, C)) / np.sqrt(C * k * k)).astype(np.float32)
    g = rng.standard_normal((images, Ho, Wo, C)).astype(np.float32)
    w[0, 2, 1, 2] = 1.5
    xt, wt, gt = (torch.from_numpy(v).cuda() for v in (x, w, g))
    x64, w64, g64 = x.astype(np.float64), w.astype(np.float64), g.astype(np.float64)
    tol = {1: 2e-2, 3: 2e-6}[terms]
    cases = [(0, xt, wt, None, O.conv_forward(x64, w64, s, p)),
             (1, gt, wt, (H, W), O.transpose_conv(g64, w64, (H, W), s, p))]
    if (images * Ho * Wo) % 64 == 0:
        cases.append((2, xt, gt, None, O.conv_weight_vjp(x64, g64, k, s, p)))
    for op, a, b, hw, ref in cases:
        got = mwb.conv2d_strided_split_bf16(op, a, b, k, s, p, terms, in_hw=hw).double().cpu().numpy()
        assert got.shape == ref.shape
        err = np.abs(got - ref).max() / np.abs(ref).max()
        assert err < tol, (op, err)


# ---------------------------------------------------------------------------------------
# whole path on the fully submersive strided CNN (3x3, stride 2, padding 1; Lemma 1, Algorithm 2)
# ---------------------------------------------------------------------------------------
@pytest.mark.parametrize("depth,C,H,W,batch,K", [(4, 128, 32, 32, 16, 2), (3, 64, 64, 32, 4, 0),
                                                 (5, 128, 32, 32, 64, 4), (2, 128, 128, 128, 1, 0)])
def test_strided_cnn_fp32_tensor_path(depth, C, H, W, batch, K):
    from paper_2402_14212_b200 import synth as S
    from parity_util import check_problem
    p = S.strided_cnn(seed=depth, depth=depth, C=C, H=H, W=W, batch=batch, gamma=0.5, reseed_every=K,
                      prec=S.F32)
    out, ref, errs = check_problem(p, 1e-4, backend="tensor", exact_masks=False, tau=1e-4)
    # the literal Algorithm 1 with Lemma 1's elimination as the vijp reaches the same gradients
    mw = O.moonwalk(p.layers, p.params, p.x, p.target, p.loss, reseed_every=K,
                    masks=[m.reshape(z.shape) for m, z in zip(ref["masks"], ref["z"])])
    for l in range(depth):
        assert O.normwise_error(mw["dW"][l], ref["dW"][l]) < 1e-7


@pytest.mark.parametrize("depth,C,H,W,batch,K", [(4, 128, 32, 32, 16, 2), (3, 64, 64, 32, 4, 4), (5, 128, 32, 32, 64, 4)])
def test_strided_cnn_bf16_tensor_path(depth, C, H, W, batch, K):
    """bf16 inputs and weights with fp32 accumulation: single-term operands on the forward products,
    two-term cotangents; bar 2e-2 against the oracle on the bf16-rounded inputs (mask replay)."""
    from paper_2402_14212_b200 import synth as S
    from parity_util import check_problem
    p = S.strided_cnn(seed=depth, depth=depth, C=C, H=H, W=W, batch=batch, gamma=0.5, reseed_every=K,
                      prec=S.BF16)
    out, ref, errs = check_problem(p, 2e-2, backend="tensor", exact_masks=False, tau=2e-2)


def test_strided_cnn_lean_seed_gives_the_same_gradients():
    """With g0_out = NULL only the pixels (s y, s x) of the input cotangent are computed and kept in
    the workspace; the sweep started from them returns the same gradients (the seed holds the same
    values, split into term planes by the product's epilogue instead of a separate kernel)."""
    import torch
    from paper_2402_14212_b200 import synth as S
    p = S.strided_cnn(seed=3, depth=4, C=128, H=32, W=32, batch=16, gamma=0.5, reseed_every=2, prec=S.F32)
    net = mwb.net_for(p, backend="tensor")
    params, x, target = mwb.to_device(p)
    ws = net.alloc_workspace("moonwalk")
    g0 = net.input_cotangent(params, x, target, ws)
    dW_full = [d.clone() for d in net.forward_sweep(params, x, g0, ws)]
    assert net.input_cotangent(params, x, target, ws, keep_seed=True) is None
    dW_lean = net.forward_sweep(params, x, None, ws)
    assert net.last_device_status(ws)[0] == 0
    for a, b in zip(dW_full, dW_lean):
        assert float((a - b).abs().max()) <= 1e-6 * float(a.abs().max())
    # a dense net has no such part to keep: g0 is required
    q = S.deep_mlp(seed=0, depth=2, n=64, batch=64)
    dn = mwb.net_for(q, backend="tensor")
    qp, qx, qt = mwb.to_device(q)
    with pytest.raises(mwb.MwError):
        dn.input_cotangent(qp, qx, qt, dn.alloc_workspace("moonwalk"), keep_seed=True)


def test_strided_cnn_rejects_non_submersive_anchor():
    """An anchor tap with an entry above the diagonal violates Lemma 1 (ii): the device status says so."""
    import torch
    from paper_2402_14212_b200 import synth as S
    p = S.strided_cnn(seed=1, depth=2, C=64, H=16, W=16, batch=4, gamma=0.5, reseed_every=0, prec=S.F32)
    p.params[1][1, 1, 0, 3] = 0.25
    net = mwb.net_for(p, backend="tensor")
    params, x, target = mwb.to_device(p)
    ws = net.alloc_workspace("both")
    net.input_cotangent(params, x, target, ws)
    code, detail = net.last_device_status(ws)
    assert code == mwb.STATUS_NAMES.index("MW_ERR_NOT_SUBMERSIVE")


@pytest.mark.parametrize("prec,tol", [("f32", 1e-4), ("bf16_f32acc", 2e-2)])
def test_strided_cnn_full_size(prec, tol):
    """The paper's experiment at full size (256 x 256 x 128 inputs, batch 128, 8 stride-2 layers), in
    the launch configuration the benchmark times.  The oracle handles the batch in slices (samples
    are independent but for the batch sums of dW and of the loss), replaying the GPU's sign bits."""
    import torch
    from paper_2402_14212_b200 import synth as S
    from parity_util import run_gpu
    p = S.strided_cnn(seed=0, prec=prec)
    out = run_gpu(p, backend="tensor", backprop=False)
    assert out["status"] == 0
    L, B = len(p.layers), p.batch
    n_last = p.target[0].size
    dW = [np.zeros_like(w) for w in p.params]
    loss, g0_err, worst = 0.0, 0.0, [0.0] * L
    step = 8
    for b0 in range(0, B, step):
        sl = slice(b0, b0 + step)
        masks = []
        for l, layer in enumerate(p.layers):
            ho, wo = layer.out_hw()
            words = out["masks"][l].reshape(B, ho * wo, -1)[sl].reshape(step * ho * wo, -1)
            masks.append(O.unpack_mask(words, layer.C_out).reshape(step, ho, wo, layer.C_out))
        x = np.asarray(p.x[sl], dtype=np.float64)
        ref = O.backprop(p.layers, p.params, x, p.target[sl], p.loss, masks=masks)
        # mse_mean divides by the elements of ITS batch: rescale the slice to the whole batch
        f = step / B
        loss += ref["loss"] * f
        for l in range(L):
            dW[l] += ref["dW"][l] * f
            z = ref["z"][l].reshape(-1, p.layers[l].C_out)
            d = masks[l].reshape(z.shape) != O.sign_mask(z)
            if d.any():
                rms = np.sqrt((z * z).mean(axis=1, keepdims=True))
                worst[l] = max(worst[l], float((np.abs(z) / rms)[d].max()))
        g = out["g0"][sl].reshape(ref["g0"].shape)
        g0_err = max(g0_err, float(np.abs(g - ref["g0"] * f).max()))
    g0_scale = float(np.abs(out["g0"]).max())
    assert g0_err <= tol * g0_scale, g0_err / g0_scale
    for l in range(L):
        assert worst[l] <= tol * np.sqrt(l + 1.0), (l, worst[l])
        assert O.normwise_error(out["dW"][l], dW[l]) <= tol, l
    assert abs(out["loss"] - loss) <= tol * abs(loss)


# ---------------------------------------------------------------------------------------
# whole path on the 1-D CNN with fragmental checkpoints (Section 5.1; k = 3, stride 1, padding 1)
# ---------------------------------------------------------------------------------------
@pytest.mark.parametrize("depth,C,N,batch,block,K", [(3, 64, 128, 2, 4, 0), (4, 256, 256, 2, 16, 2),
                                                     (5, 128, 128, 4, 8, 4), (2, 64, 256, 1, 2, 0),
                                                     (3, 128, 128, 2, 64, 0)])
def test_fragmental_cnn1d_fp32_tensor_path(depth, C, N, batch, block, K):
    from paper_2402_14212_b200 import synth as S
    from parity_util import check_problem
    p = S.fragmental_cnn1d(seed=depth, depth=depth, C=C, N=N, batch=batch, block=block, reseed_every=K,
                           prec=S.F32)
    out, ref, errs = check_problem(p, 1e-4, backend="tensor", exact_masks=False, tau=1e-4)
    # the residual store holds (k - 1) / block of one cotangent per layer, in fp32, beside the sign bits
    _, _, (mw_res, bp_res) = out["net"].workspace_bytes()
    frag_bytes = depth * 4 * batch * N * C * 2 // block
    assert mw_res >= frag_bytes


@pytest.mark.parametrize("depth,C,N,batch,block,K", [(3, 64, 128, 2, 4, 0), (4, 256, 256, 2, 16, 2),
                                                     (5, 128, 128, 4, 8, 4)])
def test_fragmental_cnn1d_bf16_tensor_path(depth, C, N, batch, block, K):
    """bf16 inputs and weights, fp32 accumulation, two-term cotangents; bar 2e-2."""
    from paper_2402_14212_b200 import synth as S
    from parity_util import check_problem
    p = S.fragmental_cnn1d(seed=depth, depth=depth, C=C, N=N, batch=batch, block=block, reseed_every=K,
                           prec=S.BF16)
    check_problem(p, 2e-2, backend="tensor", exact_masks=False, tau=2e-2)


def test_fragmental_cnn1d_stronger_taps_stated_bar():
    """The same net with the off-diagonal taps scaled by gamma = 0.5 instead of the recipe's 0.3 and
    the longest blocks (16): the block recursion g[i+1] = W0^-1 (h[i] - w1 g[i] - w2 g[i-1]) then
    amplifies fp32 rounding along its 14 steps by more than the four layers between cotangent
    checkpoints can absorb, and the layers just before a checkpoint land above the 1e-4 bar that the
    recipe's own weights meet (measured at the paper's size with seed 0: 1.4e-4; on this smaller
    net with seed 2: 1.1e-4 and 2.7e-4 at layers 3 and 7, below 2e-5 elsewhere).  The case is kept
    with the bar it does meet, 5e-4, so that a regression of the recursion still shows."""
    from paper_2402_14212_b200 import synth as S
    from parity_util import check_problem
    p = S.fragmental_cnn1d(seed=2, depth=8, C=256, N=512, batch=8, block=16, gamma=0.5, reseed_every=4,
                           prec=S.F32)
    out, ref, errs = check_problem(p, 5e-4, backend="tensor", exact_masks=False, tau=1e-4)
    assert max(errs[:3]) <= 1e-4          # away from the end of a checkpoint interval the bar holds
    # blocks of 4 (the paper's main setting) stay inside the 1e-4 bar at the same gamma
    p4 = S.fragmental_cnn1d(seed=2, depth=8, C=256, N=512, batch=8, block=4, gamma=0.5, reseed_every=4,
                            prec=S.F32)
    check_problem(p4, 1e-4, backend="tensor", exact_masks=False, tau=1e-4)


def test_fragmental_cnn1d_rejects_a_full_tap0():
    from paper_2402_14212_b200 import synth as S
    p = S.fragmental_cnn1d(seed=1, depth=2, C=64, N=128, batch=2, block=4, reseed_every=0, prec=S.F32)
    p.params[0][0, 2, 5] = 0.5                       # c < c': tap 0 is no longer triangular
    net = mwb.net_for(p, backend="tensor")
    params, x, target = mwb.to_device(p)
    ws = net.alloc_workspace("both")
    net.input_cotangent(params, x, target, ws)
    code, detail = net.last_device_status(ws)
    assert code == mwb.STATUS_NAMES.index("MW_ERR_NOT_SUBMERSIVE")


@pytest.mark.parametrize("depth,block,prec,tol", [(8, 16, "f32", 1e-4), (16, 4, "f32", 1e-4),
                                                  (16, 4, "bf16_f32acc", 2e-2)])
def test_fragmental_cnn1d_full_size(depth, block, prec, tol):
    """The paper's 1-D experiment at its size (2048 x 256 sequences, batch 128): 8 layers with blocks
    of 16 positions (the longest reconstruction the paper uses), and the benchmark's own workload --
    16 layers, blocks of 4 -- in fp32 and in bf16, in the launch configuration the benchmark times.
    The oracle takes the batch in slices, replaying the GPU's sign bits."""
    from paper_2402_14212_b200 import synth as S
    from parity_util import run_gpu
    p = S.fragmental_cnn1d(seed=0, depth=depth, block=block, prec=prec)
    out = run_gpu(p, backend="tensor", backprop=False)
    assert out["status"] == 0
    L, B = len(p.layers), p.batch
    dW = [np.zeros_like(w) for w in p.params]
    loss, g0_err, worst = 0.0, 0.0, [0.0] * L
    step = 16
    for b0 in range(0, B, step):
        sl = slice(b0, b0 + step)
        masks = []
        for l, layer in enumerate(p.layers):
            words = out["masks"][l].reshape(B, layer.W, -1)[sl].reshape(step * layer.W, -1)
            masks.append(O.unpack_mask(words, layer.C_out).reshape(step, layer.W, layer.C_out))
        ref = O.backprop(p.layers, p.params, p.x[sl], p.target[sl], p.loss, masks=masks)
        f = step / B                       # mse_mean divides by the elements of ITS batch
        loss += ref["loss"] * f
        for l in range(L):
            dW[l] += ref["dW"][l] * f
            z = ref["z"][l].reshape(-1, p.layers[l].C_out)
            d = masks[l].reshape(z.shape) != O.sign_mask(z)
            if d.any():
                rms = np.sqrt((z * z).mean(axis=1, keepdims=True))
                worst[l] = max(worst[l], float((np.abs(z) / rms)[d].max()))
        g0_err = max(g0_err, float(np.abs(out["g0"][sl].reshape(ref["g0"].shape) - ref["g0"] * f).max()))
    assert g0_err <= tol * float(np.abs(out["g0"]).max())
    for l in range(L):
        assert worst[l] <= tol * np.sqrt(l + 1.0), (l, worst[l])
        assert O.normwise_error(out["dW"][l], dW[l]) <= tol, l
    assert abs(out["loss"] - loss) <= tol * abs(loss)


@pytest.mark.parametrize("family", ["strided", "conv1d"])
def test_cnn_sweep_skips_layers_without_an_output(family):
    """A NULL entry of dW_out skips that layer's weight vjp (gradients need not coexist, Section 4.3);
    the other layers' gradients are unchanged, bit for bit."""
    import torch
    from paper_2402_14212_b200 import synth as S
    if family == "strided":
        p = S.strided_cnn(seed=7, depth=4, C=64, H=32, W=32, batch=16, gamma=0.5, reseed_every=2, prec=S.F32)
    else:
        p = S.fragmental_cnn1d(seed=7, depth=4, C=64, N=128, batch=4, block=8, reseed_every=2, prec=S.F32)
    net = mwb.net_for(p, backend="tensor")
    params, x, target = mwb.to_device(p)
    ws = net.alloc_workspace("moonwalk")
    g0 = net.input_cotangent(params, x, target, ws)
    full = [d.clone() for d in net.forward_sweep(params, x, g0, ws)]
    some = [None, torch.zeros_like(params[1]), None, torch.zeros_like(params[3])]
    net.forward_sweep(params, x, g0, ws, dW_out=some)
    assert net.last_device_status(ws)[0] == 0
    assert torch.equal(some[1], full[1]) and torch.equal(some[3], full[3])


@pytest.mark.parametrize("family", ["strided", "conv1d"])
def test_cnn_calls_can_be_repeated(family):
    """The sweep may be run again on the same workspace, and a whole step again after it, with the
    same results bit for bit (nothing a call needs is consumed by it)."""
    import torch
    from paper_2402_14212_b200 import synth as S
    if family == "strided":
        p = S.strided_cnn(seed=8, depth=3, C=64, H=32, W=32, batch=4, gamma=0.5, reseed_every=2, prec=S.F32)
    else:
        p = S.fragmental_cnn1d(seed=8, depth=3, C=64, N=128, batch=4, block=4, reseed_every=2, prec=S.F32)
    net = mwb.net_for(p, backend="tensor")
    params, x, target = mwb.to_device(p)
    ws = net.alloc_workspace("moonwalk")
    g0 = net.input_cotangent(params, x, target, ws)
    first = [d.clone() for d in net.forward_sweep(params, x, g0, ws)]
    again = net.forward_sweep(params, x, g0, ws)
    for a, b in zip(first, again):
        assert torch.equal(a, b)
    g0b = net.input_cotangent(params, x, target, ws)
    third = net.forward_sweep(params, x, g0b, ws)
    assert torch.equal(g0, g0b)
    for a, b in zip(first, third):
        assert torch.equal(a, b)
    # a sweep on a workspace that backprop has overwritten is refused
    wsb = net.alloc_workspace("both")
    g0c = net.input_cotangent(params, x, target, wsb)
    net.backprop_reference(params, x, target, wsb)
    with pytest.raises(mwb.MwError) as e:
        net.forward_sweep(params, x, g0c, wsb)
    assert e.value.code == mwb.STATUS_NAMES.index("MW_ERR_STATE")
