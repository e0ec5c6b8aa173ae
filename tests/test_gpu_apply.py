"""The sweep with Algorithm 1's last line fused in ("apply g_i to theta_i"): parameters after one
step of gradient descent against the oracle's, on the same seeded inputs, replaying the GPU's sign
bits."""
import numpy as np
import pytest

from oracle import moonwalk_oracle as O
from paper_2402_14212_b200 import binding as mwb
from paper_2402_14212_b200 import synth as S
from parity_util import oracle_masks_from_words

pytestmark = pytest.mark.gpu


def problems():
    return [
        ("dense", S.deep_mlp(seed=1, depth=6, n=256, batch=64, reseed_every=2)),
        ("dense_transient", S.deep_mlp(seed=2, depth=5, n=128, batch=128, reseed_every=4)),
        ("conv", S.submersive_cnn(seed=3, depth=3, C=64, H=8, W=16, batch=2, gamma=0.05, classes=10,
                                  reseed_every=2, conv_vijp_iters=10, prec=S.F32)),
        ("strided", S.strided_cnn(seed=4, depth=3, C=128, H=32, W=32, batch=4, gamma=0.5, reseed_every=2,
                                  prec=S.F32)),
        ("conv1d", S.fragmental_cnn1d(seed=6, depth=3, C=64, N=128, batch=4, block=8, reseed_every=2,
                                      prec=S.F32)),
    ]


@pytest.mark.parametrize("name,p", problems(), ids=[n for n, _ in problems()])
@pytest.mark.parametrize("in_place", [False, True])
def test_fused_update_matches_oracle(name, p, in_place):
    import torch
    net = mwb.net_for(p, backend="tensor", resident_inverse=(name != "dense_transient"))
    params, x, target = mwb.to_device(p)
    ws = net.alloc_workspace("moonwalk")
    g0 = net.input_cotangent(params, x, target, ws)
    masks = oracle_masks_from_words(p, [net.export_masks(ws, l) for l in range(len(p.layers))])
    ref_grad = O.backprop(p.layers, p.params, p.x, p.target, p.loss, masks=masks)["dW"]
    lr = 0.05 * max(float(np.abs(w).max()) for w in p.params) / max(float(np.abs(g).max()) for g in ref_grad)
    ref = O.moonwalk_sgd_step(p.layers, p.params, p.x, p.target, p.loss, lr, reseed_every=p.reseed_every,
                              masks=masks, conv_iters=p.conv_vijp_iters or None, frag_block=p.frag_block)
    before = [w.clone() for w in params]
    out = params if in_place else [torch.empty_like(w) for w in params]
    net.forward_sweep_apply(params, x, g0, lr, ws, params_out=out)
    assert net.last_device_status(ws)[0] == 0
    for l, (got, want, g, w0) in enumerate(zip(out, ref, ref_grad, before)):
        got = got.double().cpu().numpy().reshape(want.shape)
        err = float(np.abs(got - want).max())
        bound = 1e-4 * lr * float(np.abs(g).max()) + 2e-7 * float(np.abs(want).max())
        assert err <= bound, (l, err, bound)
        if not in_place:
            assert torch.equal(params[l], w0)          # the inputs are left alone
        # and the step is not a no-op
        assert float(np.abs(got - w0.double().cpu().numpy().reshape(want.shape)).max()) > 100 * bound


def test_fused_update_unsupported_precisions():
    p = S.mixed_mlp(seed=0, depth=2, n=128, batch=64)
    net = mwb.net_for(p, backend="tensor")
    params, x, target = mwb.to_device(p)
    ws = net.alloc_workspace("moonwalk")
    g0 = net.input_cotangent(params, x, target, ws)
    with pytest.raises(mwb.MwError):
        net.forward_sweep_apply(params, x, g0, 0.1, ws)


@pytest.mark.parametrize("name", ["dense", "strided", "conv1d"])
def test_gradient_descent_loop_follows_the_oracle(name):
    """A few steps of plain gradient descent with the update fused into the sweep, in place: the loss
    falls, and it falls the way the oracle's own loop (fp64, Algorithm 1 with theta_i updated as g_i
    appears) says it should."""
    import torch
    if name == "dense":
        p = S.deep_mlp(seed=5, depth=4, n=128, batch=64, reseed_every=2)
    elif name == "strided":
        p = S.strided_cnn(seed=5, depth=3, C=64, H=32, W=32, batch=4, gamma=0.5, reseed_every=2, prec=S.F32)
    else:
        p = S.fragmental_cnn1d(seed=5, depth=3, C=64, N=128, batch=4, block=8, reseed_every=2, prec=S.F32)
    g = O.backprop(p.layers, p.params, p.x, p.target, p.loss)["dW"]
    lr = 0.02 * max(float(np.abs(w).max()) for w in p.params) / max(float(np.abs(d).max()) for d in g)
    steps = 4
    theta = [np.array(w) for w in p.params]
    want = []
    for _ in range(steps):
        want.append(O.backprop(p.layers, theta, p.x, p.target, p.loss)["loss"])
        theta = O.moonwalk_sgd_step(p.layers, theta, p.x, p.target, p.loss, lr, reseed_every=p.reseed_every,
                                    frag_block=p.frag_block)
    net = mwb.net_for(p, backend="tensor")
    params, x, target = mwb.to_device(p)
    ws = net.alloc_workspace("moonwalk")
    loss = torch.zeros(1, dtype=torch.float64, device="cuda")
    got = []
    for _ in range(steps):
        g0 = net.input_cotangent(params, x, target, ws, loss_out=loss)
        got.append(float(loss.item()))
        net.forward_sweep_apply(params, x, g0, lr, ws)
    assert net.last_device_status(ws)[0] == 0
    assert all(b < a for a, b in zip(got, got[1:]))
    for a, b in zip(got, want):
        assert abs(a - b) <= 2e-4 * abs(b), (got, want)
    for w, t in zip(params, theta):
        assert O.normwise_error(w.double().cpu().numpy().reshape(t.shape), t) <= 1e-4
