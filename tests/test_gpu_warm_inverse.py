"""warm_inverse: the workspace keeps every W^-1 between steps and mw_input_cotangent refreshes it
with the last Newton-Schulz step instead of starting over.  Gradients of a short training loop
against the oracle at every step, and the report when the weights jumped too far."""
import numpy as np
import pytest

from oracle import moonwalk_oracle as O
from paper_2402_14212_b200 import binding as mwb
from paper_2402_14212_b200 import synth as S
from parity_util import oracle_masks_from_words

pytestmark = pytest.mark.gpu


def grads_against_oracle(net, p, params, x, target, ws, theta, tol):
    g0 = net.input_cotangent(params, x, target, ws)
    dW = net.forward_sweep(params, x, g0, ws)
    code, detail = net.last_device_status(ws)
    assert code == 0, detail
    masks = oracle_masks_from_words(p, [net.export_masks(ws, l) for l in range(len(p.layers))])
    ref = O.backprop(p.layers, theta, p.x, p.target, p.loss, masks=masks)
    errs = [O.normwise_error(d.double().cpu().numpy(), r) for d, r in zip(dW, ref["dW"])]
    assert max(errs) <= tol, errs
    return ref["dW"]


@pytest.mark.parametrize("kind", ["fp32", "bf16", "bf16_pair"])
def test_refreshed_inverses_follow_a_training_loop(kind):
    import torch
    if kind == "fp32":
        p, tol = S.deep_mlp(seed=3, depth=6, n=256, batch=64, reseed_every=3), 1e-4
    elif kind == "bf16":
        p, tol = S.mixed_mlp(seed=3, depth=6, n=256, batch=96, reseed_every=3), 2e-2
    else:
        p, tol = S.sweep_mlp(seed=3, depth=5, n=256, batch=256, reseed_every=2), 2e-2
    net = mwb.net_for(p, backend="tensor", warm_inverse=True)
    params, x, target = mwb.to_device(p)
    ws = net.alloc_workspace("moonwalk")
    theta = [np.array(w, dtype=np.float64) for w in p.params]
    for step in range(4):          # step 0 starts from scratch, the others refresh
        g = grads_against_oracle(net, p, params, x, target, ws, theta, tol)
        # a fine-tuning-sized step of gradient descent (the Frobenius norm of every layer's change
        # stays below the refresh's bound), rounded to the storage type as the caller would keep it
        bound = 2e-4 if p.prec == S.F32 else 2e-3
        lr = min(bound / float(np.sqrt((d * d).sum())) for d in g)
        theta = [S.round_storage(w - lr * d, p.prec) for w, d in zip(theta, g)]
        for dst, w in zip(params, theta):
            dst.copy_(torch.from_numpy(np.ascontiguousarray(w)).to(dst.dtype))


def test_a_step_too_large_for_a_refresh_is_reported_not_absorbed():
    """A change of the weights whose Frobenius norm exceeds the refresh's bound trips the check even
    when it is concentrated in one direction (rank one), where an rms criterion would let it pass."""
    import torch
    p = S.deep_mlp(seed=6, depth=3, n=256, batch=64, reseed_every=0)
    net = mwb.net_for(p, backend="tensor", warm_inverse=True)
    params, x, target = mwb.to_device(p)
    ws = net.alloc_workspace("moonwalk")
    theta = [np.array(w, dtype=np.float64) for w in p.params]
    grads_against_oracle(net, p, params, x, target, ws, theta, 1e-4)
    rng = np.random.default_rng(0)
    u, v = rng.standard_normal(256), rng.standard_normal(256)
    bump = 3e-3 * np.outer(u / np.linalg.norm(u), v / np.linalg.norm(v))      # ||.||_F = ||.||_2 = 3e-3
    params[1].copy_(torch.from_numpy((theta[1] + bump).astype(np.float32)))
    net.input_cotangent(params, x, target, ws)
    code, detail = net.last_device_status(ws)
    assert code == mwb.STATUS_NAMES.index("MW_ERR_NOT_SUBMERSIVE") and detail[0] == 1


def test_a_jump_of_the_weights_is_reported_and_the_next_call_starts_over():
    import torch
    p = S.deep_mlp(seed=4, depth=4, n=128, batch=64, reseed_every=2)
    net = mwb.net_for(p, backend="tensor", warm_inverse=True)
    params, x, target = mwb.to_device(p)
    ws = net.alloc_workspace("moonwalk")
    theta = [np.array(w, dtype=np.float64) for w in p.params]
    grads_against_oracle(net, p, params, x, target, ws, theta, 1e-4)
    # new, unrelated weights: the kept inverses are useless for them
    q = S.deep_mlp(seed=5, depth=4, n=128, batch=64, reseed_every=2)
    for dst, w in zip(params, q.params):
        dst.copy_(torch.from_numpy(np.ascontiguousarray(w)).to(dst.dtype))
    net.input_cotangent(params, x, target, ws)
    code, detail = net.last_device_status(ws)
    assert code == mwb.STATUS_NAMES.index("MW_ERR_NOT_SUBMERSIVE")
    # the report dropped the kept inverses: this call computes them from scratch and is right
    theta = [np.array(w, dtype=np.float64) for w in q.params]
    grads_against_oracle(net, p, params, x, target, ws, theta, 1e-4)
