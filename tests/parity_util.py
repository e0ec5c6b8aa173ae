"""Helpers shared by the GPU parity tests: run the CUDA path through the C ABI, run the oracle on
the same arrays, compare."""
import numpy as np

from oracle import moonwalk_oracle as O
from paper_2402_14212_b200 import binding as mwb


def run_gpu(problem, backend="auto", resident_inverse=True, inverse_iters=0, backprop=True,
            want_masks=True):
    import torch
    net = mwb.net_for(problem, backend=backend, resident_inverse=resident_inverse,
                      inverse_iters=inverse_iters)
    params, x, target = mwb.to_device(problem)
    ws = net.alloc_workspace("both")
    loss = torch.zeros(1, dtype=torch.float64, device="cuda")
    g0 = net.input_cotangent(params, x, target, ws, loss_out=loss)
    dW = net.forward_sweep(params, x, g0, ws)
    code, detail = net.last_device_status(ws)
    out = dict(net=net, status=code, detail=detail, loss=float(loss.item()),
               g0=g0.double().cpu().numpy(), dW=[d.double().cpu().numpy() for d in dW])
    if want_masks:
        out["masks"] = [net.export_masks(ws, l) for l in range(len(problem.layers))]
    if backprop:
        loss2 = torch.zeros(1, dtype=torch.float64, device="cuda")
        dWb = net.backprop_reference(params, x, target, ws, loss_out=loss2)
        code2, _ = net.last_device_status(ws)
        out.update(bp_status=code2, bp_loss=float(loss2.item()),
                   bp_dW=[d.double().cpu().numpy() for d in dWb])
    return out


def oracle_masks_from_words(problem, words_list):
    """GPU-exported words -> boolean masks shaped like each layer's z (for mask replay)."""
    ms = []
    for layer, words in zip(problem.layers, words_list):
        if layer.kind == "conv1d":
            m = O.unpack_mask(words, layer.C_out).reshape(problem.batch, layer.out_hw()[1], layer.C_out)
        elif layer.kind == "conv2d":
            ho, wo = layer.out_hw()
            m = O.unpack_mask(words, layer.C_out).reshape(problem.batch, ho, wo, layer.C_out)
        else:
            m = O.unpack_mask(words, layer.n_out)
        ms.append(m)
    return ms


def oracle_reference(problem, masks=None):
    return O.backprop(problem.layers, problem.params, problem.x, problem.target, problem.loss,
                      masks=masks)


def mask_disagreement(problem, gpu_words, ref, per_layer=None):
    """Sign bits of the GPU against the signs of the oracle's pre-activations `ref["z"]`.  Returns
    the Hamming distance and, per layer, the largest |z| (relative to the row rms) at a disagreeing
    element (0 where the layer agrees everywhere); `per_layer` (a list) receives (disagreeing bits,
    bits) of every layer."""
    flips, worst = 0, []
    for l, (layer, words) in enumerate(zip(problem.layers, gpu_words)):
        w = 0.0
        if layer.act != "none":
            z = ref["z"][l].reshape(words.shape[0], -1)
            mg = O.unpack_mask(words, z.shape[1])
            d = mg != O.sign_mask(z)
            if per_layer is not None:
                per_layer.append((int(d.sum()), int(d.size)))
            if d.any():
                flips += int(d.sum())
                rms = np.sqrt((z * z).mean(axis=1, keepdims=True))
                w = float((np.abs(z) / rms)[d].max())
        elif per_layer is not None:
            per_layer.append((0, 1))
        worst.append(w)
    return flips, worst


def grad_errors(gpu_dW, ref_dW):
    return [O.normwise_error(a.reshape(b.shape), b) for a, b in zip(gpu_dW, ref_dW)]


def check_problem(p, tol, backend="simt", inverse_iters=0, resident=True, exact_masks=True, tau=0.0):
    """Whole path against the oracle.  exact_masks: the sign bits must equal the oracle's own.
    Otherwise (fp32 / bf16 arithmetic) the oracle is evaluated on the GPU's exported bits (mask
    replay) and a bit may contradict the sign of the oracle's pre-activation only where that
    pre-activation is within rounding of zero: |z| <= tau * sqrt(l + 1) * rms(z_row) at layer l
    (the per-layer rounding errors of the chain add up like a random walk along the depth), and
    only a fraction 0.1 * tau * sqrt(l + 1) of a layer's bits may do so (two bits always may).
    tests/test_sign_bit_law.py pins both laws on the CPU."""
    out = run_gpu(p, backend=backend, resident_inverse=resident, inverse_iters=inverse_iters)
    assert out["status"] == 0 and out["bp_status"] == 0
    if exact_masks:
        ref = oracle_reference(p)
        flips, worst = mask_disagreement(p, out["masks"], ref)
        assert flips == 0
    else:
        ref = oracle_reference(p, oracle_masks_from_words(p, out["masks"]))
        counts = []
        flips, worst = mask_disagreement(p, out["masks"], ref, per_layer=counts)
        for l, w in enumerate(worst):
            assert w <= tau * np.sqrt(l + 1.0), (l, w, flips)
            bad, bits = counts[l]
            assert bad <= max(2.0, 0.1 * tau * np.sqrt(l + 1.0) * bits), (l, bad, bits)
    errs = grad_errors(out["dW"], ref["dW"])
    errs_bp = grad_errors(out["bp_dW"], ref["dW"])
    assert O.normwise_error(out["g0"].reshape(ref["g0"].shape), ref["g0"]) <= tol
    assert max(errs) <= tol, errs
    assert max(errs_bp) <= tol, errs_bp
    assert abs(out["loss"] - ref["loss"]) <= max(tol, 1e-12) * max(1.0, abs(ref["loss"]))
    assert abs(out["bp_loss"] - ref["loss"]) <= max(tol, 1e-12) * max(1.0, abs(ref["loss"]))
    out["flips"], out["worst"] = flips, worst
    return out, ref, errs
