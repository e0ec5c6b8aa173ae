"""GPU parity of the CUDA-core pipelines and the stand-alone residual-store kernels against the
CPU oracle (same seeded arrays on both sides).  Integer work is compared bit for bit."""
import numpy as np
import pytest

from oracle import moonwalk_oracle as O
from paper_2402_14212_b200 import binding as mwb
from paper_2402_14212_b200 import synth as S
from parity_util import check_problem

pytestmark = pytest.mark.gpu


def torch_cuda():
    import torch
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    return torch


# ---------------------------------------------------------------------------------------
# stand-alone kernels: bit-exact
# ---------------------------------------------------------------------------------------
@pytest.mark.parametrize("rows,cols", [(1, 1), (5, 31), (7, 100), (64, 128), (33, 1024), (300, 2048 + 64)])
@pytest.mark.parametrize("dtype", ["float32", "float64", "bfloat16"])
def test_pack_sign_bits_bit_exact(rows, cols, dtype):
    torch = torch_cuda()
    z = S.random_preacts(rows * 1000 + cols, rows, cols)
    zt = torch.from_numpy(z).to(getattr(torch, dtype)).cuda()
    words = mwb.pack_sign_bits(zt).cpu().numpy().view(np.uint32)
    ref = O.pack_mask(O.sign_mask(zt.double().cpu().numpy()))
    assert np.array_equal(words, ref)


def test_pack_empty_input():
    torch = torch_cuda()
    z = torch.zeros((0, 64), device="cuda")
    assert mwb.pack_sign_bits(z).numel() == 0


@pytest.mark.parametrize("rows,cols", [(1, 5), (9, 70), (128, 256), (513, 2048), (1500, 96)])
def test_relu_fragment_store_bit_exact(rows, cols):
    torch = torch_cuda()
    rng = np.random.default_rng(rows + cols)
    z = S.random_preacts(rows + 7 * cols, rows, cols)
    if rows > 3:
        z[1] = 1.0       # a row with no dead unit
        z[2] = -1.0      # a row that is all dead
    mask = O.sign_mask(z.astype(np.float64))
    h = rng.standard_normal((rows, cols)).astype(np.float32)
    words = mwb.pack_sign_bits(torch.from_numpy(z).cuda())
    ht = torch.from_numpy(h).cuda()
    cnt, off, vals, total = mwb.relu_fragment_compact(ht, words)
    rc, ro, rv = O.relu_fragments(h.astype(np.float64), mask)
    assert np.array_equal(cnt.cpu().numpy().view(np.uint32), rc.astype(np.uint32))
    assert np.array_equal(off.cpu().numpy().view(np.uint32), ro.astype(np.uint32))
    assert int(total.item()) == int(rc.sum())
    got = vals.cpu().numpy()[: int(rc.sum())]
    assert np.array_equal(got, rv.astype(np.float32))
    # restore: live units take g_z, dead units the stored values; g_z zeroed at dead units
    gz = rng.standard_normal((rows, cols)).astype(np.float32)
    hout, gzo = mwb.activation_vijp(torch.from_numpy(gz).cuda(), words, "relu", 0.0, off, vals,
                                    want_gz=True)
    ref = O.relu_restore(gz.astype(np.float64), mask, ro, rv)
    assert np.array_equal(hout.cpu().numpy(), ref.astype(np.float32))
    assert np.array_equal(gzo.cpu().numpy(), np.where(mask, gz, 0.0).astype(np.float32))


@pytest.mark.parametrize("rows,cols", [(3, 40), (256, 1024)])
def test_leaky_vijp_closed_form(rows, cols):
    torch = torch_cuda()
    z = S.random_preacts(11, rows, cols)
    gz = np.random.default_rng(1).standard_normal((rows, cols)).astype(np.float32)
    words = mwb.pack_sign_bits(torch.from_numpy(z).cuda())
    h = mwb.activation_vijp(torch.from_numpy(gz).cuda(), words, "leaky_relu", 0.1).cpu().numpy()
    ref = np.where(z > 0, gz, gz / np.float32(0.1))
    assert np.array_equal(h, ref)


# ---------------------------------------------------------------------------------------
# whole path, fp64 (config 1 and ragged variants): masks bit-exact, gradients to 1e-9
# ---------------------------------------------------------------------------------------
def test_config1_tiny_mlp_fp64():
    # literal Algorithm 1 (no re-seeding): 4 layers stay within 1e-9 in fp64
    check_problem(S.tiny_mlp(seed=0), 1e-9)
    check_problem(S.tiny_mlp(seed=1), 1e-9, resident=False)


def test_fp64_ragged_mixed_activations_with_reseed():
    p = S.dense_chain("ragged", 70, 6, 13, S.F64, S.LOSS_HALF_SSE, [S.ACT_LEAKY, S.ACT_RELU], 0.1,
                      lambda rng, n, l: S.orthogonal(rng, n) + 0.05 * rng.standard_normal((n, n)) / np.sqrt(n),
                      3, 2)
    check_problem(p, 1e-9)


def test_fp64_wide_layer_uses_newton_schulz_inverse():
    p = S.deep_mlp(seed=2, depth=4, n=96, batch=8, reseed_every=2, prec=S.F64)
    check_problem(p, 1e-9)


def test_fp32_cuda_core_path_with_mask_replay():
    p = S.deep_mlp(seed=0, depth=12, n=128, batch=64, reseed_every=4, prec=S.F32)
    check_problem(p, 1e-4, exact_masks=False, tau=1e-4)


def test_small_cnn_fp64():
    p = S.submersive_cnn(seed=0, depth=3, C=8, H=8, W=8, batch=3, gamma=0.05, classes=5,
                         reseed_every=2, conv_vijp_iters=30, prec=S.F64)
    check_problem(p, 1e-9)


def test_small_cnn_fp32_fixed_iterations_match_truncated_oracle():
    p = S.submersive_cnn(seed=1, depth=4, C=16, H=12, W=10, batch=2, gamma=0.05, classes=10,
                         reseed_every=2, conv_vijp_iters=10, prec=S.F32)
    check_problem(p, 1e-4, exact_masks=False, tau=1e-4)


def test_config3_submersive_cnn_full_size():
    # 32 stride-1 3x3 convolutions, 64 channels, 32x32, batch 128, fp32, head + cross-entropy
    p = S.submersive_cnn(seed=0)
    check_problem(p, 1e-4, backend="auto", exact_masks=False, tau=1e-4)


def test_sweep_requires_matching_cotangent_pass():
    torch = torch_cuda()
    p = S.tiny_mlp()
    net = mwb.net_for(p)
    params, x, target = mwb.to_device(p)
    ws = net.alloc_workspace("both")
    g0 = torch.zeros_like(x)
    with pytest.raises(mwb.MwError) as e:
        net.forward_sweep(params, x, g0, ws)
    assert e.value.code == 4
    g0 = net.input_cotangent(params, x, target, ws)
    net.forward_sweep(params, x, g0, ws)
    net.backprop_reference(params, x, target, ws)          # overwrites the stores
    with pytest.raises(mwb.MwError):
        net.forward_sweep(params, x, g0, ws)


def test_singular_layer_is_reported_not_faulted():
    torch = torch_cuda()
    p = S.tiny_mlp()
    p.params[2] = np.zeros_like(p.params[2])
    net = mwb.net_for(p)
    params, x, target = mwb.to_device(p)
    ws = net.alloc_workspace("both")
    net.input_cotangent(params, x, target, ws)
    code, detail = net.last_device_status(ws)
    assert code == 5 and detail[0] == 2


def test_a_device_side_wait_that_cannot_end_runs_out_cleanly():
    """Failure detection: a launch whose product waits for something that never completes gives up
    after its (here 5 ms) bound, reports MW_ERR_TIMEOUT and leaves the GPU usable: an ordinary
    product on the same stream right after it is correct."""
    import torch
    code = mwb.selftest_bounded_wait(limit_ms=5)
    assert code == mwb.STATUS_NAMES.index("MW_ERR_TIMEOUT")
    rng = np.random.default_rng(0)
    A = rng.standard_normal((128, 192)).astype(np.float32)
    B = rng.standard_normal((64, 192)).astype(np.float32)
    D = mwb.gemm_split_bf16(torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda(), False, False, 3)
    ref = A.astype(np.float64) @ B.astype(np.float64).T
    assert np.abs(D.double().cpu().numpy() - ref).max() <= 2e-6 * np.abs(ref).max()
    # and again: counters and tensor memory were left in order
    assert mwb.selftest_bounded_wait(limit_ms=5) == mwb.STATUS_NAMES.index("MW_ERR_TIMEOUT")


def test_general_invertible_weights_exact_path_and_reported_on_the_iterative_one():
    """The dense vijp only needs W invertible (Section 3.1).  The CUDA-core path inverts with pivoted
    Gauss-Jordan and handles a Gaussian (He-scaled) W; the tensor-core path's Newton-Schulz iteration
    starts from (n / ||W||_F^2) W^T, which converges only while the largest squared singular value
    stays below twice the mean one (near-orthogonal weights, the benchmark's recipes): a Gaussian W
    is outside that domain and must be REPORTED (MW_ERR_NOT_SUBMERSIVE), not answered wrongly."""
    import torch
    rng = np.random.default_rng(11)
    p = S.tiny_mlp(seed=11, depth=3, n=64, batch=16, reseed_every=1)
    for l in range(len(p.params)):
        p.params[l] = rng.standard_normal((64, 64)) / 8.0
    out, ref, errs = check_problem(p, 1e-7, backend="simt")
    assert max(errs) <= 1e-7
    q = S.deep_mlp(seed=11, depth=2, n=128, batch=64, reseed_every=1)
    for l in range(len(q.params)):
        q.params[l] = S.round_storage(rng.standard_normal((128, 128)) / np.sqrt(128.0), q.prec)
    net = mwb.net_for(q, backend="tensor")
    params, x, target = mwb.to_device(q)
    ws = net.alloc_workspace("moonwalk")
    net.input_cotangent(params, x, target, ws)
    code, detail = net.last_device_status(ws)
    assert code == mwb.STATUS_NAMES.index("MW_ERR_NOT_SUBMERSIVE")
