"""mw_gemm_split_bf16_static, the entry point for callers that cannot allocate scratch memory,
against mw_gemm_split_bf16 on the same inputs.

The file name sorts last on purpose: the entry point keeps its scratch in an array built into the
library, shared by all calls, so this test runs after every other test has used the GPU and must
pass there as well as alone in a fresh process.
"""
import numpy as np
import pytest

from paper_2402_14212_b200 import binding as mwb

pytestmark = pytest.mark.gpu

TOL = {1: 2e-2, 2: 2e-4, 3: 2e-6}     # the tolerances of the product's own unit test


def _case(rng, M, N, K, a_mn, b_mn):
    import torch
    A = rng.standard_normal((M, K)).astype(np.float32)
    B = rng.standard_normal((N, K)).astype(np.float32)
    ref = A.astype(np.float64) @ B.astype(np.float64).T
    At = torch.from_numpy(np.ascontiguousarray(A.T if a_mn else A)).cuda()
    Bt = torch.from_numpy(np.ascontiguousarray(B.T if b_mn else B)).cuda()
    return At, Bt, ref


@pytest.mark.parametrize("terms", [1, 2, 3])
def test_static_scratch_product_matches_caller_scratch_product_twice(terms):
    import torch
    assert torch.cuda.is_available()
    rng = np.random.default_rng(40 + terms)
    # two calls in a row; the second is smaller and has other layouts, so it finds the first
    # call's planes still sitting in the shared array
    for (M, N, K, a_mn, b_mn) in [(256, 1024, 1024, False, True), (192, 128, 320, True, False)]:
        At, Bt, ref = _case(rng, M, N, K, a_mn, b_mn)
        want = mwb.gemm_split_bf16(At, Bt, a_mn, b_mn, terms).double().cpu().numpy()
        got = mwb.gemm_split_bf16_static(At, Bt, a_mn, b_mn, terms).double().cpu().numpy()
        scale = np.abs(ref).max()
        assert np.abs(got - want).max() / scale <= TOL[terms]
        assert np.abs(got - ref).max() / scale <= TOL[terms]


def test_static_scratch_rejects_sizes_beyond_its_array():
    import torch
    assert torch.cuda.is_available()
    M = N = K = 2048                      # 3 terms need 256 + 6 * (M*K + N*K) bytes = 48 MiB
    assert 6 * (M * K + N * K) > mwb.GEMM_STATIC_SCRATCH_BYTES
    A = torch.zeros((M, K), device="cuda")
    B = torch.zeros((N, K), device="cuda")
    with pytest.raises(mwb.MwError) as e:
        mwb.gemm_split_bf16_static(A, B, False, False, 3)
    assert e.value.code == 3              # MW_ERR_WORKSPACE
