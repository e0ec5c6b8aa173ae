"""Tensor-core product (tcgen05 + TMA) against its plain definition: D = A B in fp64 (numpy matmul),
for every operand layout the Moonwalk steps use and every split depth."""
import numpy as np
import pytest

from paper_2402_14212_b200 import binding as mwb

pytestmark = pytest.mark.gpu

TOL = {1: 2e-2, 2: 2e-4, 3: 2e-6}     # normwise, against bf16 eps 2^-9 per term


@pytest.mark.parametrize("a_mn,b_mn", [(False, False), (False, True), (True, True), (True, False)])
@pytest.mark.parametrize("terms", [1, 2, 3])
@pytest.mark.parametrize("M,N,K", [(128, 64, 64), (64, 128, 128), (192, 192, 320), (256, 1024, 1024),
                                   (1024, 1024, 256), (2048, 2048, 512)])
def test_split_bf16_product(a_mn, b_mn, terms, M, N, K):
    import torch
    assert torch.cuda.is_available()
    rng = np.random.default_rng(M + 3 * N + 7 * K + terms)
    A = rng.standard_normal((M, K)).astype(np.float32)
    B = rng.standard_normal((N, K)).astype(np.float32)          # D = A B^T
    # a few structured entries catch transposition / offset mistakes that random data could hide
    A[0, :] = 0.0; A[0, 0] = 1.0
    B[:, 0] = np.arange(N, dtype=np.float32) / N
    ref = A.astype(np.float64) @ B.astype(np.float64).T
    At = torch.from_numpy(np.ascontiguousarray(A.T if a_mn else A)).cuda()
    Bt = torch.from_numpy(np.ascontiguousarray(B.T if b_mn else B)).cuda()
    D = mwb.gemm_split_bf16(At, Bt, a_mn, b_mn, terms).double().cpu().numpy()
    err = np.abs(D - ref).max() / np.abs(ref).max()
    assert err <= TOL[terms], err
    assert np.abs(D[0] - ref[0]).max() <= TOL[terms] * 2.0      # the unit row selects column 0 of B


@pytest.fixture
def pair_mode():
    """Runs a test in one form of the product kernel and restores the setting afterwards."""
    state = {}

    def choose(enable):
        state.setdefault("old", mwb.set_pair_mode(enable))

    yield choose
    if "old" in state:
        mwb.set_pair_mode(state["old"])


@pytest.mark.parametrize("pair", [False, True])
@pytest.mark.parametrize("a_mn,b_mn", [(False, False), (False, True), (True, True), (True, False)])
@pytest.mark.parametrize("terms", [1, 2])
@pytest.mark.parametrize("M,N,K", [(256, 128, 64), (512, 384, 192), (256, 4096, 512), (1024, 2048, 1024)])
def test_split_bf16_product_both_kernel_forms(pair_mode, pair, a_mn, b_mn, terms, M, N, K):
    """Sizes that qualify for the CTA-pair form (M % 256 == 0, N % 128 == 0, at most two terms), once
    with the pair form switched off and once with it on: both against the fp64 product."""
    import torch
    pair_mode(pair)
    rng = np.random.default_rng(11 * M + 3 * N + 7 * K + terms)
    A = rng.standard_normal((M, K)).astype(np.float32)
    B = rng.standard_normal((N, K)).astype(np.float32)
    A[M // 2 + 1, :] = 0.0; A[M // 2 + 1, K - 1] = 1.0          # a unit row in the second half of a 256-row tile
    B[:, K - 1] = np.arange(N, dtype=np.float32) / N
    ref = A.astype(np.float64) @ B.astype(np.float64).T
    At = torch.from_numpy(np.ascontiguousarray(A.T if a_mn else A)).cuda()
    Bt = torch.from_numpy(np.ascontiguousarray(B.T if b_mn else B)).cuda()
    D = mwb.gemm_split_bf16(At, Bt, a_mn, b_mn, terms).double().cpu().numpy()
    err = np.abs(D - ref).max() / np.abs(ref).max()
    assert err <= TOL[terms], err
    r = M // 2 + 1
    assert np.abs(D[r] - ref[r]).max() <= TOL[terms] * 2.0
