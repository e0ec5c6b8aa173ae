"""LU-parameterised dense layers on the GPU against the oracle: the layer's array holds the factors
of W = L U, the inverse comes from block substitution (no iteration), gradients come back for the
factors.  Through the C ABI, like every parity test."""
import numpy as np
import pytest

from paper_2402_14212_b200 import synth as S
from parity_util import check_problem

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("n,depth,batch,K", [(128, 3, 40, 0), (256, 5, 64, 2), (384, 4, 96, 3), (640, 3, 128, 4)])
def test_lu_mlp_small(n, depth, batch, K):
    # one diagonal block, a power of two of them, and counts that leave an odd segment on a level
    p = S.lu_mlp(seed=n, depth=depth, n=n, batch=batch, reseed_every=K)
    out, ref, errs = check_problem(p, 1e-4, backend="tensor", exact_masks=False, tau=1e-4)
    assert len(errs) == depth


def test_lu_mlp_config2_size():
    # the sizes of config 2 (64 layers of width 1024, batch 256, fp32), every layer LU-parameterised
    p = S.lu_mlp(seed=0)
    out, ref, errs = check_problem(p, 1e-4, backend="tensor", exact_masks=False, tau=1e-4)
    assert len(errs) == 64


def test_lu_zero_pivot_is_reported():
    from paper_2402_14212_b200 import binding as mwb
    p = S.lu_mlp(seed=1, depth=2, n=256, batch=32, reseed_every=0)
    p.params[1][200, 200] = 0.0                   # a zero on the diagonal of U: W is singular
    net = mwb.net_for(p, backend="tensor")
    params, x, target = mwb.to_device(p)
    ws = net.alloc_workspace("moonwalk")
    net.input_cotangent(params, x, target, ws)
    code, detail = net.last_device_status(ws)
    assert code == mwb.STATUS_NAMES.index("MW_ERR_NOT_SUBMERSIVE") and detail[0] == 1 and detail[1] == 1


def test_lu_needs_fp32_tensor_backend():
    from paper_2402_14212_b200 import binding as mwb
    layers = [S.Layer(S.DENSE, S.ACT_LEAKY, 0.1, 256, 256, lu=True)]
    with pytest.raises(RuntimeError):
        mwb.Net(layers, 32, S.BF16, S.LOSS_MSE_MEAN)
    with pytest.raises(ValueError):
        mwb.Net(layers + [S.Layer(S.DENSE, S.ACT_LEAKY, 0.1, 256, 256)], 32, S.F32, S.LOSS_MSE_MEAN)
