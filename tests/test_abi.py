"""The C-ABI library loads and exports every entry point the header declares; host-side argument
checks reject bad calls before any GPU work (runs without a GPU)."""
import ctypes as C
import os
import re

import pytest

from paper_2402_14212_b200 import binding as mwb
from paper_2402_14212_b200 import synth as S

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    names = set()
    inc = os.path.join(ROOT, "include")
    for f in os.listdir(inc):
        if f.endswith(".h"):
            text = open(os.path.join(inc, f)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(mw_[a-z0-9_]+)\s*\(", text))
    return sorted(names)


def test_library_exports_every_declared_symbol():
    L = mwb.lib()
    syms = declared_symbols()
    assert len(syms) >= 12
    for s in syms:
        assert hasattr(L, s), f"{s} declared in include/ but not exported"


def test_status_strings():
    L = mwb.lib()
    seen = {L.mw_status_string(i) for i in range(8)}
    assert len(seen) == 8 and b"ok" in seen


def test_net_create_rejects_bad_descriptions():
    with pytest.raises(mwb.MwError) as e:
        mwb.Net([S.Layer(S.DENSE, S.ACT_LEAKY, 0.1, 8, 12)], 4, S.F64, S.LOSS_MSE_MEAN)
    assert e.value.code == 2          # non-square dense layer: unsupported
    with pytest.raises(mwb.MwError) as e:
        mwb.Net([S.Layer(S.HEAD, S.ACT_NONE, 0.0, 8, 3), S.Layer(S.DENSE, S.ACT_LEAKY, 0.1, 3, 3)],
                4, S.F64, S.LOSS_MSE_MEAN)
    assert e.value.code == 2          # head must be last
    with pytest.raises(mwb.MwError) as e:
        mwb.Net([S.Layer(S.DENSE, S.ACT_LEAKY, 0.1, 8, 8), S.Layer(S.DENSE, S.ACT_LEAKY, 0.1, 16, 16)],
                4, S.F64, S.LOSS_MSE_MEAN)
    assert e.value.code == 1          # widths do not chain
    with pytest.raises(mwb.MwError):
        mwb.Net([S.Layer(S.CONV2D, S.ACT_LEAKY, 0.1, H=8, W=8, C_in=4, C_out=4, k=3, stride=2, pad=1)],
                2, S.F32, S.LOSS_MSE_MEAN)
    # a leaky-ReLU of slope 0 (or a non-finite slope) is not submersive: its vijp would divide by zero
    for slope in (0.0, float("nan"), float("inf")):
        with pytest.raises(mwb.MwError) as e:
            mwb.Net([S.Layer(S.DENSE, S.ACT_LEAKY, slope, 8, 8)], 4, S.F64, S.LOSS_MSE_MEAN)
        assert e.value.code == 2, slope


def test_net_create_convolution_families():
    def sconv(H, C=128, k=3, s=2, p=1, act=S.ACT_LEAKY):
        l = S.Layer(S.CONV2D, act, 0.1, H=H, W=H, C_in=C, C_out=C, k=k, stride=s, pad=p)
        ho, wo = l.out_hw()
        l.n_in, l.n_out = H * H * C, ho * wo * C
        return l
    # the paper's submersive CNN: stride 2, padding 1, halving resolution
    net = mwb.Net([sconv(32), sconv(16), sconv(8)], 16, S.F32, S.LOSS_MSE_MEAN)
    mw_b, bp_b, (mw_res, bp_res) = net.workspace_bytes()
    assert mw_b > mw_res > 0 and bp_res > 0
    # its first call may leave g0 out; a dense net's may not (checked before any GPU work)
    L = mwb.lib()
    arr = (C.c_void_p * 3)(1, 1, 1)
    assert L.mw_input_cotangent(net._h, arr, 1, 1, None, None, None, 1 << 30, None) == 3   # reaches the workspace check
    dense = mwb.net_for(S.tiny_mlp())
    arr4 = (C.c_void_p * 4)(1, 1, 1, 1)
    assert L.mw_input_cotangent(dense._h, arr4, 1, 1, None, None, 256, 1 << 30, None) == 1
    for bad in ([sconv(32), sconv(8)],                 # resolutions do not chain
                [sconv(32, C=96)],                     # channels not a multiple of 64
                [sconv(30)],                           # 15 x 15 output: tiles are not boxes
                [sconv(32, k=5)],                      # taps of other pixels reach the positions s*i'
                [sconv(32, act=S.ACT_RELU)]):
        with pytest.raises(mwb.MwError):
            mwb.Net(bad, 16, S.F32, S.LOSS_MSE_MEAN)
    with pytest.raises(mwb.MwError):
        mwb.Net([sconv(32)], 16, S.F64, S.LOSS_MSE_MEAN)          # tensor cores only: fp32 nets
    # 1-D convolutions need a block size for their fragmental checkpoints
    c1 = [S.Layer(S.CONV1D, S.ACT_LEAKY, 0.1, 128 * 64, 128 * 64, H=1, W=128, C_in=64, C_out=64, k=3,
                  stride=1, pad=1) for _ in range(3)]
    with pytest.raises(mwb.MwError):
        mwb.Net(c1, 4, S.F32, S.LOSS_MSE_MEAN)
    with pytest.raises(mwb.MwError):
        mwb.Net(c1, 4, S.F32, S.LOSS_MSE_MEAN, frag_block=3)      # does not divide the length
    n4 = mwb.Net(c1, 4, S.F32, S.LOSS_MSE_MEAN, frag_block=4)
    n16 = mwb.Net(c1, 4, S.F32, S.LOSS_MSE_MEAN, frag_block=16)
    r4, r16 = n4.workspace_bytes()[2][0], n16.workspace_bytes()[2][0]
    frag = lambda blk: 3 * 4 * 4 * 128 * 64 * 2 // blk
    assert r4 - r16 == frag(4) - frag(16)              # fragments: 2 of every `block` positions, fp32
    # the fused update is for fp32 nets on the tensor cores
    assert L.mw_forward_sweep_apply(dense._h, arr4, 1, 1, 0.1, arr4, 256, 1 << 30, None) == 2


def test_nets_can_be_created_and_destroyed_repeatedly():
    # host objects only (descriptions, layouts, tensor-map caches): no device memory is involved
    probs = [S.deep_mlp(depth=4, n=128, batch=64), S.mixed_mlp(depth=4, n=128, batch=64),
             S.strided_cnn(depth=2, C=64, H=16, W=16, batch=16), S.fragmental_cnn1d(depth=2, C=64, N=128, batch=2)]
    sizes = []
    for _ in range(50):
        for p in probs:
            net = mwb.net_for(p, backend="tensor")
            sizes.append(net.workspace_bytes()[0])
            net.close()
            net.close()                      # closing twice is harmless
    assert sizes[:4] == sizes[-4:]


def test_workspace_sizes_and_residual_accounting():
    p = S.deep_mlp(depth=8, n=128, batch=64, reseed_every=4)
    net = mwb.net_for(p, backend="simt")
    mw_b, bp_b, (mw_res, bp_res) = net.workspace_bytes()
    masks = 8 * 64 * 128 // 8
    # Moonwalk keeps sign bits + one cotangent checkpoint (l = 4); backprop keeps 7 activations
    assert mw_res >= masks + 64 * 128 * 4 and mw_res < masks + 2 * 64 * 128 * 4 + 16384
    assert bp_res >= masks + 7 * 64 * 128 * 4
    assert mw_b > mw_res and bp_b > bp_res
    p0 = S.deep_mlp(depth=8, n=128, batch=64, reseed_every=0)
    _, _, (r0, _) = mwb.net_for(p0, backend="simt").workspace_bytes()
    assert r0 < mw_res                 # literal Algorithm 1 keeps only the sign bits


def test_calls_reject_null_and_small_workspace_without_touching_a_gpu():
    p = S.tiny_mlp()
    net = mwb.net_for(p)
    L = mwb.lib()
    arr = (C.c_void_p * 4)(1, 1, 1, 1)
    # null x
    assert L.mw_input_cotangent(net._h, arr, None, 1, 1, None, 256, 1 << 30, None) == 1
    # null workspace / misaligned / too small
    assert L.mw_input_cotangent(net._h, arr, 1, 1, 1, None, None, 1 << 30, None) == 3
    assert L.mw_input_cotangent(net._h, arr, 1, 1, 1, None, 257, 1 << 30, None) == 3
    assert L.mw_input_cotangent(net._h, arr, 1, 1, 1, None, 256, 1024, None) == 3
    # sweep before any cotangent pass
    assert L.mw_forward_sweep(net._h, arr, 1, 1, arr, 256, 1 << 30, None) == 4
    # null entry in params
    arr0 = (C.c_void_p * 4)(1, None, 1, 1)
    assert L.mw_backprop_reference(net._h, arr0, 1, 1, arr, None, 256, 1 << 30, None) == 1
    # stand-alone kernels: negative sizes, empty inputs
    assert L.mw_pack_sign_bits(None, 1, -1, 4, None, None) == 1
    assert L.mw_pack_sign_bits(None, 1, 0, 4, None, None) == 0
    assert L.mw_pack_sign_bits(1, 7, 2, 4, 1, None) == 1
    assert L.mw_activation_vijp(1, 1, 2, 4, 1, 0.0, None, None, 1, None, None) == 1   # slope 0


def test_net_create_lu_parameterised_layers():
    lu = lambda n: S.Layer(S.DENSE, S.ACT_LEAKY, 0.1, n, n, lu=True)
    net = mwb.Net([lu(256), lu(256)], 64, S.F32, S.LOSS_MSE_MEAN, backend="tensor")
    mw_b, bp_b, _ = net.workspace_bytes()
    assert mw_b > bp_b > 0
    for bad in [dict(prec=S.BF16), dict(prec=S.F64), dict(backend="simt"), dict(resident_inverse=False),
                dict(warm_inverse=True)]:
        kw = dict(prec=S.F32, backend="tensor")
        kw.update(bad)
        prec = kw.pop("prec")
        with pytest.raises(mwb.MwError) as e:
            mwb.Net([lu(256)], 64, prec, S.LOSS_MSE_MEAN, **kw)
        assert e.value.code == 2, bad
    with pytest.raises(mwb.MwError):      # widths must be multiples of the 128-wide diagonal blocks
        mwb.Net([lu(192)], 64, S.F32, S.LOSS_MSE_MEAN, backend="tensor")
    with pytest.raises(ValueError):       # all layers or none
        mwb.Net([lu(256), S.Layer(S.DENSE, S.ACT_LEAKY, 0.1, 256, 256)], 64, S.F32, S.LOSS_MSE_MEAN)
