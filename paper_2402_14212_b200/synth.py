"""Seeded synthetic inputs for the Moonwalk gradient step.

This module only draws random numbers and describes networks.  It holds none of
the method's arithmetic (no forward pass, no cotangents, no masks): both the
CPU oracle and the CUDA path receive exactly the arrays built here, bit for bit.

Network notation follows the paper (Section 3.1): layer i maps x_{i-1} to
x_i = phi(z_i), z_i = linear_i(x_{i-1}); dense weights are stored
[n_out][n_in] row-major, convolution tensors are channel-last (NHWC) and conv
kernels are w[kh][kw][c_in][c_out] as in Lemma 1.

Generators use numpy's PCG64 `default_rng(seed)` in fp64; every array is then
rounded ONCE to the problem's storage type (fp64 / fp32 / bf16) and the rounded
value is what both sides see (returned as fp64 holding exactly representable
values, plus the storage dtype name).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional

import numpy as np

# layer kinds / activations / losses / precisions (strings on the Python side;
# the C-ABI enums carry the same names)
DENSE, CONV2D, HEAD, CONV1D = "dense", "conv2d", "head", "conv1d"
ACT_NONE, ACT_LEAKY, ACT_RELU = "none", "leaky_relu", "relu"
LOSS_HALF_SSE, LOSS_MSE_MEAN, LOSS_XENT_MEAN = "half_sse", "mse_mean", "xent_mean"
F64, F32, BF16 = "f64", "f32", "bf16_f32acc"


@dataclass
class Layer:
    kind: str
    act: str = ACT_NONE
    slope: float = 0.0
    n_in: int = 0
    n_out: int = 0
    # conv geometry (NHWC input H x W x C_in, output Ho x Wo x C_out)
    H: int = 0
    W: int = 0
    C_in: int = 0
    C_out: int = 0
    k: int = 0
    stride: int = 1
    pad: int = 0
    lu: bool = False    # dense: the parameter array holds the factors of W = L U (L unit lower, U upper)

    def out_hw(self):
        wo = (self.W + 2 * self.pad - self.k) // self.stride + 1
        if self.kind == CONV1D:
            return 1, wo
        ho = (self.H + 2 * self.pad - self.k) // self.stride + 1
        return ho, wo


@dataclass
class Problem:
    name: str
    layers: List[Layer]
    params: List[np.ndarray]          # fp64 arrays holding storage-exact values
    x: np.ndarray                     # [B, n0] or [B, H, W, C]
    target: np.ndarray                # [B, n_L] floats, or int64 labels [B] for xent
    loss: str
    prec: str
    batch: int
    reseed_every: int = 4
    conv_vijp_iters: int = 0
    frag_block: int = 0               # block size of the fragmental checkpoints of 1-D convolutions
    seed: int = 0
    notes: dict = field(default_factory=dict)


# ----------------------------------------------------------------------------
# rounding to the storage type
# ----------------------------------------------------------------------------
def round_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """fp64 -> bf16 bit patterns (uint16), round-to-nearest-even on the fp32 image."""
    f = np.ascontiguousarray(a, dtype=np.float32)
    u = f.view(np.uint32)
    bias = ((u >> 16) & 1) + np.uint32(0x7FFF)
    return ((u + bias) >> 16).astype(np.uint16)


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def round_storage(a: np.ndarray, prec: str) -> np.ndarray:
    """Round an fp64 array once to the storage type of `prec`, return it as fp64."""
    if prec == F64:
        return np.ascontiguousarray(a, dtype=np.float64)
    if prec == F32:
        return a.astype(np.float32).astype(np.float64)
    if prec == BF16:
        return bf16_bits_to_f64(round_to_bf16_bits(a)).reshape(a.shape)
    raise ValueError(prec)


# ----------------------------------------------------------------------------
# weight recipes
# ----------------------------------------------------------------------------
def orthogonal(rng: np.random.Generator, n: int) -> np.ndarray:
    """Q factor of a Gaussian matrix, column signs fixed by sign(diag R)."""
    q, r = np.linalg.qr(rng.standard_normal((n, n)))
    s = np.sign(np.diag(r))
    s[s == 0] = 1.0
    return q * s[None, :]


def dense_chain(name, n, depth, batch, prec, loss, acts, slope, weight_fn, seed,
                reseed_every) -> Problem:
    rng = np.random.default_rng(seed)
    layers, params = [], []
    for l in range(depth):
        act = acts[l % len(acts)]
        layers.append(Layer(DENSE, act, slope if act == ACT_LEAKY else 0.0, n, n))
        params.append(round_storage(weight_fn(rng, n, l), prec))
    x = round_storage(rng.standard_normal((batch, n)), prec)
    t = round_storage(rng.standard_normal((batch, n)),
                      F32 if prec == BF16 else prec)
    return Problem(name, layers, params, x, t, loss, prec, batch,
                   reseed_every=reseed_every, seed=seed)


def tiny_mlp(seed=0, depth=4, n=64, batch=32, reseed_every=0) -> Problem:
    """Config 1: square dense layers, W = I + 0.1*N(0,1)/8, leaky 0.1, fp64, 0.5*||y-t||^2."""
    w = lambda rng, n, l: np.eye(n) + 0.1 * rng.standard_normal((n, n)) / np.sqrt(n)
    return dense_chain("tiny_mlp", n, depth, batch, F64, LOSS_HALF_SSE, [ACT_LEAKY], 0.1, w,
                       seed, reseed_every)


def deep_mlp(seed=0, depth=64, n=1024, batch=256, reseed_every=4, prec=F32) -> Problem:
    """Config 2: W = orthogonal + 0.05*N(0,1)/sqrt(n), leaky 0.1, fp32, MSE."""
    w = lambda rng, n, l: orthogonal(rng, n) + 0.05 * rng.standard_normal((n, n)) / np.sqrt(n)
    return dense_chain("deep_mlp", n, depth, batch, prec, LOSS_MSE_MEAN, [ACT_LEAKY], 0.1, w,
                       seed, reseed_every)


def lu_mlp(seed=0, depth=64, n=1024, batch=256, reseed_every=4, prec=F32) -> Problem:
    """Dense leaky-ReLU MLP whose layers are parameterised by triangular factors (`Layer.lu`):
    the array of layer l holds L below its diagonal (unit diagonal implied) and U on and above it,
    L = I + 0.3*N(0,1)/sqrt(n) strictly below, U = diag(+-(1 + 0.1*u)) + 0.3*N(0,1)/sqrt(n) strictly
    above, u uniform in [-1, 1] (W = L U has singular values in about [0.6, 1.5]).  Sizes of
    config 2."""
    rng = np.random.default_rng(seed)
    layers, params = [], []
    for l in range(depth):
        lo = np.tril(rng.standard_normal((n, n)), -1) * (0.3 / np.sqrt(n))
        up = np.triu(rng.standard_normal((n, n)), 1) * (0.3 / np.sqrt(n))
        d = np.where(rng.random(n) < 0.5, -1.0, 1.0) * (1.0 + 0.1 * (2.0 * rng.random(n) - 1.0))
        layers.append(Layer(DENSE, ACT_LEAKY, 0.1, n, n, lu=True))
        params.append(round_storage(lo + up + np.diag(d), prec))
    x = round_storage(rng.standard_normal((batch, n)), prec)
    t = round_storage(rng.standard_normal((batch, n)), F32 if prec == BF16 else prec)
    return Problem("lu_mlp", layers, params, x, t, LOSS_MSE_MEAN, prec, batch,
                   reseed_every=reseed_every, seed=seed)


def mixed_mlp(seed=0, depth=128, n=2048, batch=512, reseed_every=4, prec=BF16) -> Problem:
    """Config 4: alternating leaky-ReLU / ReLU, W = orthogonal + 0.02*N(0,1)/sqrt(n), bf16."""
    w = lambda rng, n, l: orthogonal(rng, n) + 0.02 * rng.standard_normal((n, n)) / np.sqrt(n)
    return dense_chain("mixed_mlp", n, depth, batch, prec, LOSS_MSE_MEAN,
                       [ACT_LEAKY, ACT_RELU], 0.1, w, seed, reseed_every)


def sweep_mlp(seed=0, depth=32, n=4096, batch=1024, reseed_every=4, prec=BF16,
              pool=0) -> Problem:
    """Config 5: dense leaky-ReLU MLP (same weight recipe as config 4).

    `pool` > 0 draws only `pool` distinct weight matrices and cycles them over
    the depth (layer l uses matrix l % pool): cost and memory depend on shapes
    only, and a QR of 4096^2 per layer would dominate a 512-layer run.
    """
    cache = {}

    def w(rng, n, l):
        if pool and (l % pool) in cache:
            return cache[l % pool]
        m = orthogonal(rng, n) + 0.02 * rng.standard_normal((n, n)) / np.sqrt(n)
        if pool:
            cache[l % pool] = m
        return m

    p = dense_chain("sweep_mlp", n, depth, batch, prec, LOSS_MSE_MEAN, [ACT_LEAKY], 0.1, w,
                    seed, reseed_every)
    p.notes["pool"] = pool
    return p


def submersive_cnn(seed=0, depth=32, C=64, H=32, W=32, batch=128, gamma=0.05, classes=10,
                   reseed_every=4, conv_vijp_iters=8, prec=F32) -> Problem:
    """Config 3: stride-1 3x3 same-size convolutions with a dominant identity centre tap.

    w = delta_centre * I + gamma * N(0, 2/(9*C)) (He scale), leaky 0.1, linear head
    N(0, 1/(H*W*C)) to `classes` logits, cross-entropy with uniform random labels.
    """
    rng = np.random.default_rng(seed)
    layers, params = [], []
    he = np.sqrt(2.0 / (9 * C))
    for l in range(depth):
        w = gamma * he * rng.standard_normal((3, 3, C, C))
        w[1, 1] += np.eye(C)
        layers.append(Layer(CONV2D, ACT_LEAKY, 0.1, H * W * C, H * W * C, H=H, W=W, C_in=C,
                            C_out=C, k=3, stride=1, pad=1))
        params.append(round_storage(w, prec))
    nf = H * W * C
    layers.append(Layer(HEAD, ACT_NONE, 0.0, nf, classes))
    params.append(round_storage(rng.standard_normal((classes, nf)) / np.sqrt(nf), prec))
    x = round_storage(rng.standard_normal((batch, H, W, C)), prec)
    labels = rng.integers(0, classes, size=(batch,), dtype=np.int64)
    return Problem("submersive_cnn", layers, params, x, labels, LOSS_XENT_MEAN, prec, batch,
                   reseed_every=reseed_every, conv_vijp_iters=conv_vijp_iters, seed=seed)


def strided_cnn(seed=0, depth=8, C=128, H=256, W=256, batch=128, gamma=0.5, reseed_every=4,
                prec=F32) -> Problem:
    """The fully submersive CNN of the paper's experiments (Section "Fully Parallel Submersive 2D
    CNN"): `depth` 3x3 convolutions with C channels, stride 2, padding 1 and leaky-ReLU 0.1,
    each halving the resolution, on a batch of H x W x C inputs (the paper: 256 x 256 x 128,
    batch 128, up to 8 layers).

    w = gamma * N(0, 2/(9*C)) (He scale) with the anchor tap w[1, 1] made lower triangular in
    (c, c') with unit diagonal (Lemma 1 (ii), (iii); Algorithm 2 normalises the diagonal to 1).
    Loss: mean squared error of the last feature map against a Gaussian target (the paper pools
    and projects to a scalar; any scalar loss of the output serves).
    """
    rng = np.random.default_rng(seed)
    layers, params = [], []
    he = np.sqrt(2.0 / (9 * C))
    h, wd = H, W
    for l in range(depth):
        w = gamma * he * rng.standard_normal((3, 3, C, C))
        w[1, 1] = np.tril(w[1, 1], -1) + np.eye(C)
        lay = Layer(CONV2D, ACT_LEAKY, 0.1, h * wd * C, 0, H=h, W=wd, C_in=C, C_out=C, k=3,
                    stride=2, pad=1)
        ho, wo = lay.out_hw()
        lay.n_out = ho * wo * C
        layers.append(lay)
        params.append(round_storage(w, prec))
        h, wd = ho, wo
    if batch * H * W * C > (1 << 26):
        # large inputs: draw in fp32 directly (an fp64 copy would not fit comfortably)
        x = rng.standard_normal((batch, H, W, C), dtype=np.float32)
        if prec == BF16:
            x = bf16_bits_to_f64(round_to_bf16_bits(x)).reshape(x.shape).astype(np.float32)
    else:
        x = round_storage(rng.standard_normal((batch, H, W, C)), prec)
    t = round_storage(rng.standard_normal((batch, h, wd, C)), F32 if prec == BF16 else prec)
    return Problem("strided_cnn", layers, params, x, t, LOSS_MSE_MEAN, prec, batch,
                   reseed_every=reseed_every, seed=seed)


def fragmental_cnn1d(seed=0, depth=8, C=256, N=2048, batch=128, block=4, gamma=0.3, reseed_every=4,
                     prec=F32) -> Problem:
    """The 1-D CNN of the paper's fragmental-checkpointing experiment: `depth` convolutions with
    k = 3, stride 1, padding 1 on N x C sequences (the paper: 2048 x 256), leaky-ReLU 0.1, shape
    kept across the layers; the output cotangent of every convolution is checkpointed at the first
    2 positions of each block of `block` positions.

    w[j, c, c'] for a [N, C] layer (H = 1, W = N): w = gamma * N(0, 2/(3*C)) with tap 0 made lower
    triangular in (c, c') with unit diagonal (Section 5.1's assumptions).  Loss: mean squared error
    against a Gaussian target.
    """
    rng = np.random.default_rng(seed)
    layers, params = [], []
    he = np.sqrt(2.0 / (3 * C))
    for l in range(depth):
        w = gamma * he * rng.standard_normal((3, C, C))
        w[0] = np.tril(w[0], -1) + np.eye(C)
        layers.append(Layer(CONV1D, ACT_LEAKY, 0.1, N * C, N * C, H=1, W=N, C_in=C, C_out=C, k=3,
                            stride=1, pad=1))
        params.append(round_storage(w, prec))
    x = round_storage(rng.standard_normal((batch, N, C)), prec)
    t = round_storage(rng.standard_normal((batch, N, C)), F32 if prec == BF16 else prec)
    return Problem("fragmental_cnn1d", layers, params, x, t, LOSS_MSE_MEAN, prec, batch,
                   reseed_every=reseed_every, frag_block=block, seed=seed)


def random_preacts(seed: int, rows: int, cols: int, zero_frac: float = 0.01) -> np.ndarray:
    """fp32 pre-activation-like array with exact zeros, negative zeros and a NaN sprinkled in
    (inputs for the sign-bit pack / fragment compaction unit tests)."""
    rng = np.random.default_rng(seed)
    z = rng.standard_normal((rows, cols)).astype(np.float32)
    if rows * cols:
        k = max(1, int(zero_frac * rows * cols))
        idx = rng.integers(0, rows * cols, size=(3, k))
        flat = z.reshape(-1)
        flat[idx[0]] = 0.0
        flat[idx[1]] = -0.0
        flat[idx[2][:1]] = np.nan
    return z
