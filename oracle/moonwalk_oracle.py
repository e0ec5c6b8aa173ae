"""CPU oracle for the Moonwalk gradient step (fp64, numpy).  TEST INFRASTRUCTURE ONLY.

This file is the slow, plain statement of what the CUDA library must compute.
Only the tests, the smoke check and the benchmark's CPU-baseline leg may import
it; the product path never does.  It shares no code with the CUDA path.

What it states, each function citing the passage of the paper it follows:

* the network of Section 3.1 (sequential layers x_i = f_i(x_{i-1}; theta_i), scalar loss J),
* the three operators of Section 3.1 (jvp is not needed; vjp and vijp are),
* the convolution of Lemma 1 and its reverse pass TransposeConv (Eq. "conv-vjp"),
* plain reverse-mode differentiation ("Backprop", Section "Complexity Analysis", item 1),
  which is the ground truth because the Moonwalk identity (Eq. "ifp-main") is exact,
* Algorithm 1 (Moonwalk) in its mixed-mode form (Section 4.1, Phases I-III) with the
  sign-bit residual store (Section "Residual Impact"), cotangent checkpointing in
  Phase II (Section 4.1) and fragmental checkpointing for ReLU (Section 5.1),
* the bit-packed mask store and the fragment store in their canonical form.

Readings where the paper is silent (the same ones the CUDA path takes):
no bias; "positive" means z > 0 strictly (0, -0.0 and NaN take the negative
branch); losses: half_sse = 0.5*sum (y-t)^2, mse_mean = mean over all B*n
entries, xent_mean = mean over the batch of -log softmax at the label; dense
vijp is the solution g of g W = h (square invertible W); a ReLU fragment holds
the output cotangent at every dead unit, row by row in increasing column
order; the stride-1 same-size convolution's vijp is the unique solution of
Eq. "conv-vjp" for h', computed with the paper's relation
w_centre h'_{i'} = h_{i'} - TransposeConv(h', w~)_{i'} used as a fixed-point
iteration with the whole C x C centre tap as the pivot block; a convolution
that meets Lemma 1 (stride above padding, triangular anchor tap) takes the
lemma's elimination itself, which is exact; a dense layer may be parameterised
by the triangular factors of its weight (W = L U, one array holding both), the
paper's constrained-layer idea carried to dense layers: its vijp is two
substitutions, its parameter cotangent the chain rule through the product.

Pinned by tests/test_oracle_*.py: finite differences, Moonwalk == Backprop,
vjp(vijp(h)) == h, closed-form leaky-ReLU inverse, explicit-Jacobian brute
force for the convolution, packbits cross-check, paper's residual-size ratios.
Constants chosen by measurement rather than by the paper (re-seed interval K,
conv noise scale gamma, mask tolerance tau) are "parity unpinned" by the paper.
"""
from __future__ import annotations

import numpy as np

DENSE, CONV2D, HEAD, CONV1D = "dense", "conv2d", "head", "conv1d"
ACT_NONE, ACT_LEAKY, ACT_RELU = "none", "leaky_relu", "relu"


# ----------------------------------------------------------------------------
# activations (Section "Residual Impact": only the sign of z is needed for the vjp)
# ----------------------------------------------------------------------------
def sign_mask(z):
    """mask bit = (z > 0); zero, negative zero and NaN give False."""
    return z > 0


def act_slope(layer):
    if layer.act == ACT_LEAKY:
        return float(layer.slope)
    if layer.act == ACT_RELU:
        return 0.0
    return 1.0


def act_forward(z, layer, mask):
    """phi(z) with the branch chosen by `mask`: z where set, slope*z elsewhere."""
    if layer.act == ACT_NONE:
        return z
    return np.where(mask, z, act_slope(layer) * z)


def act_derivative(layer, mask):
    if layer.act == ACT_NONE:
        return np.ones(mask.shape)
    return np.where(mask, 1.0, act_slope(layer))


# ----------------------------------------------------------------------------
# linear maps: dense, and the convolution of Lemma 1
# ----------------------------------------------------------------------------
def conv_forward(x, w, stride, pad):
    """Lemma 1: x'[i', c'] = sum_{j, c} w[j, c, c'] * x[s i' + j - p, c], zero outside."""
    B, H, W, C = x.shape
    k = w.shape[0]
    Ho = (H + 2 * pad - k) // stride + 1
    Wo = (W + 2 * pad - k) // stride + 1
    xp = np.zeros((B, H + 2 * pad, W + 2 * pad, C))
    xp[:, pad:pad + H, pad:pad + W, :] = x
    out = np.zeros((B, Ho, Wo, w.shape[3]))
    for j0 in range(k):
        for j1 in range(k):
            patch = xp[:, j0:j0 + stride * (Ho - 1) + 1:stride,
                       j1:j1 + stride * (Wo - 1) + 1:stride, :]
            out += patch @ w[j0, j1]
    return out


def transpose_conv(hp, w, n_hw, stride, pad):
    """Eq. "conv-vjp": h[i, c] = sum_{j, c'} w[j, c, c'] * hbar'[i + p - j, c'],
    hbar' being h' dilated by the stride (hbar'[s i'] = h'[i'], zero elsewhere)."""
    B, Ho, Wo, Cp = hp.shape
    H, W = n_hw
    k = w.shape[0]
    # dilated cotangent, embedded with a margin so that every index i + p - j is valid
    m = k
    hb = np.zeros((B, H + 2 * m, W + 2 * m, Cp))
    hb[:, m:m + stride * (Ho - 1) + 1:stride, m:m + stride * (Wo - 1) + 1:stride, :] = hp
    h = np.zeros((B, H, W, w.shape[2]))
    for j0 in range(k):
        for j1 in range(k):
            o0 = m + pad - j0
            o1 = m + pad - j1
            h += hb[:, o0:o0 + H, o1:o1 + W, :] @ w[j0, j1].T
    return h


def conv_weight_vjp(x, gz, k, stride, pad):
    """vjp(f, theta, .) of the Lemma 1 convolution:
    dw[j, c, c'] = sum_{b, i'} x[b, s i' + j - p, c] * gz[b, i', c']."""
    B, H, W, C = x.shape
    _, Ho, Wo, Cp = gz.shape
    xp = np.zeros((B, H + 2 * pad, W + 2 * pad, C))
    xp[:, pad:pad + H, pad:pad + W, :] = x
    dw = np.zeros((k, k, C, Cp))
    g2 = gz.reshape(-1, Cp)
    for j0 in range(k):
        for j1 in range(k):
            patch = xp[:, j0:j0 + stride * (Ho - 1) + 1:stride,
                       j1:j1 + stride * (Wo - 1) + 1:stride, :]
            dw[j0, j1] = patch.reshape(-1, C).T @ g2
    return dw


def conv1d_forward(x, w, stride, pad):
    """Lemma 1 with one spatial dimension: x'[i', c'] = sum_{j, c} w[j, c, c'] x[s i' + j - p, c].
    x: [B, N, C], w: [k, C, C']."""
    B, N, C = x.shape
    k = w.shape[0]
    No = (N + 2 * pad - k) // stride + 1
    xp = np.zeros((B, N + 2 * pad, C))
    xp[:, pad:pad + N, :] = x
    out = np.zeros((B, No, w.shape[2]))
    for j in range(k):
        out += xp[:, j:j + stride * (No - 1) + 1:stride, :] @ w[j]
    return out


def transpose_conv1d(hp, w, n, stride, pad):
    """Eq. "conv-vjp" with one spatial dimension: h[i, c] = sum_{j, c'} w[j, c, c'] hbar'[i + p - j, c']."""
    B, No, Cp = hp.shape
    k = w.shape[0]
    m = k
    hb = np.zeros((B, n + 2 * m, Cp))
    hb[:, m:m + stride * (No - 1) + 1:stride, :] = hp
    h = np.zeros((B, n, w.shape[1]))
    for j in range(k):
        o = m + pad - j
        h += hb[:, o:o + n, :] @ w[j].T
    return h


def conv1d_weight_vjp(x, gz, k, stride, pad):
    """dw[j, c, c'] = sum_{b, i'} x[b, s i' + j - p, c] gz[b, i', c']."""
    B, N, C = x.shape
    _, No, Cp = gz.shape
    xp = np.zeros((B, N + 2 * pad, C))
    xp[:, pad:pad + N, :] = x
    dw = np.zeros((k, C, Cp))
    g2 = gz.reshape(-1, Cp)
    for j in range(k):
        dw[j] = xp[:, j:j + stride * (No - 1) + 1:stride, :].reshape(-1, C).T @ g2
    return dw


def is_lu(layer):
    """A dense layer whose parameter array holds the factors of its weight (see lu_factors)."""
    return layer.kind == DENSE and bool(getattr(layer, "lu", False))


def lu_factors(p):
    """LU-parameterised dense layer: the paper constrains its convolutions so that the vijp is
    cheap by construction (Section "Constrained Convolutions"); the same idea for a square dense
    layer is to learn the triangular factors of W instead of W.  One n x n array p holds both:
    L = I + strictly lower part of p (unit diagonal, not a parameter), U = upper part of p with
    its diagonal.  The layer's weight is W = L U, invertible whenever diag(U) has no zero."""
    p = np.asarray(p, dtype=np.float64)
    return np.tril(p, -1) + np.eye(p.shape[0]), np.triu(p)


def lu_weight(p):
    L, U = lu_factors(p)
    return L @ U


def dense_weight(layer, w):
    return lu_weight(w) if is_lu(layer) else w


def linear_forward(layer, w, x):
    if layer.kind == CONV1D:
        return conv1d_forward(x, w, layer.stride, layer.pad)
    if layer.kind == CONV2D:
        return conv_forward(x, w, layer.stride, layer.pad)
    x2 = x.reshape(x.shape[0], -1)
    return x2 @ dense_weight(layer, w).T


def linear_vjp_input(layer, w, g, in_shape):
    """vjp(f, x, g) of the linear part (Section 3.1)."""
    if layer.kind == CONV1D:
        return transpose_conv1d(g, w, layer.W, layer.stride, layer.pad)
    if layer.kind == CONV2D:
        return transpose_conv(g, w, (layer.H, layer.W), layer.stride, layer.pad)
    return (g @ dense_weight(layer, w)).reshape(in_shape)


def linear_vjp_param(layer, x, g, w=None):
    """vjp(f, theta, g) of the linear part: Eq. "g_i".  An LU-parameterised layer needs its
    parameters `w`: with G = g^T x the cotangent of W = L U, the chain rule through the product
    gives dJ/dL = G U^T on the strictly lower entries and dJ/dU = L^T G on the upper ones."""
    if layer.kind == CONV1D:
        return conv1d_weight_vjp(x, g, layer.k, layer.stride, layer.pad)
    if layer.kind == CONV2D:
        return conv_weight_vjp(x, g, layer.k, layer.stride, layer.pad)
    G = g.T @ x.reshape(x.shape[0], -1)
    if is_lu(layer):
        L, U = lu_factors(w)
        return np.tril(G @ U.T, -1) + np.triu(L.T @ G)
    return G


# ----------------------------------------------------------------------------
# vijp (Section 3.1: v (df/dx)^+, any right inverse; unique here)
# ----------------------------------------------------------------------------
def vijp_dense(w, h):
    """The g with g W = h, by an LU solve with partial pivoting (never forms W^-1)."""
    return np.linalg.solve(w.T, h.reshape(h.shape[0], -1).T).T


def vijp_dense_lu(p, h):
    """The g with g L U = h for the factors held in p, by two substitutions and no inverse:
    first y U = h column by column from the left (U upper triangular), then g L = y column by
    column from the right (L unit lower triangular)."""
    L, U = lu_factors(p)
    h2 = h.reshape(h.shape[0], -1)
    n = h2.shape[1]
    y = np.zeros_like(h2, dtype=np.float64)
    for j in range(n):
        y[:, j] = (h2[:, j] - y[:, :j] @ U[:j, j]) / U[j, j]
    g = np.zeros_like(y)
    for j in range(n - 1, -1, -1):
        g[:, j] = y[:, j] - g[:, j + 1:] @ L[j + 1:, j]
    return g


def vijp_conv_fixed_point(layer, w, h, tol=1e-14, max_iters=400, iters=None, trace=None):
    """Stride-1, same-size convolution with an invertible centre tap W_c = w[p, p].

    Solves h = TransposeConv(g, w) for g with the paper's elimination relation
    (Proof outline of Lemma 1) read as an iteration:
        g <- (h - TransposeConv(g, w~)) W_c^{-T},   w~ = w with the centre tap zeroed,
    started from g = h W_c^{-T}.  With `iters` given, exactly that many updates
    are applied (what a fixed-iteration implementation computes); otherwise it
    runs until the relative residual falls below `tol`.
    """
    assert layer.stride == 1 and 2 * layer.pad + 1 == layer.k
    p = layer.pad
    wc = w[p, p]                       # [c_in][c_out]:  h[i] has the term  g[i] @ wc.T
    wt = w.copy()
    wt[p, p] = 0.0
    solve_c = lambda r: np.linalg.solve(wc, r.reshape(-1, r.shape[-1]).T).T.reshape(r.shape)
    g = solve_c(h)
    hn = np.sqrt((h * h).sum())
    n = 0
    while True:
        if iters is not None and n >= iters:
            break
        if iters is None:
            res = transpose_conv(g, w, (layer.H, layer.W), 1, p) - h
            r = np.sqrt((res * res).sum()) / max(hn, 1e-300)
            if trace is not None:
                trace.append(r)
            if r <= tol or n >= max_iters:
                break
        g = solve_c(h - transpose_conv(g, wt, (layer.H, layer.W), 1, p))
        n += 1
    return g


def submersive_conditions(layer, w):
    """Lemma 1, conditions (i)-(iii), for one spatial size n x n' per dimension; returns the
    list of violated conditions (empty = submersive by the lemma)."""
    k, s, p = layer.k, layer.stride, layer.pad
    bad = []
    for n in (layer.H, layer.W):
        n_out = (n + 2 * p - k) // s + 1
        if not (k > p and s > p and n > s * (n_out - 1)):
            bad.append("(i) spatial bounds")
            break
    m, mp = w.shape[2], w.shape[3]
    anchor = w[p, p] if k > p else np.zeros((m, mp))
    if mp > m or np.any(np.triu(anchor, 1) != 0.0):          # entries with c < c'
        bad.append("(ii) channel-wise triangularity")
    if np.any(np.diagonal(anchor)[:mp] == 0.0):
        bad.append("(iii) diagonal support")
    return bad


def vijp_conv_submersive(layer, w, h):
    """vijp of a convolution that meets Lemma 1, by the elimination of its proof: in
    lexicographic order of (i', c'),
        w[p, c', c'] h'[i', c'] = h[s i', c'] - TransposeConv(h', w~)[s i', c'],
    w~ = w with the diagonal of the anchor tap w[p] zeroed; every h' entry that appears on the
    right with a non-zero coefficient has a smaller index and is already known.  Terms from
    other pixels (taps j with p - j a non-zero multiple of s) are taken first, then the
    channels of pixel i' itself are eliminated one after the other through the triangular
    anchor tap (Algorithm 2).  h: [B, H, W, m] -> h': [B, H', W', m']."""
    bad = submersive_conditions(layer, w)
    if bad:
        raise ValueError("not submersive by Lemma 1: " + ", ".join(bad))
    k, s, p = layer.k, layer.stride, layer.pad
    B = h.shape[0]
    Ho, Wo = layer.out_hw()
    mp = w.shape[3]
    hp = np.zeros((B, Ho, Wo, mp))
    for i0 in range(Ho):
        for i1 in range(Wo):
            r = h[:, s * i0, s * i1, :mp].copy()
            for j0 in range(k):
                for j1 in range(k):
                    d0, d1 = p - j0, p - j1
                    if (d0 == 0 and d1 == 0) or d0 % s != 0 or d1 % s != 0:
                        continue                      # anchor tap, or a zero of the dilated h'
                    q0, q1 = i0 + d0 // s, i1 + d1 // s
                    if 0 <= q0 < Ho and 0 <= q1 < Wo:
                        r -= hp[:, q0, q1, :] @ w[j0, j1, :mp, :].T
            for c in range(mp):
                v = r[:, c] - hp[:, i0, i1, :c] @ w[p, p, c, :c]
                hp[:, i0, i1, c] = v / w[p, p, c, c]
    return hp


def conv1d_fragments(hp, k, block):
    """Fragmental checkpoint of an output cotangent h' [B, N, C'] (Section 5.1): the first k - 1
    positions of every block of `block` positions; [B, N / block, k - 1, C']."""
    B, N, Cp = hp.shape
    assert N % block == 0 and block >= k - 1
    return hp.reshape(B, N // block, block, Cp)[:, :, :k - 1, :].copy()


def vijp_conv1d_fragmental(layer, w, h, frags, block):
    """Stride-1 convolution with padding 1 (Section 5.1, Appendix "Fragmental Gradient
    Checkpointing"): the reverse pass reads h[i] = sum_j w[j] h'[i + 1 - j], whose newest unknown
    is h'[i + 1] with coefficient w[0], lower triangular in (c, c') with a non-zero diagonal (the
    paper normalises it to 1).  Given the first k - 1 positions of a block, the rest follow one
    position after the other,
        w[0] h'[i + 1] = h[i] - sum_{j >= 1} w[j] h'[i + 1 - j],
    channel by channel through the triangle; blocks are independent of one another.
    h: [B, N, C], frags: [B, N / block, k - 1, C'] -> h': [B, N, C']."""
    k = layer.k
    assert layer.stride == 1 and layer.pad == 1
    w0 = w[0]
    if np.any(np.triu(w0, 1) != 0.0) or np.any(np.diagonal(w0) == 0.0):
        raise ValueError("tap 0 must be lower triangular in (c, c') with a non-zero diagonal")
    B, N, C = h.shape
    Cp = w.shape[2]
    nb = N // block
    hp = np.zeros((B, N, Cp))
    for b in range(nb):
        base = b * block
        hp[:, base:base + k - 1, :] = frags[:, b]
        for t in range(k - 1, block):
            i = base + t - 1                       # the equation of h[i] yields h'[i + 1]
            r = h[:, i, :Cp].copy()
            for j in range(1, k):
                q = i + 1 - j
                if q >= 0:
                    r -= hp[:, q, :] @ w[j, :Cp, :].T
            for c in range(Cp):
                v = r[:, c] - hp[:, i + 1, :c] @ w0[c, :c]
                hp[:, i + 1, c] = v / w0[c, c]
    return hp


def vijp_linear(layer, w, h, conv_iters=None):
    if layer.kind == CONV1D:
        raise ValueError("a stride-1 1-D convolution needs its fragments: vijp_conv1d_fragmental")
    if layer.kind == CONV2D:
        if layer.stride > layer.pad:
            return vijp_conv_submersive(layer, w, h)
        return vijp_conv_fixed_point(layer, w, h, iters=conv_iters)
    if is_lu(layer):
        return vijp_dense_lu(w, h)
    return vijp_dense(w, h)


def vijp_leaky(layer, mask, g):
    """Closed form: the leaky-ReLU Jacobian is diag(1 or slope), so divide by it."""
    return np.where(mask, g, g / float(layer.slope))


# ----------------------------------------------------------------------------
# loss J and its cotangent h_L = dJ/dx_L (Section 3.1: scalar loss of the output)
# ----------------------------------------------------------------------------
def loss_and_cotangent(y, target, kind):
    B = y.shape[0]
    if kind == "half_sse":
        d = y - target
        return 0.5 * float((d * d).sum()), d
    if kind == "mse_mean":
        d = y - target
        return float((d * d).mean()), 2.0 * d / d.size
    if kind == "xent_mean":
        zmax = y.max(axis=1, keepdims=True)
        e = np.exp(y - zmax)
        s = e.sum(axis=1, keepdims=True)
        logp = (y - zmax) - np.log(s)
        J = -float(logp[np.arange(B), target].mean())
        p = e / s
        p[np.arange(B), target] -= 1.0
        return J, p / B
    raise ValueError(kind)


# ----------------------------------------------------------------------------
# Backprop: the ground truth (store every residual, vjp both ways)
# ----------------------------------------------------------------------------
def forward(layers, params, x0, masks=None):
    """x_i = f_i(x_{i-1}).  With `masks` given, those bits choose the activation branch
    (mask replay); otherwise bits are (z > 0).  Returns activations, masks, pre-activations."""
    xs, ms, zs = [x0], [], []
    for l, (layer, w) in enumerate(zip(layers, params)):
        z = linear_forward(layer, w, xs[-1])
        m = sign_mask(z) if masks is None or masks[l] is None else masks[l].reshape(z.shape)
        if layer.act == ACT_NONE:
            m = np.ones(z.shape, dtype=bool)
        ms.append(m)
        zs.append(z)
        xs.append(act_forward(z, layer, m))
    return xs, ms, zs


def backprop(layers, params, x0, target, loss, masks=None):
    """Reverse mode, all residuals kept: g_z = h_l * phi'(z_l), dW_l = vjp(f_l, theta_l, .),
    h_{l-1} = vjp(f_l, x_{l-1}, .).  Returns dict(loss, dW, h (list, h[l] = dJ/dx_l), g0, masks)."""
    xs, ms, zs = forward(layers, params, x0, masks)
    J, hL = loss_and_cotangent(xs[-1], target, loss)
    L = len(layers)
    hs = [None] * (L + 1)
    hs[L] = hL
    dW = [None] * L
    for l in range(L - 1, -1, -1):
        gz = hs[l + 1] * act_derivative(layers[l], ms[l])
        dW[l] = linear_vjp_param(layers[l], xs[l], gz, params[l])
        hs[l] = linear_vjp_input(layers[l], params[l], gz, xs[l].shape)
    return dict(loss=J, dW=dW, h=hs, g0=hs[0], masks=ms, x=xs, z=zs)


# ----------------------------------------------------------------------------
# residual stores in canonical form
# ----------------------------------------------------------------------------
def pack_mask(mask2d):
    """Rows of bits -> uint32 words [rows][ceil(cols/32)]; bit (j & 31) of word (j >> 5) is
    element j (least significant bit first); padding bits are zero."""
    rows, cols = mask2d.shape
    nw = (cols + 31) // 32
    words = np.zeros((rows, nw), dtype=np.uint32)
    for j in range(cols):
        words[:, j >> 5] |= (mask2d[:, j].astype(np.uint32) << np.uint32(j & 31))
    return words


def unpack_mask(words, cols):
    rows = words.shape[0]
    out = np.zeros((rows, cols), dtype=bool)
    for j in range(cols):
        out[:, j] = (words[:, j >> 5] >> np.uint32(j & 31)) & 1
    return out


def relu_fragments(h_out, mask2d):
    """Fragment store of a ReLU layer (Section 5.1 applied to ReLU): the output-cotangent
    elements the vijp cannot reconstruct are exactly those at dead units.  cnt[b] = number of
    dead units in row b, off = exclusive prefix sum of cnt, values in row order, increasing j."""
    dead = ~mask2d
    cnt = dead.sum(axis=1).astype(np.uint64)
    off = np.concatenate([[0], np.cumsum(cnt)[:-1]]).astype(np.uint64)
    vals = h_out.reshape(mask2d.shape)[dead]          # row-major order of True entries
    return cnt, off, vals


def relu_restore(gz, mask2d, off, vals):
    """Inverse of relu_fragments inside the sweep: live units take g_z (phi' = 1), dead
    units pop their stored value at off[b] + (rank of j among the dead units of row b)."""
    out = np.array(gz, dtype=np.float64).reshape(mask2d.shape).copy()
    for b in range(mask2d.shape[0]):
        dead_cols = np.nonzero(~mask2d[b])[0]
        o = int(off[b])
        out[b, dead_cols] = vals[o:o + dead_cols.size]
    return out


# ----------------------------------------------------------------------------
# Algorithm 1 (Moonwalk), mixed mode: Phases I, II, III of Section 4.1
# ----------------------------------------------------------------------------
def input_cotangent(layers, params, x0, target, loss, reseed_every=0, masks=None, frag_block=0):
    """Phase I + Phase II.  Phase I keeps only the sign bits.  Phase II walks back computing
    input cotangents only; on the way it writes (a) the ReLU fragments and (b) a full cotangent
    checkpoint h_l for every l that is a multiple of `reseed_every` (0 < l < L)."""
    L = len(layers)
    x = x0
    ms = []
    for l, (layer, w) in enumerate(zip(layers, params)):           # Phase I
        z = linear_forward(layer, w, x)
        m = sign_mask(z) if masks is None or masks[l] is None else masks[l].reshape(z.shape)
        if layer.act == ACT_NONE:
            m = np.ones(z.shape, dtype=bool)
        ms.append(m)
        x = act_forward(z, layer, m)
    J, h = loss_and_cotangent(x, target, loss)
    store = dict(masks=ms, fragments={}, reseed={}, loss=J, h_last=h, conv_fragments={},
                 frag_block=frag_block)
    in_shapes = [x0.shape]
    for layer in layers[:-1]:
        if layer.kind == CONV2D:
            ho, wo = layer.out_hw()
            in_shapes.append((x0.shape[0], ho, wo, layer.C_out))
        elif layer.kind == CONV1D:
            in_shapes.append((x0.shape[0], layer.out_hw()[1], layer.C_out))
        else:
            in_shapes.append((x0.shape[0], layer.n_out))
    for l in range(L - 1, -1, -1):                                  # Phase II
        layer = layers[l]
        if layer.act == ACT_RELU:
            m2 = ms[l].reshape(ms[l].shape[0], -1)
            store["fragments"][l] = relu_fragments(h, m2)
        if reseed_every and (l + 1) % reseed_every == 0 and (l + 1) < L:
            store["reseed"][l + 1] = h.copy()
        gz = h * act_derivative(layer, ms[l])
        if layer.kind == CONV1D:
            # the convolution's own output cotangent g_z is what its vijp has to rebuild
            store["conv_fragments"][l] = conv1d_fragments(gz, layer.k, frag_block)
        h = linear_vjp_input(layer, params[l], gz, in_shapes[l])
    store["g0"] = h
    return h, store


def forward_sweep(layers, params, x0, g0, store, conv_iters=None, apply=None):
    """Phase III = the loop body of Algorithm 1: x_i = f_i(x_{i-1}); h_i = vijp(f_i, x_{i-1},
    h_{i-1}) (Eq. "h_i"); g_i = vjp(f_i, theta_i, h_i) (Eq. "g_i"); "apply g_i to theta_i":
    `apply(i, g_i)` is called as soon as g_i exists.  The last layer's output cotangent is the
    loss cotangent itself when that layer has no vijp (classification head)."""
    L = len(layers)
    ms = store["masks"]
    x, h = x0, g0
    dW = [None] * L
    hs = [g0]
    for l, (layer, w) in enumerate(zip(layers, params)):
        z = linear_forward(layer, w, x)
        if layer.kind == HEAD:
            gz = store["h_last"]                      # no vijp through a non-square last layer
        elif layer.kind == CONV1D:
            gz = vijp_conv1d_fragmental(layer, w, h, store["conv_fragments"][l], store["frag_block"])
        else:
            gz = vijp_linear(layer, w, h, conv_iters).reshape(z.shape)
        m = ms[l]
        if layer.act == ACT_RELU:
            gz = np.where(m, gz, 0.0)                 # phi' = 0: exact zeros at dead units
            _, off, vals = store["fragments"][l]
            hn = relu_restore(gz, m.reshape(m.shape[0], -1), off, vals).reshape(z.shape)
        elif layer.act == ACT_LEAKY:
            hn = vijp_leaky(layer, m, gz)
        else:
            hn = gz
        dW[l] = linear_vjp_param(layer, x, gz, w)
        if apply is not None:
            apply(l, dW[l])
        x = act_forward(z, layer, m)
        h = hn
        if (l + 1) in store["reseed"]:
            h = store["reseed"][l + 1]
        hs.append(h)
    return dict(dW=dW, h=hs)


def trainable_entries(layer, w):
    """Section "Constrained Convolutions": layers are parameterised so that the conditions of their
    vijp hold by construction.  The entries that Lemma 1 (ii) fixes at zero (anchor tap w[p], c < c')
    -- for the stride-1 1-D convolution of Section 5.1 those of tap 0 -- are not parameters.
    Returns 1.0 at trainable entries, 0.0 at fixed ones."""
    m = np.ones(w.shape)
    if layer.kind == CONV2D and layer.stride > layer.pad:
        m[layer.pad, layer.pad] = np.tril(np.ones(w.shape[2:]))
    elif layer.kind == CONV1D:
        m[0] = np.tril(np.ones(w.shape[1:]))
    return m


def moonwalk_sgd_step(layers, params, x0, target, loss, lr, reseed_every=0, masks=None,
                      conv_iters=None, frag_block=0):
    """One step of gradient descent with Algorithm 1 as printed: every g_i is applied to theta_i
    (theta_i <- theta_i - lr g_i) the moment it is formed and then dropped.  Layer i's own
    parameters are not read again after that, so the result equals theta - lr grad J."""
    g0, store = input_cotangent(layers, params, x0, target, loss, reseed_every, masks, frag_block)
    new = [np.array(p, dtype=np.float64) for p in params]

    def apply(i, g):
        new[i] = new[i] - lr * g * trainable_entries(layers[i], params[i])

    forward_sweep(layers, params, x0, g0, store, conv_iters, apply=apply)
    return new


def moonwalk(layers, params, x0, target, loss, reseed_every=0, masks=None, conv_iters=None,
             frag_block=0):
    g0, store = input_cotangent(layers, params, x0, target, loss, reseed_every, masks, frag_block)
    out = forward_sweep(layers, params, x0, g0, store, conv_iters)
    out.update(loss=store["loss"], g0=g0, masks=store["masks"], store=store)
    return out


# ----------------------------------------------------------------------------
# comparison helpers used by the parity tests
# ----------------------------------------------------------------------------
def normwise_error(a, ref):
    """max |a - ref| / max |ref|  (the per-layer 'max relative error')."""
    ref = np.asarray(ref, dtype=np.float64)
    den = np.abs(ref).max()
    return float(np.abs(np.asarray(a, dtype=np.float64) - ref).max() / (den if den > 0 else 1.0))
