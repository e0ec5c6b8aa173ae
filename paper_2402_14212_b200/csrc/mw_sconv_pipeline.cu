// Tensor-core pipelines of the three calls for the fully submersive CNN of the paper's experiments
// (Section "Fully Parallel Submersive 2D CNN"): a chain of k x k convolutions with C channels in
// and out, stride 2 and padding below the stride, each halving the resolution, leaky-ReLU (or
// no) activation, a loss on the last feature map.  MW_F32.
//
// Each layer meets Lemma 1: the anchor tap w[p] is lower triangular in (c, c') with a non-zero
// diagonal, and with k - 1 - p < s no other tap reaches the positions s*i' of the input
// cotangent.  The elimination of the lemma's proof (Algorithm 2) then recovers h'[i', :] from
// h[s i', :] alone by a triangular solve per pixel; here the anchor tap is inverted once per
// step and the vijp of all pixels is ONE product with that inverse:
//     g_z[i', :] = h[s i', :] A^-T,   A = w[p]  indexed [c][c'].
// Every step is a product of the persistent tcgen05 kernel (mw_conv_tensor.cu):
//   Phase I    x_{l+1} = phi(conv(x_l, w_l))            strided window      -> sign words + planes
//   Phase II   h_l = TransposeConv(g_z, w_l)            four parity classes -> checkpoint, next g_z
//   sweep      recompute x_{l+1}; g_z = vijp (above) with the activation's vijp in the epilogue
//              (Eq. "h_i"); dw_l = weight vjp(x_l, g_z) (Eq. "g_i").
#include "mw_conv_tensor.cuh"
#include "mw_tensor.cuh"

namespace mw {

namespace {

struct SCtx {
  mw_net* n;
  const Layout* lay;
  void* ws;
  cudaStream_t s;
  TcMapCache* cache;
  DeviceStatus* st;
  int L, C;
  // bf16 terms per operand.  MW_F32: three for everything on the chains, two for the weight vjp.
  // MW_BF16_F32ACC: x and w are bf16 in memory and serve as their own single plane; cotangents
  // and the inverse anchor tap carry two terms.
  bool bf16;
  int px, pw, pg, ph, pinv, pwg;
  const void* const* params;
  const void* x;
  template <typename T> T* at(const Region& r) const { return mw::at<T>(ws, r); }
  ConvGeom geom(int l) const {
    const mw_layer_desc& d = n->layers[l];
    return ConvGeom{n->B, d.H, d.W, d.k, d.pad, d.C_in, d.stride};
  }
  int64_t in_elems(int l) const { return n->info[l].in_elems; }
  int64_t out_elems(int l) const { return n->info[l].out_elems; }
};

SCtx make_sctx(mw_net* n, const Layout& lay, void* ws, cudaStream_t s, const void* const* params,
               const void* x) {
  SCtx c;
  c.n = n; c.lay = &lay; c.ws = ws; c.s = s;
  c.params = params; c.x = x;
  c.bf16 = n->opts.prec == MW_BF16_F32ACC;
  c.px = c.bf16 ? 1 : 3; c.pw = c.bf16 ? 1 : 3;
  c.pg = c.bf16 ? 2 : 3; c.ph = c.bf16 ? 2 : 3; c.pinv = c.bf16 ? 2 : 3;
  c.pwg = c.bf16 ? 1 : 2;
  c.cache = static_cast<TensorState*>(n->tc)->cache;
  c.st = status_of(ws, lay);
  c.L = n->L;
  c.C = n->layers[0].C_in;
  return c;
}

// can a tile of `span` consecutive pixels of Ho x Wo images be one box: part of a row, whole
// rows of one image, or whole images
bool tiles_ok(int Ho, int Wo, int span) {
  const int bx = Wo < span ? Wo : span;
  if (span % bx != 0 || Wo % bx != 0) return false;
  const int by = span / bx < Ho ? span / bx : Ho;
  if (Ho % by != 0) return false;
  return bx * by * (span / (bx * by)) == span;
}

// Inverse of the lower triangular anchor taps of up to kSmallBatch layers, one CTA per layer
// and one thread per column: x_i = (delta_ij - sum_{m<i} A[i][m] x_m) / A[i][i], in double.
// A tap with an entry above the diagonal or a zero on it violates Lemma 1 (ii) / (iii).
__device__ __forceinline__ float as_float(float v) { return v; }
__device__ __forceinline__ float as_float(__nv_bfloat16 v) { return __bfloat162float(v); }

template <typename T>
__global__ void __launch_bounds__(256)
anchor_inverse_kernel(SmallBatch ws, int64_t offset, int n, float* __restrict__ inv0,
                      DeviceStatus* st, int layer0) {
  extern __shared__ double xs[];            // [n][n], column j owned by thread j
  const T* A = static_cast<const T*>(ws.p[blockIdx.x]) + offset;
  float* inv = inv0 + (int64_t)blockIdx.x * n * n;
  __shared__ int bad;
  if (threadIdx.x == 0) bad = 0;
  __syncthreads();
  for (int e = threadIdx.x; e < n * n; e += blockDim.x) {
    const int i = e / n, j = e - i * n;
    const float v = as_float(A[e]);
    if ((j > i && v != 0.f) || (j == i && !(fabsf(v) > 0.f))) bad = 1;
  }
  __syncthreads();
  if (bad) {
    if (threadIdx.x == 0)
      record_error(st, MW_ERR_NOT_SUBMERSIVE, (unsigned)(layer0 + blockIdx.x), 0u, 2u, 0u);
    return;
  }
  for (int j = threadIdx.x; j < n; j += blockDim.x) {
    for (int i = 0; i < n; ++i) {
      double a = i == j ? 1.0 : 0.0;
      if (i > j)
        for (int m = j; m < i; ++m) a -= (double)as_float(A[i * n + m]) * xs[m * n + j];
      xs[i * n + j] = i < j ? 0.0 : a / (double)as_float(A[i * n + i]);
    }
    for (int i = 0; i < n; ++i) inv[i * n + j] = (float)xs[i * n + j];
  }
}

// fp32 pixel array [images][H][W][C] -> term planes of its pixels (s*y, s*x): [images][H/s][W/s][C]
__global__ void __launch_bounds__(256)
split_subsampled_kernel(const float* __restrict__ in, int Ho, int Wo, int s, int C4, int64_t n4,
                        __nv_bfloat16* __restrict__ out, int planes, int64_t plane_stride) {
  const int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x;
  if (i >= n4) return;
  const int c4 = (int)(i % C4);
  const int64_t pix = i / C4;
  const int x = (int)(pix % Wo);
  const int64_t r = pix / Wo;
  const int y = (int)(r % Ho);
  const int64_t b = r / Ho;
  const int64_t src = ((b * Ho * s + (int64_t)y * s) * (Wo * s) + (int64_t)x * s) * C4 + c4;
  const float4 v = reinterpret_cast<const float4*>(in)[src];
  float rem[4] = {v.x, v.y, v.z, v.w};
  for (int p = 0; p < planes; ++p) {
    __nv_bfloat16 t[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      t[k] = __float2bfloat16_rn(rem[k]);
      rem[k] -= __bfloat162float(t[k]);
    }
    uint2 pk;
    pk.x = (uint32_t)__bfloat16_as_ushort(t[0]) | ((uint32_t)__bfloat16_as_ushort(t[1]) << 16);
    pk.y = (uint32_t)__bfloat16_as_ushort(t[2]) | ((uint32_t)__bfloat16_as_ushort(t[3]) << 16);
    reinterpret_cast<uint2*>(out + (int64_t)p * plane_stride)[i] = pk;
  }
}

// per-step preparation: kernel term planes; for Moonwalk also the anchor-tap inverses
mw_status prep(const SCtx& c, const void* const* params, bool inverse) {
  const Layout& lay = *c.lay;
  const int C = c.C;
  if (!c.bf16)
    for (int l = 0; l < c.L; ++l) {
      const int64_t we = c.geom(l).kernel_elems();
      MW_TRY(split_planes((const float*)params[l], we, c.at<__nv_bfloat16>(lay.cw[l]), 3, we, c.s));
    }
  if (!inverse) return MW_OK;
  static bool attr_done = false;
  const size_t smem = sizeof(double) * C * C;
  if (!attr_done) {
    MW_CUDA_OK(cudaFuncSetAttribute(anchor_inverse_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    200 * 1024));
    MW_CUDA_OK(cudaFuncSetAttribute(anchor_inverse_kernel<__nv_bfloat16>,
                                    cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
    attr_done = true;
  }
  float* inv = c.at<float>(lay.cwinv_f32);       // [kSmallBatch][C*C]
  for (int l0 = 0; l0 < c.L; l0 += kSmallBatch) {
    const int G = c.L - l0 < kSmallBatch ? c.L - l0 : kSmallBatch;
    SmallBatch ws{};
    for (int g = 0; g < G; ++g) ws.p[g] = params[l0 + g];
    const mw_layer_desc& d = c.n->layers[l0];
    const int64_t off = (int64_t)(d.pad * d.k + d.pad) * C * C;
    if (c.bf16) anchor_inverse_kernel<__nv_bfloat16><<<G, 128, smem, c.s>>>(ws, off, C, inv, c.st, l0);
    else anchor_inverse_kernel<float><<<G, 128, smem, c.s>>>(ws, off, C, inv, c.st, l0);
    MW_TRY(launch_ok());
    for (int g = 0; g < G; ++g)
      MW_TRY(split_planes(inv + (int64_t)g * C * C, (int64_t)C * C, c.at<__nv_bfloat16>(lay.cwinv[l0 + g]),
                          c.pinv, (int64_t)C * C, c.s));
  }
  return MW_OK;
}

// x planes of layer l's input: the largest one (l = 0) has a buffer of its own, the others rotate
__nv_bfloat16* x_planes(const SCtx& c, int l) {
  // a bf16 input is its own (single) term plane
  if (l == 0 && c.bf16) return const_cast<__nv_bfloat16*>(static_cast<const __nv_bfloat16*>(c.x));
  return c.at<__nv_bfloat16>(l == 0 ? c.lay->xp[0] : c.lay->xp[1 + ((l - 1) & 1)]);
}

const __nv_bfloat16* w_planes(const SCtx& c, int l) {
  return c.bf16 ? static_cast<const __nv_bfloat16*>(c.params[l]) : c.at<__nv_bfloat16>(c.lay->cw[l]);
}

// Phase I (or backprop's forward): sign words, x_{l+1} planes (kept per layer for backprop);
// the last output lands in fp32 (cxf) for the loss
mw_status forward_pass(const SCtx& c, const void* const* params, const void* x, bool store_acts) {
  const Layout& lay = *c.lay;
  MW_TRY(prep(c, params, !store_acts));
  if (!c.bf16) MW_TRY(split_planes((const float*)x, c.in_elems(0), x_planes(c, 0), 3, c.in_elems(0), c.s));
  const __nv_bfloat16* xin = x_planes(c, 0);
  for (int l = 0; l < c.L; ++l) {
    const mw_layer_desc& ld = c.n->layers[l];
    const bool last = l + 1 == c.L;
    __nv_bfloat16* xout = store_acts && !last ? c.at<__nv_bfloat16>(lay.stored_act[l + 1]) : x_planes(c, l + 1);
    TcEpilogue e;
    e.mode = TC_EPI_FWD;
    e.mask = c.at<uint32_t>(lay.mask[l]);
    e.write_mask = 1;
    e.act = ld.act;
    e.slope = (float)ld.slope;
    if (!last) { e.planes = xout; e.n_planes = c.px; e.plane_stride = c.out_elems(l); }
    else e.out_f32 = c.at<float>(lay.cxf);
    TcGemm g = conv_forward_product(c.geom(l), xin, c.px, w_planes(c, l), c.pw, e);
    MW_TRY(tc_gemm_group(c.cache, &g, 1, c.st, c.s));
    xin = xout;
  }
  return MW_OK;
}

// loss and g_z of the last layer as three term planes in hp[0]
mw_status loss_top(const SCtx& c, const void* target, double* loss_out) {
  const Layout& lay = *c.lay;
  const int l = c.L - 1;
  const mw_layer_desc& ld = c.n->layers[l];
  const int64_t rows = c.n->info[l].rows;
  float* h = c.at<float>(lay.cot[0]);
  MW_TRY(loss_cotangent<float>(c.at<float>(lay.cxf), target, rows, c.C, c.n->opts.loss, h,
                               c.at<double>(lay.partials), loss_out, c.s));
  const float* src = h;
  if (ld.act != MW_ACT_NONE) {
    float* g = c.at<float>(lay.cot[1]);
    MW_TRY(scale_by_mask<float>(h, c.at<uint32_t>(lay.mask[l]), rows, c.C, ld.act, ld.slope, g, c.s));
    src = g;
  }
  return split_planes(src, c.out_elems(l), c.at<__nv_bfloat16>(lay.hp[0]), c.pg, c.out_elems(l), c.s);
}

// h_l = TransposeConv(g_z(l), w_l) through its parity classes, one launch; `e` is the epilogue of
// every class
// `checkpoint` (optional): term planes of h_l at the pixels (s*y, s*x), which is all the vijp of
// layer l reads of it; they are the rows of class (0, 0)
// With `only_checkpoint` nothing but those pixels is computed (one class, one ninth of the work).
mw_status transpose_classes(const SCtx& c, int l, const __nv_bfloat16* gz, const TcEpilogue& e,
                            __nv_bfloat16* checkpoint, bool only_checkpoint = false) {
  const ConvGeom g = c.geom(l);
  TcGemm cls[kTcMaxGroup];
  int n = 0;
  for (int py = 0; py < g.stride; ++py)
    for (int px = 0; px < g.stride; ++px) {
      if (only_checkpoint && (py || px)) continue;
      if (n == kTcMaxGroup) return MW_ERR_UNSUPPORTED;
      if (!conv_transpose_class_product(g, py, px, gz, c.pg, w_planes(c, l), c.pw, e, &cls[n]))
        return MW_ERR_UNSUPPORTED;
      if (checkpoint && py == 0 && px == 0) {
        TcEpilogue& ce = cls[n].epi;
        ce.planes2 = checkpoint; ce.n_planes2 = c.ph; ce.plane_stride2 = c.out_elems(l); ce.compact2 = 1;
      }
      ++n;
    }
  return tc_gemm_group(c.cache, cls, n, c.st, c.s);
}

// the backward walk shared by Phase II and backprop: for l = L-1 .. 0 (optionally the weight
// vjp of layer l first) h_l -> g0 / checkpoint, g_z(l-1) planes
mw_status backward_pass(const SCtx& c, void* g0, __nv_bfloat16* seed, void* const* dW, bool checkpoints) {
  const Layout& lay = *c.lay;
  int cur = 0;
  for (int l = c.L - 1; l >= 0; --l) {
    const __nv_bfloat16* gz = c.at<__nv_bfloat16>(lay.hp[cur]);
    if (dW && dW[l]) {
      const __nv_bfloat16* xl = l == 0 ? x_planes(c, 0) : c.at<__nv_bfloat16>(lay.stored_act[l]);
      MW_TRY(conv_wgrad_tensor(c.cache, c.geom(l), xl, gz, c.pwg, c.at<float>(lay.cpart), (float*)dW[l], c.st, c.s));
    }
    if (l == 0 && !g0 && !seed) break;
    TcEpilogue e;
    e.mode = TC_EPI_BWD;
    if (l == 0) {
      // the input cotangent: in full when the caller wants it; the sweep itself only needs its
      // pixels (s*y, s*x), kept as term planes
      e.out_f32 = (float*)g0;
      MW_TRY(transpose_classes(c, 0, gz, e, seed, g0 == nullptr));
      break;
    } else {
      const mw_layer_desc& below = c.n->layers[l - 1];
      e.act = below.act;
      e.slope = (float)below.slope;
      e.mask = c.at<uint32_t>(lay.mask[l - 1]);
      e.planes = c.at<__nv_bfloat16>(lay.hp[cur ^ 1]);
      e.n_planes = c.pg;
      e.plane_stride = c.in_elems(l);
    }
    MW_TRY(transpose_classes(c, l, gz, e, l > 0 && checkpoints && is_reseed(c.n, l)
                                                ? c.at<__nv_bfloat16>(lay.reseed[l]) : nullptr));
    cur ^= 1;
  }
  return MW_OK;
}

}  // namespace

bool sconv_tensor_supported(const mw_net* n) {
  if (n->opts.prec != MW_F32 && n->opts.prec != MW_BF16_F32ACC) return false;
  if (n->opts.loss == MW_LOSS_XENT_MEAN) return false;
  const int C = n->layers[0].C_in;
  if (C < 64 || C % 64 != 0 || C > 128) return false;     // the anchor inverse keeps C*C doubles on chip
  for (int l = 0; l < n->L; ++l) {
    const mw_layer_desc& d = n->layers[l];
    if (d.kind != MW_CONV2D || d.C_in != C || d.C_out != C) return false;
    if (d.act == MW_ACT_RELU) return false;
    if (d.act == MW_ACT_LEAKY_RELU && !(d.slope != 0.0)) return false;
    // Lemma 1 (i), two parity classes per dimension, and no tap but the anchor at positions s*i'
    if (d.stride != 2 || d.pad >= d.stride || d.k <= d.pad || d.k - 1 - d.pad >= d.stride ||
        d.k * d.k > kTcMaxTaps)
      return false;
    const int Ho = (d.H + 2 * d.pad - d.k) / d.stride + 1, Wo = (d.W + 2 * d.pad - d.k) / d.stride + 1;
    if (d.H != 2 * Ho || d.W != 2 * Wo) return false;
    if (!tiles_ok(Ho, Wo, 128) || !tiles_ok(Ho, Wo, 64) || 2 * Wo > 256) return false;
    if (((int64_t)n->B * Ho * Wo) % 64 != 0) return false;
    if (l + 1 < n->L && (n->layers[l + 1].H != Ho || n->layers[l + 1].W != Wo)) return false;
    if ((int64_t)n->B * d.H * d.W >= ((int64_t)1 << 31) / C) return false;
  }
  return true;
}

void sconv_tensor_layout(mw_net* n, bool backprop, Layout& lay, size_t start) {
  struct B2 {
    size_t cur;
    Region take(size_t bytes) {
      Region r; r.off = cur; r.bytes = bytes; cur = align_up(cur + bytes, 256); return r;
    }
  } b{start};
  const int L = n->L;
  const int C = n->layers[0].C_in;
  const size_t P0 = (size_t)n->info[0].in_elems, P1 = (size_t)n->info[0].out_elems;
  const size_t PL = (size_t)n->info[L - 1].out_elems;
  size_t we = 0, part = 0;
  for (int l = 0; l < L; ++l) {
    const size_t w = (size_t)n->info[l].w_elems;
    if (w > we) we = w;
    const size_t p = 4 * (size_t)conv_wgrad_tensor_slices(n->info[l].rows, C, n->layers[l].k * n->layers[l].k) * w;
    if (p > part) part = p;
  }
  // bf16 terms per operand (see SCtx); a bf16 net reads x and w in place
  const bool bf16 = n->opts.prec == MW_BF16_F32ACC;
  const size_t px = bf16 ? 1 : 3, pg = bf16 ? 2 : 3, pwg = bf16 ? 1 : 2;
  for (int i = 0; i < 2; ++i) lay.cot[i] = b.take(4 * PL);
  lay.cxf = b.take(4 * PL);
  lay.xp[0] = b.take(bf16 ? 256 : 2 * 3 * P0);          // x_0 planes
  for (int i = 1; i < 3; ++i) lay.xp[i] = b.take(2 * px * P1);
  for (int i = 0; i < 2; ++i) lay.hp[i] = b.take(2 * pg * P1);  // g_z planes (backward walk), h planes (sweep)
  lay.cw.resize(L); lay.cwinv.resize(L);
  for (int l = 0; l < L; ++l) lay.cw[l] = b.take(bf16 ? 256 : 2 * 3 * (size_t)n->info[l].w_elems);
  lay.cpart = b.take(part);
  if (!backprop) {
    lay.cg[0] = b.take(2 * pwg * P1);                   // g_z planes of the sweep, as the weight vjp reads them
    lay.cseed = b.take(2 * pg * P1);                    // h_0 at the pixels (s*y, s*x): survives to the sweep
    lay.residual += 2 * pg * P1;
    for (int l = 0; l < L; ++l) lay.cwinv[l] = b.take(2 * pg * (size_t)C * C);
    lay.cwinv_f32 = b.take(4 * (size_t)C * C * kSmallBatch);
  }
  lay.total = b.cur;
}

mw_status sconv_tensor_input_cotangent(mw_net* n, const void* const* params, const void* x,
                                       const void* target, void* g0, double* loss_out, void* ws,
                                       cudaStream_t s) {
  const Layout& lay = n->mwl;
  SCtx c = make_sctx(n, lay, ws, s, params, x);
  MW_CUDA_OK(cudaMemsetAsync(at<char>(ws, lay.status), 0, 256, s));
  MW_TRY(forward_pass(c, params, x, false));          // Phase I (+ per-step preparation)
  MW_TRY(loss_top(c, target, loss_out));
  return backward_pass(c, g0, c.at<__nv_bfloat16>(lay.cseed), nullptr, true);   // Phase II
}

mw_status sconv_tensor_forward_sweep(mw_net* n, const void* const* params, const void* x,
                                     const void* g0, void* const* dW, void* ws, cudaStream_t s) {
  const Layout& lay = n->mwl;
  SCtx c = make_sctx(n, lay, ws, s, params, x);
  const int L = c.L, C = c.C;
  // the term planes of an fp32 x (xp[0]) are still those Phase I made from the same x
  const __nv_bfloat16* hcur = c.at<__nv_bfloat16>(lay.cseed);   // Phase II's own seed
  if (g0) {
    // only the pixels s*i' of the input cotangent enter the vijp: split those
    const mw_layer_desc& d = n->layers[0];
    const int Ho = d.H / d.stride, Wo = d.W / d.stride;
    const int64_t n4 = c.out_elems(0) / 4;
    split_subsampled_kernel<<<(unsigned)((n4 + 255) / 256), 256, 0, s>>>(
        (const float*)g0, Ho, Wo, d.stride, C / 4, n4, c.at<__nv_bfloat16>(lay.hp[0]), c.ph, c.out_elems(0));
    MW_TRY(launch_ok());
    hcur = c.at<__nv_bfloat16>(lay.hp[0]);
  }
  for (int l = 0; l < L; ++l) {
    const mw_layer_desc& ld = n->layers[l];
    const ConvGeom g = c.geom(l);
    uint32_t* words = c.at<uint32_t>(lay.mask[l]);
    const __nv_bfloat16* xin = x_planes(c, l);
    const __nv_bfloat16* hin = hcur;
    __nv_bfloat16* hout = c.at<__nv_bfloat16>(lay.hp[(l + 1) & 1]);   // l = 0 reads hp[0] or the seed
    const bool more = l + 1 < L;
    const bool reseed_next = more && is_reseed(n, l + 1);
    const bool want_h = more && !reseed_next;
    if (more) {                                        // recompute x_{l+1}
      TcEpilogue e;
      e.mode = TC_EPI_FWD;
      e.mask = words;
      e.write_mask = 0;
      e.act = ld.act;
      e.slope = (float)ld.slope;
      e.planes = x_planes(c, l + 1); e.n_planes = c.px; e.plane_stride = c.out_elems(l);
      TcGemm p = conv_forward_product(g, xin, c.px, w_planes(c, l), c.pw, e);
      MW_TRY(tc_gemm_group(c.cache, &p, 1, c.st, s));
    }
    if (dW[l] || want_h) {
      // vijp of the convolution (one product with the inverse anchor tap) and of the activation
      TcGemm p;
      p.B.base = c.at<__nv_bfloat16>(lay.cwinv[l]); p.B.rows = C; p.B.cols = C; p.B.planes = c.pinv;
      p.B.plane_stride = (int64_t)C * C; p.B.mn_major = false;
      p.M = (int)g.out_pixels(); p.N = C; p.K = C;
      // h_l is kept at the pixels s*i' only (all that the elimination reads)
      p.A = pixel_operand(hin, g.out_pixels(), c.ph, c.out_elems(l), false, C);
      TcEpilogue& e = p.epi;
      e.mode = TC_EPI_VIJP;
      e.act = ld.act;
      e.slope = (float)ld.slope;
      e.mask = words;
      if (want_h) {
        const mw_layer_desc& nd = n->layers[l + 1];
        e.planes2 = hout; e.n_planes2 = c.ph; e.plane_stride2 = c.out_elems(l + 1);
        e.sub2_s = nd.stride; e.sub2_h = nd.H; e.sub2_w = nd.W;
      }
      if (dW[l]) { e.planes = c.at<__nv_bfloat16>(lay.cg[0]); e.n_planes = c.pwg; e.plane_stride = c.out_elems(l); }
      MW_TRY(tc_gemm_group(c.cache, &p, 1, c.st, s));
    }
    // the recursion restarts from the stored cotangent h_{l+1} (term planes) where there is one
    hcur = reseed_next ? c.at<__nv_bfloat16>(lay.reseed[l + 1]) : hout;
    if (dW[l])
      MW_TRY(conv_wgrad_tensor(c.cache, g, xin, c.at<__nv_bfloat16>(lay.cg[0]), c.pwg, c.at<float>(lay.cpart),
                               (float*)dW[l], c.st, s,
                               n->apply_params ? (const float*)n->apply_params[l] : nullptr, n->apply_lr));
    if (dW[l] && n->apply_params)   // the zeros of the anchor tap are structure, not parameters
      MW_TRY(conv_zero_fixed_entries((float*)dW[l], (int64_t)(ld.pad * ld.k + ld.pad) * C * C, C, s));
  }
  return MW_OK;
}

mw_status sconv_tensor_backprop(mw_net* n, const void* const* params, const void* x,
                                const void* target, void* const* dW, double* loss_out, void* ws,
                                cudaStream_t s) {
  const Layout& lay = n->bpl;
  SCtx c = make_sctx(n, lay, ws, s, params, x);
  MW_CUDA_OK(cudaMemsetAsync(at<char>(ws, lay.status), 0, 256, s));
  MW_TRY(forward_pass(c, params, x, true));
  MW_TRY(loss_top(c, target, loss_out));
  return backward_pass(c, nullptr, nullptr, dW, false);
}

}  // namespace mw
