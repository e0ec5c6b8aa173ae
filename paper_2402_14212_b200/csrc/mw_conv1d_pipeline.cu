// Tensor-core pipelines of the three calls for the 1-D CNN of the paper's fragmental-checkpointing
// experiment (Section "Fragmental Checkpointing"): a chain of k = 3, stride-1, padding-1
// convolutions on [N positions][C channels] sequences with leaky-ReLU, shape kept.  MW_F32.
//
// Such a layer is not submersive by Lemma 1 (s = p).  Its reverse pass reads
//     h[i] = w[0] g[i+1] + w[1] g[i] + w[2] g[i-1]          (g = the convolution's output cotangent)
// and with tap 0 lower triangular in (c, c') (Section 5.1) the newest unknown follows from the two
// before it:  g[i+1] = W0^-1 h[i] - (W0^-1 w[1]) g[i] - (W0^-1 w[2]) g[i-1].
// Phase II keeps g at the first two positions of every block of `frag_block` positions (the
// fragments: 2 / frag_block of a full checkpoint); the sweep rebuilds every block from them, all
// blocks of all samples in parallel and the positions of a block one after the other:
//   c     = h W0^-T                        one product over all positions (fp32, kept)
//   step t = 2 .. block-1:  g[.., t] = c[.., t-1] - [g[.., t-2] | g[.., t-1]] [w^2 | w^1]^T
//                           one product per step: rows = (sample, block), K = 2 C
// (Algorithm 3, with the triangular term of tap 0 that its listing leaves out folded into W0^-1).
// Forward, TransposeConv and weight vjp are products with shifted windows as for the 2-D nets.
#include "mw_conv_tensor.cuh"
#include "mw_tensor.cuh"

namespace mw {

namespace {

struct C1 {
  mw_net* n;
  const Layout* lay;
  void* ws;
  cudaStream_t s;
  TcMapCache* cache;
  DeviceStatus* st;
  int L, C, N, k, blk;
  // bf16 terms per operand: MW_F32 three on the chains and two in the weight vjp; MW_BF16_F32ACC:
  // x and w are bf16 in memory and serve as their own single plane, cotangents and W0^-1 two terms
  bool bf16;
  int px, pw, pg, pwg;
  const void* const* params;
  const void* x;
  int64_t P;          // elements of one activation: B * N * C
  int64_t we;         // elements of one kernel: k * C * C
  template <typename T> T* at(const Region& r) const { return mw::at<T>(ws, r); }
};

C1 make_c1(mw_net* n, const Layout& lay, void* ws, cudaStream_t s, const void* const* params,
           const void* x) {
  C1 c;
  c.n = n; c.lay = &lay; c.ws = ws; c.s = s;
  c.params = params; c.x = x;
  c.bf16 = n->opts.prec == MW_BF16_F32ACC;
  c.px = c.bf16 ? 1 : 3; c.pw = c.px; c.pg = c.bf16 ? 2 : 3; c.pwg = c.bf16 ? 1 : 2;
  c.cache = static_cast<TensorState*>(n->tc)->cache;
  c.st = status_of(ws, lay);
  const mw_layer_desc& d = n->layers[0];
  c.L = n->L; c.C = d.C_in; c.N = d.W; c.k = d.k; c.blk = n->opts.frag_block;
  c.P = (int64_t)n->B * d.W * d.C_in;
  c.we = (int64_t)d.k * d.C_in * d.C_in;
  return c;
}

// ---- small kernels ---------------------------------------------------------------------------
// inverse of the lower triangular tap 0 of up to kSmallBatch layers: CTA (layer, group of 64
// columns), one thread per column, x_i = (delta_ij - sum_{m<i} A[i][m] x_m) / A[i][i] in double,
// the columns of the group in shared memory ([n][64] doubles)
constexpr int kTriCols = 64;
__device__ __forceinline__ float ld_f(const float* p) { return __ldg(p); }
__device__ __forceinline__ float ld_f(const __nv_bfloat16* p) { return __bfloat162float(*p); }

template <typename T>
__global__ void __launch_bounds__(kTriCols)
tri_inverse_kernel(SmallBatch ws, int n, float* __restrict__ inv0, DeviceStatus* st, int layer0) {
  extern __shared__ double xs[];            // [n][kTriCols]
  const T* A = static_cast<const T*>(ws.p[blockIdx.x]);
  float* inv = inv0 + (int64_t)blockIdx.x * n * n;
  __shared__ int bad;
  if (threadIdx.x == 0) bad = 0;
  __syncthreads();
  for (int e = threadIdx.x; e < n * n; e += blockDim.x) {
    const int i = e / n, j = e - i * n;
    const float v = ld_f(A + e);
    if ((j > i && v != 0.f) || (j == i && !(fabsf(v) > 0.f))) bad = 1;
  }
  __syncthreads();
  if (bad) {
    if (threadIdx.x == 0 && blockIdx.y == 0)
      record_error(st, MW_ERR_NOT_SUBMERSIVE, (unsigned)(layer0 + blockIdx.x), 0u, 3u, 0u);
    return;
  }
  const int t = threadIdx.x, j = blockIdx.y * kTriCols + t;
  if (j >= n) return;
  for (int i = 0; i < n; ++i) {
    double a = i == j ? 1.0 : 0.0;
    if (i > j) {
      // four independent partial sums: the chain of dependent fp64 adds is what takes the time
      const T* Ai = A + (int64_t)i * n;
      double s0 = 0.0, s1 = 0.0, s2 = 0.0, s3 = 0.0;
      int m = j;
      for (; m + 3 < i; m += 4) {
        s0 += (double)ld_f(Ai + m) * xs[m * kTriCols + t];
        s1 += (double)ld_f(Ai + m + 1) * xs[(m + 1) * kTriCols + t];
        s2 += (double)ld_f(Ai + m + 2) * xs[(m + 2) * kTriCols + t];
        s3 += (double)ld_f(Ai + m + 3) * xs[(m + 3) * kTriCols + t];
      }
      for (; m < i; ++m) s0 += (double)ld_f(Ai + m) * xs[m * kTriCols + t];
      a -= (s0 + s1) + (s2 + s3);
    }
    const double x = i < j ? 0.0 : a / (double)ld_f(A + (int64_t)i * n + i);
    xs[i * kTriCols + t] = x;
    inv[(int64_t)i * n + j] = (float)x;
  }
}

// eight bf16 values of one 128-bit load, as floats
__device__ __forceinline__ void unpack8(const uint4& u, float (&f)[8]) {
  const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    f[2 * i] = __uint_as_float(w[i] << 16);
    f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
  }
}

// fold[c][(q, c')] = sum_m W0inv[c][m] w[k-1-q][m][c'], q = 0 .. k-2: the B operand of a
// reconstruction step, whose K runs over the k - 1 previous positions, oldest first
template <typename T>
__global__ void __launch_bounds__(256)
fold1d_kernel(SmallBatch ws, const float* __restrict__ inv0, int C, int k, float* __restrict__ fold0) {
  const int c = blockIdx.x, q = blockIdx.y, cp = threadIdx.x;
  const T* w = static_cast<const T*>(ws.p[blockIdx.z]);
  const float* inv = inv0 + (int64_t)blockIdx.z * C * C;
  float* fold = fold0 + (int64_t)blockIdx.z * C * (k - 1) * C;
  const T* wj = w + (int64_t)(k - 1 - q) * C * C;
  for (int t = cp; t < C; t += blockDim.x) {
    float a = 0.f;
    for (int m = 0; m < C; ++m) a = fmaf(inv[c * C + m], ld_f(wj + (int64_t)m * C + t), a);
    fold[((int64_t)c * (k - 1) + q) * C + t] = a;
  }
}

// fragments of g (term planes, [rows = samples*N][C]) -> fp32 [samples*N/blk][keep*C]; eight
// channels per thread (C a multiple of 8)
__global__ void __launch_bounds__(256)
frag_gather_kernel(const __nv_bfloat16* __restrict__ planes, int n_planes, int64_t plane_stride, int C,
                   int blk, int keep, int64_t total8, float* __restrict__ frags) {
  const int64_t i8 = (int64_t)blockIdx.x * 256 + threadIdx.x;   // over [blocks][keep][C / 8]
  if (i8 >= total8) return;
  const int C8 = C >> 3;
  const int c = (int)(i8 % C8) * 8;
  const int64_t r = i8 / C8;
  const int q = (int)(r % keep);
  const int64_t b = r / keep;
  const int64_t src = (b * blk + q) * C + c;
  float a[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
  for (int p = n_planes - 1; p >= 0; --p) {
    float f[8];
    unpack8(*reinterpret_cast<const uint4*>(planes + (int64_t)p * plane_stride + src), f);
#pragma unroll
    for (int k = 0; k < 8; ++k) a[k] += f[k];
  }
  float4* dst = reinterpret_cast<float4*>(frags + i8 * 8);
  dst[0] = make_float4(a[0], a[1], a[2], a[3]);
  dst[1] = make_float4(a[4], a[5], a[6], a[7]);
}

// the inverse: fp32 fragments -> term planes at the first `keep` positions of every block
__global__ void __launch_bounds__(256)
frag_scatter_kernel(const float* __restrict__ frags, int C, int blk, int keep, int64_t total8,
                    __nv_bfloat16* __restrict__ planes, int n_planes, int64_t plane_stride) {
  const int64_t i8 = (int64_t)blockIdx.x * 256 + threadIdx.x;
  if (i8 >= total8) return;
  const int C8 = C >> 3;
  const int c = (int)(i8 % C8) * 8;
  const int64_t r = i8 / C8;
  const int q = (int)(r % keep);
  const int64_t b = r / keep;
  const int64_t dst = (b * blk + q) * C + c;
  const float4* src = reinterpret_cast<const float4*>(frags + i8 * 8);
  const float4 u = src[0], v = src[1];
  float a[8] = {u.x, u.y, u.z, u.w, v.x, v.y, v.z, v.w};
  for (int p = 0; p < n_planes; ++p) {
    uint32_t w[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const __nv_bfloat16 t0 = __float2bfloat16_rn(a[2 * k]), t1 = __float2bfloat16_rn(a[2 * k + 1]);
      a[2 * k] -= __bfloat162float(t0);
      a[2 * k + 1] -= __bfloat162float(t1);
      w[k] = (uint32_t)__bfloat16_as_ushort(t0) | ((uint32_t)__bfloat16_as_ushort(t1) << 16);
    }
    *reinterpret_cast<uint4*>(planes + (int64_t)p * plane_stride + dst) = make_uint4(w[0], w[1], w[2], w[3]);
  }
}

// leaky-ReLU vijp on term planes (n and the plane strides multiples of 8; 128-bit accesses)
__global__ void __launch_bounds__(256)
planes_leaky_vijp_kernel(const __nv_bfloat16* __restrict__ g, int gp, int64_t gs,
                         const uint32_t* __restrict__ words, int act, float slope, int64_t n8,
                         __nv_bfloat16* __restrict__ h, int hp, int64_t hs) {
  const int64_t i8 = (int64_t)blockIdx.x * 256 + threadIdx.x;
  if (i8 >= n8) return;
  const int64_t i = i8 * 8;
  float a[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
  for (int p = gp - 1; p >= 0; --p) {
    float f[8];
    unpack8(*reinterpret_cast<const uint4*>(g + (int64_t)p * gs + i), f);
#pragma unroll
    for (int k = 0; k < 8; ++k) a[k] += f[k];
  }
  if (act == MW_ACT_LEAKY_RELU) {
    const uint32_t bits = words[i >> 5] >> (i & 31);
#pragma unroll
    for (int k = 0; k < 8; ++k)
      if (!((bits >> k) & 1u)) a[k] = a[k] / slope;
  }
  for (int p = 0; p < hp; ++p) {
    uint32_t w[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const __nv_bfloat16 t0 = __float2bfloat16_rn(a[2 * k]), t1 = __float2bfloat16_rn(a[2 * k + 1]);
      a[2 * k] -= __bfloat162float(t0);
      a[2 * k + 1] -= __bfloat162float(t1);
      w[k] = (uint32_t)__bfloat16_as_ushort(t0) | ((uint32_t)__bfloat16_as_ushort(t1) << 16);
    }
    *reinterpret_cast<uint4*>(h + (int64_t)p * hs + i) = make_uint4(w[0], w[1], w[2], w[3]);
  }
}

// ---- products --------------------------------------------------------------------------------
TcConv window_list(const C1& c, bool transpose) {
  TcConv cv;
  cv.mode = TC_CONV_PIXELS; cv.H = 1; cv.W = c.N; cv.C = c.C; cv.stride = 1; cv.Ho = 1; cv.Wo = c.N;
  cv.k = c.k; cv.pad = 1;
  for (int j = 0; j < c.k; ++j) {
    cv.dy[j] = 0;
    cv.dx[j] = (signed char)(transpose ? 1 - j : j - 1);     // x'[i] reads x[i+j-1]; h[i] reads g[i+1-j]
    cv.tb[j] = (signed char)j;
  }
  cv.ntaps = c.k;
  cv.b_tap_rows = transpose ? 1 : 0;
  return cv;
}

TcGemm forward_product(const C1& c, const __nv_bfloat16* x, const __nv_bfloat16* w, const TcEpilogue& e) {
  TcGemm p;
  p.A = pixel_operand(x, c.P / c.C, c.px, c.P, false, c.C);
  p.B.base = w; p.B.rows = c.k * c.C; p.B.cols = c.C; p.B.planes = c.pw; p.B.plane_stride = c.we;
  p.B.mn_major = true;                                        // w[j][ci][co]: K = (j, ci), N = co
  p.M = (int)(c.P / c.C); p.N = c.C; p.K = c.k * c.C;
  p.epi = e;
  p.conv = window_list(c, false);
  return p;
}

TcGemm transpose_product(const C1& c, const __nv_bfloat16* g, const __nv_bfloat16* w, const TcEpilogue& e) {
  TcGemm p;
  p.A = pixel_operand(g, c.P / c.C, c.pg, c.P, false, c.C);
  p.B.base = w; p.B.rows = c.k * c.C; p.B.cols = c.C; p.B.planes = c.pw; p.B.plane_stride = c.we;
  p.B.mn_major = false;                                       // rows (j, c), K = c'
  p.M = (int)(c.P / c.C); p.N = c.C; p.K = c.k * c.C;
  p.epi = e;
  p.conv = window_list(c, true);
  return p;
}

mw_status wgrad(const C1& c, const __nv_bfloat16* x, const __nv_bfloat16* g, int64_t g_stride, float* dw,
                int layer) {
  const int64_t px = c.P / c.C;
  const int slices = conv_wgrad_tensor_slices(px, c.C, c.k);
  const int rows = c.k * c.C;
  TcGemm p;
  p.A = pixel_operand(x, px, c.pwg, c.P, true, c.C);
  p.B = pixel_operand(g, px, c.pwg, g_stride, true, c.C);
  p.M = rows; p.N = c.C; p.K = (int)(px / slices); p.batch = slices;
  p.epi.mode = TC_EPI_PLAIN;
  float* part = c.at<float>(c.lay->cpart);
  p.epi.out_f32 = slices > 1 ? part : dw;
  p.epi.bs_f32 = (int64_t)rows * c.C;
  const float* theta = c.n->apply_params ? (const float*)c.n->apply_params[layer] : nullptr;
  if (theta && slices == 1) { p.epi.alpha = -c.n->apply_lr; p.epi.addend = theta; }
  p.conv.mode = TC_CONV_WGRAD; p.conv.H = 1; p.conv.W = c.N; p.conv.C = c.C; p.conv.stride = 1;
  p.conv.Ho = 1; p.conv.Wo = c.N; p.conv.k = c.k; p.conv.pad = 1; p.conv.one_d = 1;
  MW_TRY(tc_gemm_group(c.cache, &p, 1, c.st, c.s));
  if (slices > 1) MW_TRY(conv_slice_sum(part, (int64_t)rows * c.C, slices, dw, theta, c.n->apply_lr, c.s));
  return MW_OK;
}

// per-step preparation: kernel term planes; for Moonwalk W0^-1 and the folded taps
mw_status prep(const C1& c, const void* const* params, bool inverse) {
  const Layout& lay = *c.lay;
  const int C = c.C;
  if (!c.bf16)
    for (int l = 0; l < c.L; ++l)
      MW_TRY(split_planes((const float*)params[l], c.we, c.at<__nv_bfloat16>(lay.cw[l]), 3, c.we, c.s));
  if (!inverse) return MW_OK;
  static bool attr_done = false;
  if (!attr_done) {
    MW_CUDA_OK(cudaFuncSetAttribute(tri_inverse_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    (int)(sizeof(double) * 256 * kTriCols)));
    MW_CUDA_OK(cudaFuncSetAttribute(tri_inverse_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    (int)(sizeof(double) * 256 * kTriCols)));
    attr_done = true;
  }
  float* inv = c.at<float>(lay.cwinv_f32);        // [kSmallBatch][C*C]
  float* fold = c.at<float>(lay.cwhat_f32);       // [kSmallBatch][C][(k-1)*C]
  const int64_t fe = (int64_t)C * (c.k - 1) * C;
  for (int l0 = 0; l0 < c.L; l0 += kSmallBatch) {
    const int G = c.L - l0 < kSmallBatch ? c.L - l0 : kSmallBatch;
    SmallBatch ws{};
    for (int g = 0; g < G; ++g) ws.p[g] = params[l0 + g];
    const dim3 tg(G, (C + kTriCols - 1) / kTriCols);
    const size_t tsm = sizeof(double) * C * kTriCols;
    if (c.bf16) {
      tri_inverse_kernel<__nv_bfloat16><<<tg, kTriCols, tsm, c.s>>>(ws, C, inv, c.st, l0);
      MW_TRY(launch_ok());
      fold1d_kernel<__nv_bfloat16><<<dim3(C, c.k - 1, G), 256, 0, c.s>>>(ws, inv, C, c.k, fold);
    } else {
      tri_inverse_kernel<float><<<tg, kTriCols, tsm, c.s>>>(ws, C, inv, c.st, l0);
      MW_TRY(launch_ok());
      fold1d_kernel<float><<<dim3(C, c.k - 1, G), 256, 0, c.s>>>(ws, inv, C, c.k, fold);
    }
    MW_TRY(launch_ok());
    for (int g = 0; g < G; ++g) {
      MW_TRY(split_planes(inv + (int64_t)g * C * C, (int64_t)C * C, c.at<__nv_bfloat16>(lay.cwinv[l0 + g]), c.pg,
                          (int64_t)C * C, c.s));
      MW_TRY(split_planes(fold + (int64_t)g * fe, fe, c.at<__nv_bfloat16>(lay.cwhat[l0 + g]), c.pg, fe, c.s));
    }
  }
  return MW_OK;
}

__nv_bfloat16* x_planes(const C1& c, int l) {
  // a bf16 input is its own (single) term plane
  if (l == 0 && c.bf16) return const_cast<__nv_bfloat16*>(static_cast<const __nv_bfloat16*>(c.x));
  return c.at<__nv_bfloat16>(l == 0 ? c.lay->xp[0] : c.lay->xp[1 + ((l - 1) & 1)]);
}

const __nv_bfloat16* w_planes(const C1& c, int l) {
  return c.bf16 ? static_cast<const __nv_bfloat16*>(c.params[l]) : c.at<__nv_bfloat16>(c.lay->cw[l]);
}

mw_status forward_pass(const C1& c, const void* const* params, const void* x, bool store_acts) {
  const Layout& lay = *c.lay;
  MW_TRY(prep(c, params, !store_acts));
  if (!c.bf16) MW_TRY(split_planes((const float*)x, c.P, x_planes(c, 0), 3, c.P, c.s));
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
    if (!last) { e.planes = xout; e.n_planes = c.px; e.plane_stride = c.P; }
    else e.out_f32 = c.at<float>(lay.cxf);
    TcGemm g = forward_product(c, xin, w_planes(c, l), e);
    MW_TRY(tc_gemm_group(c.cache, &g, 1, c.st, c.s));
    xin = xout;
  }
  return MW_OK;
}

mw_status loss_top(const C1& c, const void* target, double* loss_out) {
  const Layout& lay = *c.lay;
  const int l = c.L - 1;
  const mw_layer_desc& ld = c.n->layers[l];
  const int64_t rows = c.P / c.C;
  float* h = c.at<float>(lay.cot[0]);
  MW_TRY(loss_cotangent<float>(c.at<float>(lay.cxf), target, rows, c.C, c.n->opts.loss, h,
                               c.at<double>(lay.partials), loss_out, c.s));
  const float* src = h;
  if (ld.act != MW_ACT_NONE) {
    float* g = c.at<float>(lay.cot[1]);
    MW_TRY(scale_by_mask<float>(h, c.at<uint32_t>(lay.mask[l]), rows, c.C, ld.act, ld.slope, g, c.s));
    src = g;
  }
  return split_planes(src, c.P, c.at<__nv_bfloat16>(lay.hp[0]), c.pg, c.P, c.s);
}

int64_t frag_elems(const C1& c) { return c.P / c.blk * (c.k - 1); }

mw_status backward_pass(const C1& c, void* g0, void* const* dW, bool moonwalk) {
  const Layout& lay = *c.lay;
  int cur = 0;
  for (int l = c.L - 1; l >= 0; --l) {
    const __nv_bfloat16* gz = c.at<__nv_bfloat16>(lay.hp[cur]);
    if (moonwalk) {
      // fragmental checkpoint of this layer's g_z: the first k - 1 positions of every block
      const int64_t total8 = frag_elems(c) / 8;
      frag_gather_kernel<<<(unsigned)((total8 + 255) / 256), 256, 0, c.s>>>(
          gz, c.pg, c.P, c.C, c.blk, c.k - 1, total8, c.at<float>(lay.cfrag[l]));
      MW_TRY(launch_ok());
    }
    if (dW && dW[l]) {
      const __nv_bfloat16* xl = l == 0 ? x_planes(c, 0) : c.at<__nv_bfloat16>(lay.stored_act[l]);
      MW_TRY(wgrad(c, xl, gz, c.P, (float*)dW[l], l));
    }
    if (l == 0 && !g0) break;
    TcEpilogue e;
    e.mode = TC_EPI_BWD;
    if (l == 0) {
      e.out_f32 = (float*)g0;
    } else {
      const mw_layer_desc& below = c.n->layers[l - 1];
      if (moonwalk && is_reseed(c.n, l)) e.out_f32 = c.at<float>(lay.reseed[l]);
      e.act = below.act;
      e.slope = (float)below.slope;
      e.mask = c.at<uint32_t>(lay.mask[l - 1]);
      e.planes = c.at<__nv_bfloat16>(lay.hp[cur ^ 1]);
      e.n_planes = c.pg;
      e.plane_stride = c.P;
    }
    TcGemm g = transpose_product(c, gz, w_planes(c, l), e);
    MW_TRY(tc_gemm_group(c.cache, &g, 1, c.st, c.s));
    cur ^= 1;
  }
  return MW_OK;
}

}  // namespace

bool conv1d_tensor_supported(const mw_net* n) {
  if ((n->opts.prec != MW_F32 && n->opts.prec != MW_BF16_F32ACC) || n->opts.loss == MW_LOSS_XENT_MEAN) return false;
  const mw_layer_desc& d0 = n->layers[0];
  const int blk = n->opts.frag_block;
  if (d0.C_in < 64 || d0.C_in % 64 != 0 || d0.C_in > 256) return false;
  if (d0.W % 128 != 0 || blk < d0.k - 1 || blk < 2 || d0.W % blk != 0 || blk > 64) return false;
  for (int l = 0; l < n->L; ++l) {
    const mw_layer_desc& d = n->layers[l];
    if (d.kind != MW_CONV1D || d.C_in != d0.C_in || d.C_out != d0.C_in || d.W != d0.W || d.H != 1) return false;
    if (d.k != 3 || d.stride != 1 || d.pad != 1) return false;
    if (d.act == MW_ACT_RELU || (d.act == MW_ACT_LEAKY_RELU && !(d.slope != 0.0))) return false;
  }
  if ((int64_t)n->B * d0.W >= ((int64_t)1 << 31) / d0.C_in) return false;
  return true;
}

void conv1d_tensor_layout(mw_net* n, bool backprop, Layout& lay, size_t start) {
  struct B2 {
    size_t cur;
    Region take(size_t bytes) {
      Region r; r.off = cur; r.bytes = bytes; cur = align_up(cur + bytes, 256); return r;
    }
  } b{start};
  const mw_layer_desc& d = n->layers[0];
  const int L = n->L, C = d.C_in, k = d.k;
  const size_t P = (size_t)n->B * d.W * C;
  const size_t we = (size_t)k * C * C;
  lay.cfrag.assign(L, Region());
  if (!backprop) {
    // fragmental checkpoints survive between the phases
    const size_t fe = P / n->opts.frag_block * (k - 1);
    for (int l = 0; l < L; ++l) lay.cfrag[l] = b.take(4 * fe);
    lay.residual += b.cur - start;
  }
  for (int i = 0; i < 2; ++i) lay.cot[i] = b.take(4 * P);
  lay.cxf = b.take(4 * P);
  const bool bf16 = n->opts.prec == MW_BF16_F32ACC;
  const size_t px = bf16 ? 1 : 3, pg = bf16 ? 2 : 3;
  lay.xp[0] = b.take(bf16 ? 256 : 2 * 3 * P);
  for (int i = 1; i < 3; ++i) lay.xp[i] = b.take(2 * px * P);
  for (int i = 0; i < 2; ++i) lay.hp[i] = b.take(2 * pg * P);
  lay.cw.resize(L); lay.cwinv.resize(L); lay.cwhat.resize(L);
  for (int l = 0; l < L; ++l) lay.cw[l] = b.take(bf16 ? 256 : 2 * 3 * we);
  lay.cpart = b.take(4 * (size_t)conv_wgrad_tensor_slices((int64_t)n->B * d.W, C, k) * we);
  if (!backprop) {
    lay.cg[0] = b.take(2 * pg * P);                     // g_z rebuilt block by block
    lay.chpf = b.take(4 * P);                           // c = h W0^-T
    for (int l = 0; l < L; ++l) {
      lay.cwinv[l] = b.take(2 * pg * (size_t)C * C);
      lay.cwhat[l] = b.take(2 * pg * (size_t)C * (k - 1) * C);
    }
    lay.cwinv_f32 = b.take(4 * (size_t)C * C * kSmallBatch);
    lay.cwhat_f32 = b.take(4 * (size_t)C * (k - 1) * C * kSmallBatch);
  }
  lay.total = b.cur;
}

mw_status conv1d_tensor_input_cotangent(mw_net* n, const void* const* params, const void* x,
                                        const void* target, void* g0, double* loss_out, void* ws,
                                        cudaStream_t s) {
  const Layout& lay = n->mwl;
  C1 c = make_c1(n, lay, ws, s, params, x);
  MW_CUDA_OK(cudaMemsetAsync(at<char>(ws, lay.status), 0, 256, s));
  MW_TRY(forward_pass(c, params, x, false));          // Phase I (+ per-step preparation)
  MW_TRY(loss_top(c, target, loss_out));
  return backward_pass(c, g0, nullptr, true);          // Phase II
}

mw_status conv1d_tensor_forward_sweep(mw_net* n, const void* const* params, const void* x,
                                      const void* g0, void* const* dW, void* ws, cudaStream_t s) {
  // the term planes of an fp32 x (xp[0]) are still those Phase I made
  const Layout& lay = n->mwl;
  C1 c = make_c1(n, lay, ws, s, params, x);
  const int L = c.L, C = c.C, blk = c.blk, k = c.k;
  const int64_t rows = c.P / C;                       // samples * N
  MW_TRY(split_planes((const float*)g0, c.P, c.at<__nv_bfloat16>(lay.hp[0]), c.pg, c.P, s));
  __nv_bfloat16* gzp = c.at<__nv_bfloat16>(lay.cg[0]);
  float* cst = c.at<float>(lay.chpf);
  for (int l = 0; l < L; ++l) {
    const mw_layer_desc& ld = n->layers[l];
    uint32_t* words = c.at<uint32_t>(lay.mask[l]);
    const __nv_bfloat16* xin = x_planes(c, l);
    const __nv_bfloat16* hin = c.at<__nv_bfloat16>(lay.hp[l & 1]);
    __nv_bfloat16* hout = c.at<__nv_bfloat16>(lay.hp[(l + 1) & 1]);
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
      e.planes = x_planes(c, l + 1); e.n_planes = c.px; e.plane_stride = c.P;
      TcGemm p = forward_product(c, xin, w_planes(c, l), e);
      MW_TRY(tc_gemm_group(c.cache, &p, 1, c.st, s));
    }
    if (dW[l] || want_h) {
      {
        // c = h W0^-T at every position
        TcGemm p;
        p.A = pixel_operand(hin, rows, c.pg, c.P, false, C);
        p.B.base = c.at<__nv_bfloat16>(lay.cwinv[l]); p.B.rows = C; p.B.cols = C; p.B.planes = c.pg;
        p.B.plane_stride = (int64_t)C * C; p.B.mn_major = false;
        p.M = (int)rows; p.N = C; p.K = C;
        p.epi.mode = TC_EPI_PLAIN;
        p.epi.out_f32 = cst;
        MW_TRY(tc_gemm_group(c.cache, &p, 1, c.st, s));
      }
      {
        const int64_t total8 = frag_elems(c) / 8;
        frag_scatter_kernel<<<(unsigned)((total8 + 255) / 256), 256, 0, s>>>(
            c.at<float>(lay.cfrag[l]), C, blk, k - 1, total8, gzp, c.pg, c.P);
        MW_TRY(launch_ok());
      }
      // position t of every block from positions t-2, t-1 (adjacent in memory: K = 2 C)
      for (int t = k - 1; t < blk; ++t) {
        TcGemm p;
        p.A.base = gzp + (int64_t)(t - (k - 1)) * C;
        p.A.rows = (int)(rows / blk); p.A.cols = (k - 1) * C; p.A.ld = (int64_t)blk * C;
        p.A.planes = c.pg; p.A.plane_stride = c.P; p.A.mn_major = false;
        p.B.base = c.at<__nv_bfloat16>(lay.cwhat[l]); p.B.rows = C; p.B.cols = (k - 1) * C; p.B.planes = c.pg;
        p.B.plane_stride = (int64_t)C * (k - 1) * C; p.B.mn_major = false;
        p.M = (int)(rows / blk); p.N = C; p.K = (k - 1) * C;
        TcEpilogue& e = p.epi;
        e.mode = TC_EPI_PLAIN;
        e.alpha = -1.f;
        e.addend = cst + (int64_t)(t - 1) * C;
        e.planes = gzp + (int64_t)t * C; e.n_planes = c.pg; e.plane_stride = c.P;
        e.ld = (int64_t)blk * C;
        MW_TRY(tc_gemm_group(c.cache, &p, 1, c.st, s));
      }
      if (want_h) {
        planes_leaky_vijp_kernel<<<(unsigned)((c.P / 8 + 255) / 256), 256, 0, s>>>(
            gzp, c.pg, c.P, words, ld.act, (float)ld.slope, c.P / 8, hout, c.pg, c.P);
        MW_TRY(launch_ok());
      }
    }
    if (reseed_next)
      MW_TRY(split_planes(c.at<float>(lay.reseed[l + 1]), c.P, hout, c.pg, c.P, s));
    if (dW[l]) {
      MW_TRY(wgrad(c, xin, gzp, c.P, (float*)dW[l], l));
      if (n->apply_params)   // the zeros of tap 0 are structure, not parameters
        MW_TRY(conv_zero_fixed_entries((float*)dW[l], 0, C, s));
    }
  }
  return MW_OK;
}

mw_status conv1d_tensor_backprop(mw_net* n, const void* const* params, const void* x,
                                 const void* target, void* const* dW, double* loss_out, void* ws,
                                 cudaStream_t s) {
  const Layout& lay = n->bpl;
  C1 c = make_c1(n, lay, ws, s, params, x);
  MW_CUDA_OK(cudaMemsetAsync(at<char>(ws, lay.status), 0, 256, s));
  MW_TRY(forward_pass(c, params, x, true));
  MW_TRY(loss_top(c, target, loss_out));
  return backward_pass(c, nullptr, dW, false);
}

}  // namespace mw
