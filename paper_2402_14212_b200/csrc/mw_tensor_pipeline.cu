// Tensor-core pipelines of the three calls for dense nets (MW_F32 and MW_BF16_F32ACC).
//
// Every matrix product runs on the persistent tcgen05 kernel (mw_tc_gemm.cu) with the step's
// elementwise work fused into its epilogue:
//   Phase I    z = x W^T          -> sign words + x_l term planes                (Section 4.1)
//   Phase II   h_{l-1} = g_z W    -> cotangent checkpoint (fp32) and ReLU fragment stream where
//                                    the layer below asks for them + next g_z term planes
//   prep       W^-1 by Newton-Schulz, X <- X + X (I - W X), low precision first
//   sweep      one launch per layer (Algorithm 1) carrying three independent products:
//              recompute x_{l+1} (as Phase I, reading the stored sign words),
//              g_z = h_l W^-1 with the activation's vijp behind it: h_{l+1} term planes (leaky:
//              divide by the slope; ReLU: dead units take their fragment back) + g_z term planes
//              (Eq. "h_i"), and the weight vjp of the layer before, dW = g_z^T x (Eq. "g_i").
// Products with too few output tiles for the machine are cut along K (deterministic meeting in
// the workspace).
#include <cstring>

#include "mw_tc_gemm.cuh"
#include "mw_tensor.cuh"

namespace mw {

namespace {

struct Prec {
  int px;    // activation / weight terms (recompute, Phase I)
  int ph;    // cotangent-chain terms (h and W^-1 in the dense vijp)
  int pg2;   // g_z terms in Phase II
  int pgw;   // g_z terms in the weight vjp
  int pw;    // weight terms
  int pxw;   // activation terms in the weight vjp
};

// The chains (activations forward, cotangents backward and forward again) carry every term: an
// error made there is passed on, and the vijp recursion amplifies it.  The weight vjp ends in
// dW_l and feeds nothing, so two terms per operand (2^-17 relative) are enough for it.
Prec prec_of(const mw_net* n) {
  if (n->opts.prec == MW_F32) return Prec{3, 3, 3, 2, 3, 2};
  return Prec{1, 2, 2, 1, 1, 1};
}

struct NsStep { int pr, pu; };   // terms in the residual product (W, X) and the update (X, R)

int ns_schedule(const mw_net* n, NsStep* out) {
  int cnt;
  if (n->opts.prec == MW_F32) {
    // residual ||I - W X|| per step on near-orthogonal weights: 1.5e-1, 2e-2, 5e-4 -> 2e-7
    const NsStep d[] = {{1, 1}, {2, 1}, {3, 2}};
    cnt = 3;
    for (int i = 0; i < cnt; ++i) out[i] = d[i];
  } else {
    // residual 6e-2 -> 4e-3 -> 2e-5, the resolution of the two-term cotangent chain
    const NsStep d[] = {{1, 1}, {2, 1}};
    cnt = 2;
    for (int i = 0; i < cnt; ++i) out[i] = d[i];
  }
  const int want = n->opts.inverse_iters;
  if (want > 0) {
    // more steps repeat the most accurate one; fewer drop the cheap leading ones last
    if (want > 16) return -1;
    NsStep full[16];
    const NsStep last = out[cnt - 1];
    if (want >= cnt) {
      for (int i = 0; i < cnt; ++i) full[i] = out[i];
      for (int i = cnt; i < want; ++i) full[i] = last;
    } else {
      for (int i = 0; i < want - 1; ++i) full[i] = out[i];
      full[want - 1] = last;
    }
    for (int i = 0; i < want; ++i) out[i] = full[i];
    cnt = want;
  }
  return cnt;
}

constexpr int kMaxGroup = 32;     // layers whose inverses are computed together
struct PtrBatch { const void* p[kMaxGroup]; };

// sum of squares of each W of the group: kFrobBlocks partial sums per matrix, then one thread
// per matrix folds them in fixed order into the Newton-Schulz start scale c = n / ||W||_F^2
constexpr int kFrobBlocks = 128;
template <typename TW>
__global__ void __launch_bounds__(256)
frob_partial_kernel(PtrBatch Ws, int64_t n2, double* __restrict__ partial) {
  __shared__ double red[256];
  const TW* W = static_cast<const TW*>(Ws.p[blockIdx.y]);
  double a = 0.0;
  for (int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x; i < n2; i += (int64_t)gridDim.x * 256) {
    const double v = (double)to_f32(W[i]);
    a += v * v;
  }
  red[threadIdx.x] = a;
  __syncthreads();
  for (int o = 128; o; o >>= 1) {
    if (threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o];
    __syncthreads();
  }
  if (threadIdx.x == 0) partial[blockIdx.y * kFrobBlocks + blockIdx.x] = red[0];
}
__global__ void frob_final_kernel(const double* __restrict__ partial, int group, int n,
                                  float* __restrict__ c_out) {
  const int g = threadIdx.x;
  if (g < group) {
    double a = 0.0;
    for (int i = 0; i < kFrobBlocks; ++i) a += partial[g * kFrobBlocks + i];
    c_out[g] = a > 0.0 ? (float)((double)n / a) : 0.f;
  }
}

// X0 = c W^T through a 64 x 64 shared tile, written once as fp32 (the iteration's running sum) and
// as its first `planes` bf16 term planes (the first step's operand); blockIdx.z = matrix of the
// group.  Matrix g writes X + g*n*n and planes P + g*group_stride + p*n*n.
template <typename TW>
__global__ void __launch_bounds__(256)
x0_kernel(PtrBatch Ws, int n, const float* __restrict__ c, float* __restrict__ X,
          __nv_bfloat16* __restrict__ P, int planes, int64_t group_stride) {
  __shared__ float tile[64][65];
  const TW* W = static_cast<const TW*>(Ws.p[blockIdx.z]);
  const int64_t nn = (int64_t)n * n;
  float* Xg = X + (int64_t)blockIdx.z * nn;
  __nv_bfloat16* Pg = P + (int64_t)blockIdx.z * group_stride;
  const int bx = blockIdx.x * 64, by = blockIdx.y * 64;
  const int tx = threadIdx.x & 63, ty = threadIdx.x >> 6;      // 64 columns x 4 rows per pass
  for (int r = ty; r < 64; r += 4) tile[r][tx] = to_f32(W[(int64_t)(by + r) * n + bx + tx]);
  __syncthreads();
  const float cc = c[blockIdx.z];
  // every thread: 4 consecutive columns of one row of the transposed tile
  const int q = (threadIdx.x & 15) * 4;
  for (int r = threadIdx.x >> 4; r < 64; r += 16) {
    float v[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) v[j] = cc * tile[q + j][r];
    const int64_t at = (int64_t)(bx + r) * n + by + q;
    *reinterpret_cast<float4*>(Xg + at) = make_float4(v[0], v[1], v[2], v[3]);
    for (int p = 0; p < planes; ++p) {
      __nv_bfloat16 b[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        b[j] = __float2bfloat16_rn(v[j]);
        v[j] -= __bfloat162float(b[j]);
      }
      uint2 pk;
      pk.x = (uint32_t)__bfloat16_as_ushort(b[0]) | ((uint32_t)__bfloat16_as_ushort(b[1]) << 16);
      pk.y = (uint32_t)__bfloat16_as_ushort(b[2]) | ((uint32_t)__bfloat16_as_ushort(b[3]) << 16);
      *reinterpret_cast<uint2*>(Pg + (int64_t)p * nn + at) = pk;
    }
  }
}

// fp32 weights of the group -> 3 bf16 term planes each (dst + g*3*n2)
__global__ void __launch_bounds__(256)
split_weights_kernel(PtrBatch Ws, int64_t n4, int64_t n2, __nv_bfloat16* __restrict__ dst0) {
  const float* src = static_cast<const float*>(Ws.p[blockIdx.y]);
  __nv_bfloat16* dst = dst0 + (int64_t)blockIdx.y * 3 * n2;
  for (int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x; i < n4; i += (int64_t)gridDim.x * 256) {
    float4 v = reinterpret_cast<const float4*>(src)[i];
    float r[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int p = 0; p < 3; ++p) {
      __nv_bfloat16 b[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        b[j] = __float2bfloat16_rn(r[j]);
        r[j] -= __bfloat162float(b[j]);
      }
      uint2 pk;
      pk.x = (uint32_t)__bfloat16_as_ushort(b[0]) | ((uint32_t)__bfloat16_as_ushort(b[1]) << 16);
      pk.y = (uint32_t)__bfloat16_as_ushort(b[2]) | ((uint32_t)__bfloat16_as_ushort(b[3]) << 16);
      reinterpret_cast<uint2*>(dst + (int64_t)p * n2)[i] = pk;
    }
  }
}

// One CTA per matrix: adds the `slots` pieces of ||I - W X||_F^2 that the residual product's
// epilogue warps left (always in the same order, so the decision does not depend on scheduling)
// and reports the layer when the rms singular value of the residual exceeds `limit` (whole =
// 1: when its Frobenius norm does, which bounds the LARGEST singular value: a refreshed inverse
// follows a training step, whose change of W is far from spread evenly over the directions).
__global__ void __launch_bounds__(256)
residual_gate_kernel(const double* __restrict__ pieces, int64_t stride, int64_t slots, int n,
                     double limit, DeviceStatus* st, int layer0, int whole = 0) {
  __shared__ double red[256];
  const double* mine = pieces + (int64_t)blockIdx.x * stride;
  double a = 0.0;
  for (int64_t i = threadIdx.x; i < slots; i += 256) a += mine[i];
  red[threadIdx.x] = a;
  __syncthreads();
  for (int o = 128; o; o >>= 1) {
    if (threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o];
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    const double r = sqrt(whole ? red[0] : red[0] / (double)n);   // rms (or root sum) of the singular values of I - W X
    if (!(r <= limit))
      record_error(st, MW_ERR_NOT_SUBMERSIVE, (unsigned)(layer0 + blockIdx.x), __float_as_uint((float)r),
                   whole ? 4u : 3u, 0u);
  }
}

// slots of ||R||_F^2 pieces per matrix, for the narrowest tile a residual product may use
size_t gate_slots(int d) { return (size_t)(d / 128 + 1) * (d / 64) * 4; }

// layers per Newton-Schulz group: enough 128x128 tiles for several waves of the 148 SMs
int ns_group(const mw_net* n) {
  if (!n->opts.resident_inverse) return 1;
  const int d = n->layers[0].n_in;
  const int tiles = ((d + 127) / 128) * ((d + 127) / 128);
  int g = 2048 / tiles;
  if (g < 1) g = 1;
  if (g > kMaxGroup) g = kMaxGroup;
  if (g > n->L) g = n->L;
  return g;
}

TcOperand operand(const void* base, int rows, int cols, int planes, bool mn) {
  TcOperand o;
  o.base = base;
  o.rows = rows;
  o.cols = cols;
  o.planes = planes;
  o.plane_stride = (int64_t)rows * cols;
  o.mn_major = mn;
  return o;
}

struct Ctx {
  mw_net* n;
  const Layout* lay;
  void* ws;
  cudaStream_t s;
  TcMapCache* cache;
  DeviceStatus* st;
  Prec pr;
  int B, dim;          // batch, width
  int64_t bn;          // B * width
  int64_t nn;          // width^2
  // rings of the sweep: x_l lives in xp[l % nx], g_z of layer l in gzp[l % ngz].  3 and 2 slots
  // are what one launch per layer needs; the chained sweep runs several layers at once and uses
  // 5 and 4, so that a slot is reused only by a product three layers behind its last reader
  int nx = 3, ngz = 2;
  template <typename T> T* at(const Region& r) const { return mw::at<T>(ws, r); }
};

Ctx make_ctx(mw_net* n, const Layout& lay, void* ws, cudaStream_t s) {
  Ctx c;
  c.n = n; c.lay = &lay; c.ws = ws; c.s = s;
  c.cache = static_cast<TensorState*>(n->tc)->cache;
  c.st = status_of(ws, lay);
  c.pr = prec_of(n);
  c.B = n->B;
  c.dim = n->layers[0].n_in;
  c.bn = (int64_t)c.B * c.dim;
  c.nn = (int64_t)c.dim * c.dim;
  return c;
}

// weight operand of layer l (MW_F32: split planes in the workspace, made here when `make`;
// bf16: the caller's array itself)
mw_status weight_planes(const Ctx& c, int l, const void* W, bool make, const __nv_bfloat16** out) {
  if (c.n->opts.lu_param) {
    // the parameters are the factors: the planes of W = L U were made by lu_prepare
    *out = c.at<__nv_bfloat16>(c.lay->w_planes[l]);
    return MW_OK;
  }
  if (c.n->opts.prec == MW_F32) {
    __nv_bfloat16* p = c.at<__nv_bfloat16>(c.lay->w_planes[l]);
    if (make) MW_TRY(split_planes((const float*)W, c.nn, p, 3, c.nn, c.s));
    *out = p;
  } else {
    *out = (const __nv_bfloat16*)W;
  }
  return MW_OK;
}

// W^-1 of layers [l0, l0+G) into their inverse regions as `ph` term planes (row-major
// X = W^-1), all G layers advancing together in batched launches.  Also leaves the split weight
// planes of those layers in w_planes (MW_F32).
mw_status newton_schulz_single(const Ctx& c, int l, const void* const* params);

mw_status newton_schulz_group(const Ctx& c, int l0, int G, const void* const* params) {
  const Layout& lay = *c.lay;
  const int d = c.dim;
  const bool f32 = c.n->opts.prec == MW_F32;
  // bf16 layers whose products fill the GPU on their own gain nothing from batching: one at a time,
  // with the cheaper product list of newton_schulz_single
  if (!f32 && (G == 1 || d >= 2048)) {
    for (int g = 0; g < G; ++g) MW_TRY(newton_schulz_single(c, l0 + g, params));
    return MW_OK;
  }
  float* X = c.at<float>(lay.ns_x);                             // [G][n*n]
  __nv_bfloat16* Rp = c.at<__nv_bfloat16>(lay.ns_r);            // [G][3][n*n]
  __nv_bfloat16* Xp[2] = {Rp + (int64_t)3 * G * c.nn, Rp + (int64_t)6 * G * c.nn};
  char* sc = c.at<char>(lay.inv_scratch);
  float* cscale = reinterpret_cast<float*>(sc + 8 * kMaxGroup); // [G]
  double* fpart = reinterpret_cast<double*>(sc + 12 * kMaxGroup + 64);   // [G][kFrobBlocks]
  double* sumsq = c.at<double>(lay.ns_sumsq);                   // [G][gate_slots]
  __nv_bfloat16* dst = c.at<__nv_bfloat16>(lay.inv[l0]);
  const int64_t dst_stride = G > 1 ? (int64_t)(lay.inv[l0 + 1].off - lay.inv[l0].off) / 2 : 0;

  PtrBatch wp{};
  for (int g = 0; g < G; ++g) wp.p[g] = params[l0 + g];
  // the weight operand of the residual product
  const __nv_bfloat16* Wbase;
  int w_batch_planes;
  if (f32) {
    __nv_bfloat16* w0 = c.at<__nv_bfloat16>(lay.w_planes[l0]);
    int64_t bx = (c.nn / 4 + 255) / 256;
    if (bx > 64) bx = 64;
    split_weights_kernel<<<dim3((unsigned)bx, (unsigned)G), 256, 0, c.s>>>(wp, c.nn / 4, c.nn, w0);
    MW_TRY(launch_ok());
    Wbase = w0;
    w_batch_planes = G > 1 ? (int)((lay.w_planes[l0 + 1].off - lay.w_planes[l0].off) / (2 * c.nn)) : 3;
  } else if (G == 1) {
    Wbase = (const __nv_bfloat16*)params[l0];
    w_batch_planes = 1;
  } else {
    __nv_bfloat16* stage = c.at<__nv_bfloat16>(lay.ns_w);        // [G][n*n] bf16 copies
    for (int g = 0; g < G; ++g)
      MW_CUDA_OK(cudaMemcpyAsync(stage + (int64_t)g * c.nn, params[l0 + g], 2 * c.nn,
                                 cudaMemcpyDeviceToDevice, c.s));
    Wbase = stage;
    w_batch_planes = 1;
  }

  NsStep sched[16];
  const int steps = ns_schedule(c.n, sched);
  if (steps < 1) return MW_ERR_INVALID_ARG;
  const int first = sched[0].pr > sched[0].pu ? sched[0].pr : sched[0].pu;
  if (f32) {
    frob_partial_kernel<float><<<dim3(kFrobBlocks, G), 256, 0, c.s>>>(wp, c.nn, fpart);
    frob_final_kernel<<<1, kMaxGroup, 0, c.s>>>(fpart, G, d, cscale);
    x0_kernel<float><<<dim3(d / 64, d / 64, G), 256, 0, c.s>>>(wp, d, cscale, X, Xp[0], first, 3 * c.nn);
  } else {
    frob_partial_kernel<__nv_bfloat16><<<dim3(kFrobBlocks, G), 256, 0, c.s>>>(wp, c.nn, fpart);
    frob_final_kernel<<<1, kMaxGroup, 0, c.s>>>(fpart, G, d, cscale);
    x0_kernel<__nv_bfloat16><<<dim3(d / 64, d / 64, G), 256, 0, c.s>>>(wp, d, cscale, X, Xp[0], first, 3 * c.nn);
  }
  MW_TRY(launch_ok(3));
  int cur = 0;
  for (int it = 0; it < steps; ++it) {
    const bool last = it + 1 == steps;
    const int pw = c.pr.pw < sched[it].pr ? c.pr.pw : sched[it].pr;
    // R = I - W X
    TcEpilogue er;
    er.mode = TC_EPI_RESID;
    er.planes = Rp; er.n_planes = sched[it].pu; er.plane_stride = c.nn; er.bs_planes = 3 * c.nn;
    if (last) { er.sumsq = sumsq; er.bs_sumsq = (int64_t)gate_slots(d); }
    TcOperand wa = operand(Wbase, d, d, pw, false);
    wa.batch_planes = w_batch_planes;
    TcOperand xb = operand(Xp[cur], d, d, sched[it].pr, true);
    xb.batch_planes = 3;
    MW_TRY(tc_gemm(c.cache, wa, xb, d, d, d, er, c.st, c.s, G));
    if (last) {
      // the update squares this residual: gate on it so a diverging layer is reported
      const double limit = f32 ? 2e-3 : 2e-2;
      residual_gate_kernel<<<G, 256, 0, c.s>>>(sumsq, (int64_t)gate_slots(d),
                                               (int64_t)tc_sumsq_slots(pw, sched[it].pr, d, d, tc_pair_ok(pw, sched[it].pr, d, d)), d, limit,
                                               c.st, l0);
      MW_TRY(launch_ok());
    }
    // X' = X + X R
    int next_terms = c.pr.ph;
    if (!last) next_terms = sched[it + 1].pr > sched[it + 1].pu ? sched[it + 1].pr : sched[it + 1].pu;
    TcEpilogue eu;
    eu.mode = TC_EPI_PLAIN;
    eu.addend = X;
    eu.out_f32 = last ? nullptr : X;
    eu.bs_f32 = c.nn;
    eu.planes = last ? dst : Xp[cur ^ 1];
    eu.n_planes = next_terms;
    eu.plane_stride = c.nn;
    eu.bs_planes = last ? dst_stride : 3 * c.nn;
    TcOperand xa = operand(Xp[cur], d, d, sched[it].pu, false);
    xa.batch_planes = 3;
    TcOperand rb = operand(Rp, d, d, sched[it].pu, true);
    rb.batch_planes = 3;
    MW_TRY(tc_gemm(c.cache, xa, rb, d, d, d, eu, c.st, c.s, G));
    cur ^= 1;
  }
  return MW_OK;
}

// x0 (caller's array) as a K-major / MN-major operand base with px terms
mw_status input_planes(const Ctx& c, const void* x, const __nv_bfloat16** out) {
  if (c.n->opts.prec == MW_F32) {
    __nv_bfloat16* p = c.at<__nv_bfloat16>(c.lay->xp[0]);
    MW_TRY(split_planes((const float*)x, c.bn, p, c.pr.px, c.bn, c.s));
    *out = p;
  } else {
    *out = (const __nv_bfloat16*)x;
  }
  return MW_OK;
}

// one product of a launch; `slot` picks the K-split meeting place (products of one launch must
// use different slots)
TcGemm product(const Ctx& c, const TcOperand& A, const TcOperand& B, int M, int N, int K,
               const TcEpilogue& e, int slot) {
  TcGemm g;
  g.A = A; g.B = B; g.M = M; g.N = N; g.K = K; g.epi = e;
  g.split_k = tc_auto_split(A.planes, B.planes, M, N, K, 1);
  if (g.split_k > 1) g.split_scratch = c.at<char>(c.lay->split[slot]);
  return g;
}

mw_status run(const Ctx& c, const TcGemm* g, int count) {
  return tc_gemm_group(c.cache, g, count, c.st, c.s);
}

mw_status clear_split_counters(const Ctx& c) {
  for (int i = 0; i < 3; ++i)
    if (c.lay->split[i].bytes)
      MW_CUDA_OK(cudaMemsetAsync(c.at<char>(c.lay->split[i]), 0, kTcSplitCounterBytes, c.s));
  return MW_OK;
}

// ---- LU-parameterised dense layers -------------------------------------------------------------
// params[l] holds L strictly below the diagonal (unit diagonal implied) and U on and above it;
// W = L U.  What Newton-Schulz does for a free W is done here exactly, from the structure:
// L^-1 and U^-1 by block substitution (diagonal blocks of 128 inverted on the CUDA cores in
// fp64, then [[A, 0], [C, D]]^-1 = [[A^-1, 0], [-D^-1 C A^-1, D^-1]] level by level on the
// tensor cores), W^-1 = U^-1 L^-1 and W = L U as two more products, everything as three bf16
// term planes (fp32-accurate).  The gradient of W that the sweep forms is mapped to the factors
// by the chain rule: dJ/dL = G U^T below the diagonal, dJ/dU = L^T G on and above it.
constexpr int kLuBlock = 128;
constexpr int kLuProgEntries = 256;   // products of one factor-preparation program

__device__ __forceinline__ void split3(float v, __nv_bfloat16* p, int64_t stride) {
  const __nv_bfloat16 a = __float2bfloat16_rn(v);
  const float r1 = v - __bfloat162float(a);
  const __nv_bfloat16 b = __float2bfloat16_rn(r1);
  const __nv_bfloat16 d = __float2bfloat16_rn(r1 - __bfloat162float(b));
  p[0] = a; p[stride] = b; p[2 * stride] = d;
}

// Inverses of the diagonal blocks of L (which = 0) and U (which = 1) of up to kMaxGroup layers:
// one CTA per block, thread j owns column j of the inverse (forward substitution; an upper block
// is handled as the lower block it becomes when rows and columns are reversed).
// out: [layer][which][n / 128][128][128] fp32, row-major blocks.
__global__ void __launch_bounds__(kLuBlock)
lu_diag_inverse_kernel(PtrBatch Ps, int n, float* __restrict__ out, DeviceStatus* st, int layer0) {
  const int blk = blockIdx.x, which = blockIdx.y, lay = blockIdx.z;
  const float* P = static_cast<const float*>(Ps.p[lay]);
  const int o = blk * kLuBlock, j = threadIdx.x, r = kLuBlock - 1;
  // the block as a lower triangular matrix M in shared memory: L's block itself (unit diagonal),
  // or U's block with rows and columns reversed, M[i][k] = U[r-i][r-k], whose inverse is U^-1
  // reversed the same way
  extern __shared__ float Msh[];                      // [kLuBlock][kLuBlock + 1]
  for (int e = threadIdx.x; e < kLuBlock * kLuBlock; e += kLuBlock) {
    const int i = e / kLuBlock, k = e - i * kLuBlock;
    float v;
    if (which == 0) v = k < i ? P[(int64_t)(o + i) * n + o + k] : (k == i ? 1.f : 0.f);
    else v = k <= i ? P[(int64_t)(o + r - i) * n + o + r - k] : 0.f;
    Msh[i * (kLuBlock + 1) + k] = v;
  }
  __syncthreads();
  // thread j owns column j of the inverse: x_i = (delta_ij - sum_{k<i} M_ik x_k) / M_ii, with the
  // sum carried as an fp32 pair (error-free product and sum) so the result is fp32-accurate
  float x[kLuBlock];
  bool bad = false;
  for (int i = 0; i < kLuBlock; ++i) {
    float hi = i == j ? 1.f : 0.f, lo = 0.f;
    const float* row = Msh + i * (kLuBlock + 1);
    for (int k = j; k < i; ++k) {
      const float m = row[k], p = -m * x[k];
      const float pe = fmaf(-m, x[k], -p);            // exact product = p + pe
      const float t = hi + p;
      const float z = t - hi;
      lo += (hi - (t - z)) + (p - z) + pe;            // two-sum remainder
      hi = t;
    }
    const float d = row[i];
    if (!(d != 0.f) || !(d - d == 0.f)) { bad = true; x[i] = 0.f; }
    else x[i] = i < j ? 0.f : (hi + lo) / d;
  }
  if (bad) record_error(st, MW_ERR_NOT_SUBMERSIVE, (unsigned)(layer0 + lay), (unsigned)blk, 5u, 0u);
  float* dst = out + (((int64_t)lay * 2 + which) * (n / kLuBlock) + blk) * kLuBlock * kLuBlock;
  for (int i = 0; i < kLuBlock; ++i) {
    if (which == 0) dst[i * kLuBlock + j] = x[i];
    else dst[(r - i) * kLuBlock + (r - j)] = x[i];
  }
}

// term planes of L (unit lower) and U (upper) of the layers of a chunk (blockIdx.y), laid out
// [layer][plane][n][n]; with `diag` also the planes of L^-1 and U^-1 holding their inverted
// diagonal blocks and zeros elsewhere
__global__ void __launch_bounds__(256)
lu_split_kernel(PtrBatch Ps, int n, __nv_bfloat16* __restrict__ Lp, __nv_bfloat16* __restrict__ Up,
                const float* __restrict__ diag, __nv_bfloat16* __restrict__ Tp,
                __nv_bfloat16* __restrict__ Sp) {
  const int64_t nn = (int64_t)n * n, base = (int64_t)blockIdx.y * 3 * nn;
  const float* P = static_cast<const float*>(Ps.p[blockIdx.y]);
  const int nb = n / kLuBlock;
  if (diag) diag += (int64_t)blockIdx.y * 2 * nb * kLuBlock * kLuBlock;
  for (int64_t e = (int64_t)blockIdx.x * 256 + threadIdx.x; e < nn; e += (int64_t)gridDim.x * 256) {
    const int i = (int)(e / n), j = (int)(e - (int64_t)i * n);
    const float v = P[e];
    split3(i > j ? v : (i == j ? 1.f : 0.f), Lp + base + e, nn);
    split3(i <= j ? v : 0.f, Up + base + e, nn);
    if (diag) {
      const int bi = i / kLuBlock, bj = j / kLuBlock;
      float t = 0.f, u = 0.f;
      if (bi == bj) {
        const int64_t off = (int64_t)bi * kLuBlock * kLuBlock + (i - bi * kLuBlock) * kLuBlock + (j - bj * kLuBlock);
        t = diag[off];
        u = diag[(int64_t)nb * kLuBlock * kLuBlock + off];
      }
      split3(t, Tp + base + e, nn);
      split3(u, Sp + base + e, nn);
    }
  }
}

// term planes of the gradients of W of a chunk of layers
__global__ void __launch_bounds__(256)
lu_gsplit_kernel(PtrBatch Gs, int64_t nn, __nv_bfloat16* __restrict__ Gp) {
  const float* G = static_cast<const float*>(Gs.p[blockIdx.y]);
  const int64_t base = (int64_t)blockIdx.y * 3 * nn;
  for (int64_t e = (int64_t)blockIdx.x * 256 + threadIdx.x; e < nn; e += (int64_t)gridDim.x * 256)
    split3(G[e], Gp + base + e, nn);
}

// dP = (a below the diagonal, b on and above it), per layer of the chunk
struct OutBatch { void* p[kMaxGroup]; };
__global__ void __launch_bounds__(256)
lu_combine_kernel(const float* __restrict__ a, const float* __restrict__ b, int n, OutBatch outs) {
  const int64_t nn = (int64_t)n * n, base = (int64_t)blockIdx.y * nn;
  float* out = static_cast<float*>(outs.p[blockIdx.y]);
  for (int64_t e = (int64_t)blockIdx.x * 256 + threadIdx.x; e < nn; e += (int64_t)gridDim.x * 256) {
    const int i = (int)(e / n), j = (int)(e - (int64_t)i * n);
    out[e] = i > j ? a[base + e] : b[base + e];
  }
}

// layers whose factors are worked on together (their planes and temporaries: 36 n^2 bytes each)
int lu_chunk(const mw_net* n) {
  const size_t d = (size_t)n->layers[0].n_in;
  size_t g = ((size_t)768 << 20) / (36 * d * d);
  if (g < 1) g = 1;
  if (g > 16) g = 16;
  if (g > (size_t)n->L) g = (size_t)n->L;
  return (int)g;
}

// a block of the n x n matrices of G layers kept as [layer][plane][n][n], as an operand / output
// of a product batched over the layers
TcOperand lu_block(const Ctx& c, const __nv_bfloat16* planes, int r0, int c0, int rows, int cols, bool mn) {
  TcOperand o = operand(planes + (int64_t)r0 * c.dim + c0, rows, cols, 3, mn);
  o.plane_stride = c.nn;
  o.batch_planes = 3;
  o.ld = c.dim;
  return o;
}
TcEpilogue lu_block_out(const Ctx& c, __nv_bfloat16* planes, int r0, int c0, float alpha) {
  TcEpilogue e;
  e.mode = TC_EPI_PLAIN;
  e.alpha = alpha;
  e.planes = planes + (int64_t)r0 * c.dim + c0;
  e.n_planes = 3;
  e.plane_stride = c.nn;
  e.bs_planes = 3 * c.nn;
  e.ld = c.dim;
  return e;
}
TcGemm lu_product(const TcOperand& A, const TcOperand& B, int M, int N, int K, const TcEpilogue& e, int batch) {
  TcGemm g;
  g.A = A; g.B = B; g.M = M; g.N = N; g.K = K; g.epi = e;
  g.batch = batch;
  g.split_k = 1;
  return g;
}
mw_status lu_run(const Ctx& c, const std::vector<TcGemm>& g) {
  for (size_t i = 0; i < g.size(); i += kTcMaxGroup) {
    const size_t k = g.size() - i < (size_t)kTcMaxGroup ? g.size() - i : (size_t)kTcMaxGroup;
    MW_TRY(run(c, g.data() + i, (int)k));
  }
  return MW_OK;
}

// Fills w_planes[l] (W = L U) of every layer and, with `inverses`, inv[l] (W^-1 = U^-1 L^-1),
// a chunk of layers at a time: every product below is one entry batched over the chunk.
mw_status lu_prepare(const Ctx& c, const void* const* params, bool inverses) {
  const Layout& lay = *c.lay;
  const int L = c.n->L, d = c.dim, nb = d / kLuBlock, chunk = lu_chunk(c.n);
  __nv_bfloat16* Lp = c.at<__nv_bfloat16>(lay.lu_l);
  __nv_bfloat16* Up = c.at<__nv_bfloat16>(lay.lu_u);
  __nv_bfloat16* Tp = inverses ? c.at<__nv_bfloat16>(lay.lu_t) : nullptr;
  __nv_bfloat16* Sp = inverses ? c.at<__nv_bfloat16>(lay.lu_s) : nullptr;
  __nv_bfloat16* Yl = inverses ? c.at<__nv_bfloat16>(lay.lu_y[0]) : nullptr;
  __nv_bfloat16* Yu = inverses ? c.at<__nv_bfloat16>(lay.lu_y[1]) : nullptr;
  float* diag = inverses ? c.at<float>(lay.lu_diag) : nullptr;
  int64_t bx = (c.nn + 255) / 256;
  if (bx > 296) bx = 296;
  for (int l0 = 0; l0 < L; l0 += chunk) {
    const int G = (L - l0) < chunk ? (L - l0) : chunk;
    PtrBatch ps{};
    for (int g = 0; g < G; ++g) ps.p[g] = params[l0 + g];
    // the regions of consecutive layers must lie 3 planes apart for the batched outputs
    for (int g = 1; g < G; ++g) {
      if (lay.w_planes[l0 + g].off - lay.w_planes[l0 + g - 1].off != (size_t)(6 * c.nn)) return MW_ERR_WORKSPACE;
      if (inverses && lay.inv[l0 + g].off - lay.inv[l0 + g - 1].off != (size_t)(6 * c.nn)) return MW_ERR_WORKSPACE;
    }
    if (inverses) {
      constexpr size_t kDiagSmem = sizeof(float) * kLuBlock * (kLuBlock + 1);
      static bool attr[16] = {};
      int dev = 0;
      MW_CUDA_OK(cudaGetDevice(&dev));
      const bool known = dev >= 0 && dev < 16;
      if (!known || !attr[dev]) {     // the opt-in belongs to the device
        MW_CUDA_OK(cudaFuncSetAttribute(lu_diag_inverse_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kDiagSmem));
        if (known) attr[dev] = true;
      }
      lu_diag_inverse_kernel<<<dim3((unsigned)nb, 2u, (unsigned)G), kLuBlock, kDiagSmem, c.s>>>(ps, d, diag, c.st, l0);
      MW_TRY(launch_ok());
    }
    lu_split_kernel<<<dim3((unsigned)bx, (unsigned)G), 256, 0, c.s>>>(ps, d, Lp, Up, diag, Tp, Sp);
    MW_TRY(launch_ok());
    // the products of this chunk, in an order in which each comes after what it reads: `phase`
    // numbers the sets of mutually independent ones, d0 / d1 name the products it waits for
    struct Item { TcGemm g; int phase, d0, d1; };
    std::vector<Item> items;
    int phase = 0, top_l = -1, top_u = -1;
    if (inverses) {
      // segments [seg[i], seg[i+1]) whose diagonal blocks of L^-1 and U^-1 are complete, and the
      // product that completed each (-1: a single block, inverted by lu_diag_inverse_kernel)
      std::vector<int> seg, zl((size_t)nb, -1), zu((size_t)nb, -1);
      for (int b = 0; b <= nb; ++b) seg.push_back(b * kLuBlock);
      while (seg.size() > 2) {
        std::vector<int> merged, mzl, mzu;
        std::vector<Item> second;
        merged.push_back(seg[0]);
        const int first_index = (int)items.size();
        int pairs = 0;
        for (size_t i = 0; i + 2 < seg.size(); i += 2) ++pairs;
        for (size_t i = 0; i + 2 < seg.size(); i += 2) {
          const int a0 = seg[i], a1 = seg[i + 1], a2 = seg[i + 2], m1 = a1 - a0, m2 = a2 - a1;
          const int yl = first_index + 2 * (int)(i / 2), yu = yl + 1;
          // L^-1[a1:a2, a0:a1] = -D^-1 C A^-1
          items.push_back({lu_product(lu_block(c, Lp, a1, a0, m2, m1, false), lu_block(c, Tp, a0, a0, m1, m1, true),
                                      m2, m1, m1, lu_block_out(c, Yl, a1, a0, 1.f), G), phase, zl[i], -1});
          second.push_back({lu_product(lu_block(c, Tp, a1, a1, m2, m2, false), lu_block(c, Yl, a1, a0, m2, m1, true),
                                       m2, m1, m2, lu_block_out(c, Tp, a1, a0, -1.f), G), phase + 1, yl, zl[i + 1]});
          // U^-1[a0:a1, a1:a2] = -A^-1 B D^-1
          items.push_back({lu_product(lu_block(c, Up, a0, a1, m1, m2, false), lu_block(c, Sp, a1, a1, m2, m2, true),
                                      m1, m2, m2, lu_block_out(c, Yu, a0, a1, 1.f), G), phase, zu[i + 1], -1});
          second.push_back({lu_product(lu_block(c, Sp, a0, a0, m1, m1, false), lu_block(c, Yu, a0, a1, m1, m2, true),
                                       m1, m2, m1, lu_block_out(c, Sp, a0, a1, -1.f), G), phase + 1, yu, zu[i]});
          merged.push_back(a2);
          // the merged segment is complete once its two second-stage products are
          mzl.push_back(first_index + 2 * pairs + 2 * (int)(i / 2));
          mzu.push_back(first_index + 2 * pairs + 2 * (int)(i / 2) + 1);
        }
        if (merged.back() != seg.back()) {       // an odd segment waits a level
          merged.push_back(seg.back());
          mzl.push_back(zl[seg.size() - 2]);
          mzu.push_back(zu[seg.size() - 2]);
        }
        for (const Item& it : second) items.push_back(it);
        phase += 2;
        seg.swap(merged);
        zl.swap(mzl);
        zu.swap(mzu);
      }
      top_l = zl[0];
      top_u = zu[0];
    }
    // W = L U and W^-1 = U^-1 L^-1 by blocks of rows: a block of rows of L ends at its diagonal
    // block, one of U^-1 starts there, so each product runs over the K range that is not zero
    const int bs = d % 256 == 0 ? 256 : kLuBlock;
    for (int r0 = 0; r0 < d; r0 += bs) {
      const int k1 = r0 + bs;
      items.push_back({lu_product(lu_block(c, Lp, r0, 0, bs, k1, false), lu_block(c, Up, 0, 0, k1, d, true), bs, d, k1,
                                  lu_block_out(c, c.at<__nv_bfloat16>(lay.w_planes[l0]), r0, 0, 1.f), G), phase, -1, -1});
      if (inverses)
        items.push_back({lu_product(lu_block(c, Sp, r0, r0, bs, d - r0, false), lu_block(c, Tp, r0, 0, d - r0, d, true),
                                    bs, d, d - r0, lu_block_out(c, c.at<__nv_bfloat16>(lay.inv[l0]), r0, 0, 1.f), G),
                         phase, top_l, top_u});
    }
    if ((int)items.size() <= kLuProgEntries) {
      // one launch for the whole chunk: every product starts when the ones it reads are complete
      TensorState* t = static_cast<TensorState*>(c.n->tc);
      const int which = inverses ? 1 : 0;
      const size_t ci = (size_t)(l0 / chunk);
      if (t->lu_prog[which].size() <= ci) {
        t->lu_prog[which].resize(ci + 1, nullptr);
        t->lu_key[which].resize(ci + 1);
      }
      const std::vector<const void*> key = {c.ws, reinterpret_cast<const void*>((uintptr_t)G)};
      if (!t->lu_prog[which][ci] || t->lu_key[which][ci] != key) {
        if (!t->lu_prog[which][ci]) t->lu_prog[which][ci] = tc_program_create();
        t->lu_key[which][ci].clear();
        TcProgram* pr = t->lu_prog[which][ci];
        tc_program_begin(pr, c.at<char>(lay.lu_table), c.at<unsigned int>(lay.lu_done), false);
        for (const Item& it : items) {
          const int deps[2] = {it.d0, it.d1};
          mw_status st;
          if (tc_program_add(pr, c.cache, it.g, deps, 2, &st, -1) < 0) return st;
        }
        t->lu_key[which][ci] = key;
      }
      MW_TRY(tc_program_launch(t->lu_prog[which][ci], c.st, c.s));
    } else {
      std::vector<TcGemm> same;
      for (size_t i = 0; i < items.size(); ++i) {
        same.push_back(items[i].g);
        if (i + 1 == items.size() || items[i + 1].phase != items[i].phase) {
          MW_TRY(lu_run(c, same));
          same.clear();
        }
      }
    }
  }
  return MW_OK;
}

// dW[l] of layers [l0, l1) hold G = dJ/dW; replaces each by the gradient of the layer's factors
mw_status lu_map_gradients(const Ctx& c, const void* const* params, void* const* dW, int l0, int l1) {
  const Layout& lay = *c.lay;
  const int d = c.dim, chunk = lu_chunk(c.n);
  __nv_bfloat16* Lp = c.at<__nv_bfloat16>(lay.lu_l);
  __nv_bfloat16* Up = c.at<__nv_bfloat16>(lay.lu_u);
  __nv_bfloat16* Gp = c.at<__nv_bfloat16>(lay.lu_g);
  int64_t bx = (c.nn + 255) / 256;
  if (bx > 296) bx = 296;
  std::vector<int> todo;
  for (int l = l0; l < l1; ++l)
    if (dW[l]) todo.push_back(l);
  for (size_t t0 = 0; t0 < todo.size(); t0 += (size_t)chunk) {
    const int G = (int)(todo.size() - t0 < (size_t)chunk ? todo.size() - t0 : (size_t)chunk);
    PtrBatch ps{}, gs{};
    OutBatch outs{};
    for (int g = 0; g < G; ++g) {
      ps.p[g] = params[todo[t0 + g]];
      gs.p[g] = dW[todo[t0 + g]];
      outs.p[g] = dW[todo[t0 + g]];
    }
    lu_split_kernel<<<dim3((unsigned)bx, (unsigned)G), 256, 0, c.s>>>(ps, d, Lp, Up, nullptr, nullptr, nullptr);
    MW_TRY(launch_ok());
    lu_gsplit_kernel<<<dim3((unsigned)bx, (unsigned)G), 256, 0, c.s>>>(gs, c.nn, Gp);
    MW_TRY(launch_ok());
    // Only the strictly lower part of G U^T and the upper part of L^T G are wanted, and U^T, L^T
    // are triangular: by blocks of columns (rows), each product covers the wanted tiles and the K
    // range that is not zero.
    const int bs = d % 256 == 0 ? 256 : kLuBlock;
    std::vector<TcGemm> g;
    for (int o = 0; o < d; o += bs) {
      const int rest = d - o;
      TcEpilogue ea, eb;
      ea.mode = eb.mode = TC_EPI_PLAIN;
      ea.out_f32 = c.at<float>(lay.lu_a) + (int64_t)o * d + o;
      eb.out_f32 = c.at<float>(lay.lu_b) + (int64_t)o * d + o;
      ea.bs_f32 = eb.bs_f32 = c.nn;
      ea.ld = eb.ld = d;
      // (G U^T)[o:, o:o+bs]: B operand [N][K] = rows o.. of U from column o on
      g.push_back(lu_product(lu_block(c, Gp, o, o, rest, rest, false), lu_block(c, Up, o, o, bs, rest, false),
                             rest, bs, rest, ea, G));
      // (L^T G)[o:o+bs, o:]: A operand MN-major = L[o:, o:o+bs] as [K][M], B = G[o:, o:] as [K][N]
      g.push_back(lu_product(lu_block(c, Lp, o, o, rest, bs, true), lu_block(c, Gp, o, o, rest, rest, true),
                             bs, rest, rest, eb, G));
    }
    MW_TRY(lu_run(c, g));
    lu_combine_kernel<<<dim3((unsigned)bx, (unsigned)G), 256, 0, c.s>>>(c.at<float>(lay.lu_a), c.at<float>(lay.lu_b), d, outs);
    MW_TRY(launch_ok());
  }
  return MW_OK;
}

mw_status forward_pass(const Ctx& c, const void* const* params, const void* x, bool store_acts) {
  const Layout& lay = *c.lay;
  const int L = c.n->L, d = c.dim;
  const __nv_bfloat16* xin = nullptr;
  MW_TRY(input_planes(c, x, &xin));
  const bool resident = c.n->opts.resident_inverse != 0;
  for (int l = 0; l < L; ++l) {
    const mw_layer_desc& ld = c.n->layers[l];
    const __nv_bfloat16* Wp = nullptr;
    // resident + Moonwalk: the planes were made by the prep at the top of mw_input_cotangent
    MW_TRY(weight_planes(c, l, params[l], !(resident && !store_acts), &Wp));
    __nv_bfloat16* xout = (store_acts && l + 1 < L) ? c.at<__nv_bfloat16>(lay.stored_act[l + 1])
                                                   : c.at<__nv_bfloat16>(lay.xp[(l + 1) % 3]);
    TcEpilogue e;
    e.mode = TC_EPI_FWD;
    e.mask = c.at<uint32_t>(lay.mask[l]);
    e.write_mask = 1;
    e.act = ld.act;
    e.slope = (float)ld.slope;
    if (l + 1 < L) {
      e.planes = xout; e.n_planes = c.pr.px; e.plane_stride = c.bn;
    } else {
      e.out_f32 = c.at<float>(lay.z);
    }
    TcGemm g = product(c, operand(xin, c.B, d, c.pr.px, false), operand(Wp, d, d, c.pr.pw, false),
                       c.B, d, d, e, 0);
    MW_TRY(run(c, &g, 1));
    xin = xout;
  }
  return MW_OK;
}

// index of layer l's fragment stream from its sign words
mw_status relu_index(const Ctx& c, int l) {
  const Layout& lay = *c.lay;
  return fragment_index(c.at<uint32_t>(lay.mask[l]), c.B, c.dim, c.at<uint32_t>(lay.frag_cnt[l]),
                        c.at<uint32_t>(lay.frag_off[l]), c.at<uint32_t>(lay.frag_rank[l]),
                        c.at<uint32_t>(lay.frag_total) + l, c.s);
}

// top of the reverse pass: loss, h_L (fp32 in cot[0]) and g_z of the last layer as term planes
mw_status loss_and_top(const Ctx& c, const void* target, double* loss_out, bool fragments) {
  const Layout& lay = *c.lay;
  const int L = c.n->L, d = c.dim;
  const mw_layer_desc& ld = c.n->layers[L - 1];
  float* h = c.at<float>(lay.cot[0]);
  MW_TRY(loss_cotangent<float>(c.at<float>(lay.z), target, c.B, d, c.n->opts.loss, h,
                               c.at<double>(lay.partials), loss_out, c.s));
  const uint32_t* words = c.at<uint32_t>(lay.mask[L - 1]);
  if (fragments && ld.act == MW_ACT_RELU) {
    MW_TRY(relu_index(c, L - 1));
    MW_TRY(fragment_compact<float>(h, words, c.B, d, c.at<uint32_t>(lay.frag_off[L - 1]),
                                   c.at<float>(lay.frag_vals[L - 1]), c.s));
  }
  float* g = c.at<float>(lay.cot[1]);
  const float* src = h;
  if (ld.act != MW_ACT_NONE) {
    MW_TRY(scale_by_mask<float>(h, words, c.B, d, ld.act, ld.slope, g, c.s));
    src = g;
  }
  return split_planes(src, c.bn, c.at<__nv_bfloat16>(lay.hp[0]), c.pr.pg2, c.bn, c.s);
}

// ---- Newton-Schulz as products of a program --------------------------------------------------
// In the program path every layer has its own iterate (fp32 X, term planes of X and of the
// residual), so that the steps of different layers can be spread over the launches that carry
// Phase I and Phase II: the chains of those phases leave most SMs waiting, the inverses fill them.

struct NsBuffers {
  float* X;
  __nv_bfloat16 *Rp, *Xp[2];
  double* sumsq;
};

NsBuffers ns_buffers(const Ctx& c) {
  const Layout& lay = *c.lay;
  const int64_t L = c.n->L;
  NsBuffers b;
  b.X = c.at<float>(lay.ns_x);
  b.Rp = c.at<__nv_bfloat16>(lay.ns_r);
  b.Xp[0] = b.Rp + 3 * L * c.nn;
  b.Xp[1] = b.Rp + 6 * L * c.nn;
  b.sumsq = c.at<double>(lay.ns_sumsq);
  return b;
}

// c_l = n / ||W_l||_F^2 of every layer: the scale of the start X_0 = c W^T.  X_0 itself is never
// formed: the first step X_1 = X_0 (2 I - W X_0) = W^T [c (2 I - c W W^T)] is two products that
// read W in place (ns_product).
mw_status ns_prepare_all(const Ctx& c, const void* const* params) {
  const Layout& lay = *c.lay;
  const int L = c.n->L, d = c.dim;
  const bool f32 = c.n->opts.prec == MW_F32;
  char* sc = c.at<char>(lay.inv_scratch);
  double* fpart = reinterpret_cast<double*>(sc + 12 * kMaxGroup + 64);
  float* cscale = c.at<float>(lay.ns_scale);
  for (int l0 = 0; l0 < L; l0 += kMaxGroup) {
    const int G = (L - l0) < kMaxGroup ? (L - l0) : kMaxGroup;
    PtrBatch wp{};
    for (int g = 0; g < G; ++g) wp.p[g] = params[l0 + g];
    if (f32) frob_partial_kernel<float><<<dim3(kFrobBlocks, G), 256, 0, c.s>>>(wp, c.nn, fpart);
    else frob_partial_kernel<__nv_bfloat16><<<dim3(kFrobBlocks, G), 256, 0, c.s>>>(wp, c.nn, fpart);
    frob_final_kernel<<<1, kMaxGroup, 0, c.s>>>(fpart, G, d, cscale + l0);
    MW_TRY(launch_ok(2));
  }
  return MW_OK;
}

// product `stage` of layer l: even = residual R = I - W X of step stage/2, odd = its update
// (the iterate alternates between its two homes Xp[0], Xp[1]; step `it` reads home side0 + it)
// (`nb`, `lb`, `scale`: the iterate's buffers, the layer's index inside them and its start scale;
// the program path keeps them per layer, the one-layer-at-a-time path has one set)
TcGemm ns_product_at(const Ctx& c, int l, const NsBuffers& nb, int lb, const float* scale, int stage,
                     const void* const* params, const NsStep* sched, int steps, int side0, bool warm) {
  const Layout& lay = *c.lay;
  const int d = c.dim, it = stage >> 1, cur = (side0 + it) & 1;
  const bool last = it + 1 == steps;
  float* X = nb.X + (int64_t)lb * c.nn;
  __nv_bfloat16* Rp = nb.Rp + (int64_t)lb * 3 * c.nn;
  __nv_bfloat16* Xc = nb.Xp[cur] + (int64_t)lb * 3 * c.nn;
  __nv_bfloat16* Xn = nb.Xp[cur ^ 1] + (int64_t)lb * 3 * c.nn;
  TcGemm g;
  g.M = d; g.N = d; g.K = d;
  g.wide_tiles = 1;      // throughput work beside the latency-bound chains
  const void* W = c.n->opts.prec == MW_F32 ? (const void*)c.at<__nv_bfloat16>(lay.w_planes[l]) : params[l];
  if (it == 0 && !warm) {
    // from scratch: X_0 = c W^T stays implicit.  Stage 0: T = c (2 I - c W W^T) (W against itself,
    // both K-major); stage 1: X_1 = W^T T (W read through its transpose), no addend.
    const int pw = c.pr.pw < sched[0].pu ? c.pr.pw : sched[0].pu;
    if (!(stage & 1)) {
      g.A = operand(W, d, d, pw, false);
      g.B = operand(W, d, d, pw, false);
      g.epi.mode = TC_EPI_RESID;
      g.epi.scale_dev = scale;
      g.epi.symmetric = 1;    // W W^T: tiles on and above the diagonal, mirrored (where the kernel form allows)
      g.epi.planes = Rp; g.epi.n_planes = sched[0].pu; g.epi.plane_stride = c.nn;
    } else {
      int next_terms = c.pr.ph;
      if (!last) next_terms = sched[1].pr > sched[1].pu ? sched[1].pr : sched[1].pu;
      g.A = operand(W, d, d, pw, true);
      g.B = operand(Rp, d, d, sched[0].pu, true);
      g.epi.mode = TC_EPI_PLAIN;
      g.epi.out_f32 = (last && !c.n->opts.warm_inverse) ? nullptr : X;
      g.epi.planes = Xn;
      g.epi.n_planes = next_terms;
      g.epi.plane_stride = c.nn;
    }
    return g;
  }
  if (!(stage & 1)) {
    const int pw = c.pr.pw < sched[it].pr ? c.pr.pw : sched[it].pr;
    g.A = operand(W, d, d, pw, false);
    g.B = operand(Xc, d, d, sched[it].pr, true);
    g.epi.mode = TC_EPI_RESID;
    g.epi.planes = Rp; g.epi.n_planes = sched[it].pu; g.epi.plane_stride = c.nn;
    // bf16 nets: X_1 = W^T T is W^T times a polynomial of W W^T, so W X_1 is symmetric up to the
    // rounding of X_1's term planes (2^-17): the residual of the second step is computed on and
    // above the diagonal and mirrored.  Not where that form is broken (measured: gradient errors
    // of 2e-4 to 5e-3 in fp32 when the asymmetric part is dropped): fp32 nets, whose first step
    // reads W rounded to one term (W round(W)^T is not symmetric); later iterates, which went
    // through an update with fewer terms, X + round(X) round(R); a kept inverse that is being
    // refreshed for a new W.
    g.epi.symmetric = (!warm && it == 1 && c.n->opts.prec != MW_F32) ? 1 : 0;
    // only the last residual is gated (the update that follows squares it)
    if (last) g.epi.sumsq = nb.sumsq + (int64_t)lb * (int64_t)gate_slots(d);
  } else {
    int next_terms = c.pr.ph;
    if (!last) next_terms = sched[it + 1].pr > sched[it + 1].pu ? sched[it + 1].pr : sched[it + 1].pu;
    g.A = operand(Xc, d, d, sched[it].pu, false);
    g.B = operand(Rp, d, d, sched[it].pu, true);
    g.epi.mode = TC_EPI_PLAIN;
    g.epi.addend = X;
    // the last iterate stays in fp32 too where the next call may refresh it
    g.epi.out_f32 = (last && !c.n->opts.warm_inverse) ? nullptr : X;
    g.epi.planes = Xn;         // the last step leaves W^-1 here: the sweep reads it in place
    g.epi.n_planes = next_terms;
    g.epi.plane_stride = c.nn;
  }
  return g;
}

TcGemm ns_product(const Ctx& c, int l, int stage, const void* const* params, const NsStep* sched,
                  int steps, int side0, bool warm) {
  return ns_product_at(c, l, ns_buffers(c), l, c.at<float>(c.lay->ns_scale) + l, stage, params, sched, steps,
                       side0, warm);
}

// One bf16 layer at a time (transient inverse slot, or a net too deep for the product tables): the
// same products as the program path -- implicit start, symmetric W W^T and second residual --
// as single launches, the last update writing the term planes the sweep reads.
mw_status newton_schulz_single(const Ctx& c, int l, const void* const* params) {
  const Layout& lay = *c.lay;
  const int d = c.dim;
  NsStep sched[16];
  const int steps = ns_schedule(c.n, sched);
  if (steps < 1) return MW_ERR_INVALID_ARG;
  char* sc = c.at<char>(lay.inv_scratch);
  float* cscale = reinterpret_cast<float*>(sc + 8 * kMaxGroup);
  double* fpart = reinterpret_cast<double*>(sc + 12 * kMaxGroup + 64);
  NsBuffers nb;
  nb.X = c.at<float>(lay.ns_x);
  nb.Rp = c.at<__nv_bfloat16>(lay.ns_r);
  nb.Xp[0] = nb.Rp + 3 * c.nn;
  nb.Xp[1] = nb.Rp + 6 * c.nn;
  nb.sumsq = c.at<double>(lay.ns_sumsq);
  PtrBatch wp{};
  wp.p[0] = params[l];
  frob_partial_kernel<__nv_bfloat16><<<dim3(kFrobBlocks, 1), 256, 0, c.s>>>(wp, c.nn, fpart);
  frob_final_kernel<<<1, kMaxGroup, 0, c.s>>>(fpart, 1, d, cscale);
  MW_TRY(launch_ok(2));
  MW_CUDA_OK(cudaMemsetAsync(nb.sumsq, 0, sizeof(double) * gate_slots(d), c.s));
  for (int stage = 0; stage < 2 * steps; ++stage) {
    TcGemm g = ns_product_at(c, l, nb, 0, cscale, stage, params, sched, steps, 0, false);
    const bool last_update = stage == 2 * steps - 1;
    if (last_update) g.epi.planes = c.at<__nv_bfloat16>(lay.inv[l]);
    MW_TRY(run(c, &g, 1));
    if (stage == 2 * (steps - 1) && steps > 1) {
      // the update squares this residual: gate on it so a diverging layer is reported
      const NsStep lastst = sched[steps - 1];
      const int pw = c.pr.pw < lastst.pr ? c.pr.pw : lastst.pr;
      residual_gate_kernel<<<1, 256, 0, c.s>>>(nb.sumsq, (int64_t)gate_slots(d),
                                               (int64_t)tc_sumsq_slots(pw, lastst.pr, d, d, tc_pair_ok(pw, lastst.pr, d, d)),
                                               d, 2e-2, c.st, l);
      MW_TRY(launch_ok());
    }
  }
  return MW_OK;
}

// the inverse steps handed out to the chain steps of Phase I and Phase II, in step-major order
// (step t of a layer sits L positions after its step t-1, so its turn comes many chain steps later)
struct NsFeed {
  const void* const* params;
  NsStep sched[16];
  int steps = 0, total = 0, next = 0, per_slot = 0;
  int side0 = 0;              // home of the iterate the first step reads
  int variant = 0;            // of the programs that carry this feed (see kProgVariants)
  std::vector<int> last;      // last product of each layer's chain inside the current program
};

// warm: only the last step of the schedule, from the inverse the workspace kept (home `side0`)
NsFeed make_feed(const Ctx& c, const void* const* params, bool warm, int side0) {
  NsFeed f;
  f.params = params;
  f.steps = ns_schedule(c.n, f.sched);
  if (warm && f.steps > 1) {
    f.sched[0] = f.sched[f.steps - 1];
    f.steps = 1;
  }
  f.side0 = side0 & 1;
  f.variant = (warm ? 2 : 0) + f.side0;
  f.total = f.steps > 0 ? 2 * f.steps * c.n->L : 0;
  f.per_slot = (f.total + 2 * c.n->L - 1) / (2 * c.n->L);
  f.last.assign(c.n->L, -1);
  return f;
}

// ---- whole phases as one launch ("programs") -------------------------------------------------
// needs every layer's weight and inverse planes resident, and room in the product table
bool use_programs(const mw_net* n) {
  return n->opts.resident_inverse != 0 && 5 * (n->L + 1) <= kTcMaxProgram;
}

TensorState* state_of(const Ctx& c) { return static_cast<TensorState*>(c.n->tc); }

bool program_ready(const Ctx& c, int idx, const std::vector<const void*>& key, int variant = 0) {
  TensorState* t = state_of(c);
  return t->prog[idx][variant] != nullptr && !t->key[idx][variant].empty() && t->key[idx][variant] == key;
}

// every product of a dense bf16 net (batch x width and width x width outputs, at most two terms
// per operand) can run in the pair form when both sizes are multiples of 256
bool net_pair(const Ctx& c) {
  return c.n->opts.prec != MW_F32 && tc_pair_ok(2, 2, c.B, c.dim) && tc_pair_ok(2, 2, c.dim, c.dim);
}

// sizes at which the sweep may run as chains (the workspace then holds the longer rings): row
// blocks of 256 for the pair form, of 128 otherwise
bool chain_sizes(const mw_net* n) {
  return n->opts.resident_inverse != 0 && n->B % 128 == 0 && n->B / 128 <= 16 && 5 * (n->L + 1) <= kTcMaxProgram;
}

TcProgram* program_begin(const Ctx& c, int idx, int slot, int variant = 0) {
  TensorState* t = state_of(c);
  if (!t->prog[idx][variant]) t->prog[idx][variant] = tc_program_create();
  t->key[idx][variant].clear();
  tc_program_begin(t->prog[idx][variant], c.at<char>(c.lay->prog_table[slot]),
                   c.at<unsigned int>(c.lay->prog_done[slot]), net_pair(c));
  return t->prog[idx][variant];
}

struct Adder {
  const Ctx& c;
  TcProgram* pr;
  mw_status status = MW_OK;
  // the next inverse steps, after a chain product (everything that is left when `all`)
  void feed(NsFeed* f, bool all) {
    if (!f) return;
    const int L = c.n->L;
    for (int k = 0; (all || k < f->per_slot) && f->next < f->total; ++k, ++f->next) {
      const int stage = f->next / L, l = f->next % L;
      f->last[l] = add(ns_product(c, l, stage, f->params, f->sched, f->steps, f->side0, (f->variant & 2) != 0),
                       f->last[l]);
    }
  }
  int add(const TcGemm& g, int d0 = -1, int d1 = -1, int d2 = -1) { return add_to(g, -1, d0, d1, d2); }
  // the same, the product also reporting to the group entry `group` (-1: none)
  int add_to(const TcGemm& g, int group, int d0 = -1, int d1 = -1, int d2 = -1) {
    if (status != MW_OK) return -1;
    const int deps[3] = {d0, d1, d2};
    mw_status st;
    const int q = tc_program_add(pr, c.cache, g, deps, 3, &st, group);
    if (q < 0) status = st;
    return q;
  }
  int group() {
    if (status != MW_OK) return -1;
    const int q = tc_program_add_group(pr);
    if (q < 0) status = MW_ERR_UNSUPPORTED;
    return q;
  }
};

std::vector<const void*> key_of(const Ctx& c, const void* const* params, const void* a,
                                const void* b, void* const* dW) {
  std::vector<const void*> k;
  k.push_back(c.ws);
  k.push_back(a);
  k.push_back(b);
  for (int l = 0; l < c.n->L; ++l) k.push_back(params[l]);
  if (dW)
    for (int l = 0; l < c.n->L; ++l) k.push_back(dW[l]);
  return k;
}

// all weights as term planes (MW_F32; the layers' plane regions are contiguous)
mw_status split_all_weights(const Ctx& c, const void* const* params) {
  if (c.n->opts.prec != MW_F32) return MW_OK;
  const Layout& lay = *c.lay;
  const int L = c.n->L;
  for (int l0 = 0; l0 < L; l0 += kMaxGroup) {
    const int G = (L - l0) < kMaxGroup ? (L - l0) : kMaxGroup;
    PtrBatch wp{};
    for (int g = 0; g < G; ++g) wp.p[g] = params[l0 + g];
    int64_t bx = (c.nn / 4 + 255) / 256;
    if (bx > 64) bx = 64;
    split_weights_kernel<<<dim3((unsigned)bx, (unsigned)G), 256, 0, c.s>>>(
        wp, c.nn / 4, c.nn, c.at<__nv_bfloat16>(lay.w_planes[l0]));
    MW_TRY(launch_ok());
  }
  return MW_OK;
}

// Phase I (or backprop's forward) as one launch; the weight term planes must already exist
mw_status forward_program(const Ctx& c, const void* const* params, const void* x, bool store_acts,
                          NsFeed* feed = nullptr) {
  const Layout& lay = *c.lay;
  const int L = c.n->L, d = c.dim;
  const int idx = store_acts ? MW_PROG_BP_FWD : MW_PROG_PHASE1;
  const __nv_bfloat16* xin = nullptr;
  MW_TRY(input_planes(c, x, &xin));
  const std::vector<const void*> key = key_of(c, params, x, nullptr, nullptr);
  const int variant = feed ? feed->variant : 0;
  if (!program_ready(c, idx, key, variant)) {
    Adder a{c, program_begin(c, idx, 0, variant)};
    int prev = -1;
    for (int l = 0; l < L; ++l) {
      const mw_layer_desc& ld = c.n->layers[l];
      const __nv_bfloat16* Wp = nullptr;
      MW_TRY(weight_planes(c, l, params[l], false, &Wp));
      __nv_bfloat16* xout = (store_acts && l + 1 < L) ? c.at<__nv_bfloat16>(lay.stored_act[l + 1])
                                                     : c.at<__nv_bfloat16>(lay.xp[(l + 1) % 3]);
      TcEpilogue e;
      e.mode = TC_EPI_FWD;
      e.mask = c.at<uint32_t>(lay.mask[l]);
      e.write_mask = 1;
      e.act = ld.act;
      e.slope = (float)ld.slope;
      if (l + 1 < L) {
        e.planes = xout; e.n_planes = c.pr.px; e.plane_stride = c.bn;
      } else {
        e.out_f32 = c.at<float>(lay.z);
      }
      prev = a.add(product(c, operand(xin, c.B, d, c.pr.px, false), operand(Wp, d, d, c.pr.pw, false),
                           c.B, d, d, e, 0), prev);
      a.feed(feed, false);
      xin = xout;
    }
    MW_TRY(a.status);
    state_of(c)->key[idx][variant] = key;
  }
  return tc_program_launch(state_of(c)->prog[idx][variant], c.st, c.s);
}

// Phase II as one launch (the g_z planes of the last layer are in hp[0])
mw_status phase2_program(const Ctx& c, const void* const* params, void* g0, NsFeed* feed) {
  const Layout& lay = *c.lay;
  mw_net* n = c.n;
  const int L = n->L, d = c.dim;
  for (int l = 0; l + 1 < L; ++l)
    if (n->layers[l].act == MW_ACT_RELU) MW_TRY(relu_index(c, l));
  const std::vector<const void*> key = key_of(c, params, g0, nullptr, nullptr);
  const int variant = feed ? feed->variant : 0;
  if (!program_ready(c, MW_PROG_PHASE2, key, variant)) {
    Adder a{c, program_begin(c, MW_PROG_PHASE2, 1, variant)};
    int prev = -1, cur = 0;
    if (feed) {
      // Phase I took its share; earlier steps of every layer ended with that launch
      const int taken = feed->per_slot * L;
      feed->next = taken < feed->total ? taken : feed->total;
      feed->last.assign(L, -1);
    }
    for (int l = L - 1; l >= 0; --l) {
      const __nv_bfloat16* Wp = nullptr;
      MW_TRY(weight_planes(c, l, params[l], false, &Wp));
      TcEpilogue e;
      e.mode = TC_EPI_BWD;
      if (l == 0) {
        e.out_f32 = (float*)g0;
      } else {
        const mw_layer_desc& below = n->layers[l - 1];
        if (is_reseed(n, l)) {
          e.planes2 = c.at<__nv_bfloat16>(lay.reseed[l]);
          e.n_planes2 = c.pr.ph;
          e.plane_stride2 = c.bn;
        }
        e.act = below.act;
        e.slope = (float)below.slope;
        e.mask = c.at<uint32_t>(lay.mask[l - 1]);
        e.planes = c.at<__nv_bfloat16>(lay.hp[cur ^ 1]);
        e.n_planes = c.pr.pg2;
        e.plane_stride = c.bn;
        if (below.act == MW_ACT_RELU) {
          e.frag_off = c.at<uint32_t>(lay.frag_off[l - 1]);
          e.frag_rank = c.at<uint32_t>(lay.frag_rank[l - 1]);
          e.frag_vals = c.at<float>(lay.frag_vals[l - 1]);
        }
      }
      prev = a.add(product(c, operand(c.at<__nv_bfloat16>(lay.hp[cur]), c.B, d, c.pr.pg2, false),
                           operand(Wp, d, d, c.pr.pw, true), c.B, d, d, e, 0), prev);
      a.feed(feed, l == 0);
      cur ^= 1;
    }
    MW_TRY(a.status);
    state_of(c)->key[MW_PROG_PHASE2][variant] = key;
  }
  return tc_program_launch(state_of(c)->prog[MW_PROG_PHASE2][variant], c.st, c.s);
}

// term planes of h_l as the vijp's operand: the checkpoint where the recursion restarts
const __nv_bfloat16* h_planes(const Ctx& c, int l) {
  return (l > 0 && is_reseed(c.n, l)) ? c.at<__nv_bfloat16>(c.lay->reseed[l])
                                      : c.at<__nv_bfloat16>(c.lay->hp[l & 1]);
}

// W^-1 of layer l as term planes: where the prep left it
const __nv_bfloat16* inverse_planes(const Ctx& c, int l) {
  if (use_programs(c.n) && !c.n->opts.lu_param) return ns_buffers(c).Xp[c.n->inv_side & 1] + (int64_t)l * 3 * c.nn;
  return c.at<__nv_bfloat16>(c.lay->inv[l]);
}

// the products of layer l of the sweep
TcGemm recompute_product(const Ctx& c, int l, const __nv_bfloat16* xl, const __nv_bfloat16* Wp) {
  const mw_layer_desc& ld = c.n->layers[l];
  TcEpilogue e;
  e.mode = TC_EPI_FWD;
  e.mask = c.at<uint32_t>(c.lay->mask[l]);
  e.write_mask = 0;
  e.act = ld.act;
  e.slope = (float)ld.slope;
  e.planes = c.at<__nv_bfloat16>(c.lay->xp[(l + 1) % c.nx]);
  e.n_planes = c.pr.px;
  e.plane_stride = c.bn;
  return product(c, operand(xl, c.B, c.dim, c.pr.px, false), operand(Wp, c.dim, c.dim, c.pr.pw, false),
                 c.B, c.dim, c.dim, e, 0);
}

TcGemm vijp_product(const Ctx& c, int l, bool want_h, bool want_gz) {
  const Layout& lay = *c.lay;
  const mw_layer_desc& ld = c.n->layers[l];
  TcEpilogue e;
  e.mode = TC_EPI_VIJP;
  e.act = ld.act;
  e.slope = (float)ld.slope;
  e.mask = c.at<uint32_t>(lay.mask[l]);
  if (ld.act == MW_ACT_RELU) {
    e.frag_off = c.at<uint32_t>(lay.frag_off[l]);
    e.frag_rank = c.at<uint32_t>(lay.frag_rank[l]);
    e.frag_vals = c.at<float>(lay.frag_vals[l]);
  }
  if (want_h) {
    e.planes2 = c.at<__nv_bfloat16>(lay.hp[(l + 1) & 1]);
    e.n_planes2 = c.pr.ph;
    e.plane_stride2 = c.bn;
  }
  if (want_gz) {
    e.planes = c.at<__nv_bfloat16>(lay.gzp[l % c.ngz]);
    e.n_planes = c.pr.pgw;
    e.plane_stride = c.bn;
  }
  return product(c, operand(h_planes(c, l), c.B, c.dim, c.pr.ph, false),
                 operand(inverse_planes(c, l), c.dim, c.dim, c.pr.ph, true), c.B, c.dim, c.dim, e, 1);
}

// `layer`: whose gradient this is (for the fused parameter update, Algorithm 1's last line)
TcGemm weight_vjp_product(const Ctx& c, const __nv_bfloat16* gz, const __nv_bfloat16* xl, float* dW,
                          int layer = -1) {
  TcEpilogue e;
  e.mode = TC_EPI_PLAIN;
  e.out_f32 = dW;
  if (c.n->apply_params && layer >= 0) {
    e.alpha = -c.n->apply_lr;
    e.addend = static_cast<const float*>(c.n->apply_params[layer]);
  }
  return product(c, operand(gz, c.B, c.dim, c.pr.pgw, true), operand(xl, c.B, c.dim, c.pr.pxw, true),
                 c.dim, c.dim, c.B, e, 2);
}

// ---- the forward sweep as chains of one program launch ---------------------------------------
// Algorithm 1 walks the layers in order, but the rows of the batch never meet before the weight
// vjp: block m of `rb` rows of h_{l+1} and x_{l+1} needs block m of h_l and x_l only.  The sweep is
// therefore B / rb independent chains of products
//   V_{l,m}  (g_z, h_{l+1})[rows m] = vijp of layer l applied to h_l[rows m]      (Eq. "h_i")
//   R_{l,m}  x_{l+1}[rows m] = phi(x_l[rows m] W_l^T)                               (recompute)
// plus, per layer, D_l = g_z^T x_l over all rows (Eq. "g_i"), which needs the whole of V_l and of
// R_{l-1} (two group counters) and feeds nothing.  One launch carries the layers [l0, l1): a
// chain's next product sits hundreds of list positions behind the one it waits for, so the CTAs
// rarely wait, and there is no launch boundary (with its idle tail) per layer.
mw_status sweep_chain_program(const Ctx& c0, TcProgram* pr, int l0, int l1, const void* const* params,
                              void* const* dW, const __nv_bfloat16* x0p, bool pair) {
  Ctx c = c0;
  c.nx = 5;
  c.ngz = 4;
  const Layout& lay = *c.lay;
  mw_net* n = c.n;
  const int L = n->L, d = c.dim;
  const int rb = pair ? 256 : 128, mt = c.B / rb;
  tc_program_begin(pr, c.at<char>(lay.prog_table[0]), c.at<unsigned int>(lay.prog_done[0]), pair);
  tc_program_balance(pr, !pair);
  Adder a{c, pr};
  auto xbuf = [&](int l) -> const __nv_bfloat16* {
    return l == 0 ? x0p : c.at<__nv_bfloat16>(lay.xp[l % c.nx]);
  };
  const int64_t blk = (int64_t)rb * d;                 // elements of one row block
  const int nl = l1 - l0;
  std::vector<int> GV((size_t)nl, -1), GR((size_t)nl, -1), D((size_t)nl, -1);
  // the latest product of each chain (layers that need no vijp leave a gap in the V chain: the
  // next V still follows the last one, which orders every reuse of the h slots of its rows)
  std::vector<int> Vprev((size_t)mt, -1), Rprev((size_t)mt, -1);
  int gz_reader[4] = {-1, -1, -1, -1};   // the latest weight vjp that read each g_z slot
  auto at_or = [&](const std::vector<int>& v, int l) { return l >= l0 && l < l1 ? v[(size_t)(l - l0)] : -1; };
  auto weight_vjp = [&](int k) {
    if (!dW[k]) return;
    TcGemm g = weight_vjp_product(c, c.at<__nv_bfloat16>(lay.gzp[k % c.ngz]), xbuf(k), (float*)dW[k], k);
    g.split_k = 1;
    g.split_scratch = nullptr;
    // g_z of layer k (all of V_k) and x_k (all of R_{k-1}); a K-split product shares its meeting
    // place with the previous weight vjp
    D[(size_t)(k - l0)] = a.add(g, at_or(GV, k), at_or(GR, k - 1), g.split_k > 1 ? at_or(D, k - 1) : -1);
    gz_reader[k % c.ngz] = D[(size_t)(k - l0)];
  };
  for (int l = l0; l < l1; ++l) {
    const bool more = l + 1 < L;
    const bool want_h = more && !is_reseed(n, l + 1);
    const bool want_v = dW[l] != nullptr || want_h;
    if (want_v) {
      GV[(size_t)(l - l0)] = a.group();
      const TcGemm full = vijp_product(c, l, want_h, dW[l] != nullptr);
      for (int m = 0; m < mt; ++m) {
        TcGemm g = full;
        g.M = rb;
        g.split_k = 1;         // (the chains run side by side: no shared meeting place)
        g.split_scratch = nullptr;
        g.A.base = static_cast<const __nv_bfloat16*>(full.A.base) + m * blk;
        g.A.rows = rb;
        TcEpilogue& e = g.epi;
        e.mask += (int64_t)m * rb * (d / 32);
        if (e.frag_off) { e.frag_off += (int64_t)m * rb; e.frag_rank += (int64_t)m * rb * (d / 64); }
        if (e.planes) e.planes += m * blk;
        if (e.planes2) e.planes2 += m * blk;
        // the chain's last V made h_l[rows m] (or, at a checkpoint, was the last to use the slot
        // h_{l+1} goes to); the g_z slot this product overwrites must have been read
        Vprev[(size_t)m] = a.add_to(g, GV[(size_t)(l - l0)], Vprev[(size_t)m], gz_reader[l % c.ngz]);
      }
    }
    if (more) {
      GR[(size_t)(l - l0)] = a.group();
      const __nv_bfloat16* Wp = nullptr;
      MW_TRY(weight_planes(c, l, params[l], false, &Wp));
      const TcGemm full = recompute_product(c, l, xbuf(l), Wp);
      for (int m = 0; m < mt; ++m) {
        TcGemm g = full;
        g.M = rb;
        g.split_k = 1;
        g.split_scratch = nullptr;
        g.A.base = static_cast<const __nv_bfloat16*>(full.A.base) + m * blk;
        g.A.rows = rb;
        g.epi.mask += (int64_t)m * rb * (d / 32);
        g.epi.planes += m * blk;
        // R_{l-1,m} made x_l[rows m]; the slot x_{l+1} goes to held x_{l+1-nx}, which the weight
        // vjp of that layer read
        Rprev[(size_t)m] = a.add_to(g, GR[(size_t)(l - l0)], Rprev[(size_t)m], at_or(D, l + 1 - c.nx));
      }
    }
    // the weight vjp of the layer before comes after this layer's chain products in the list:
    // by then its g_z is usually complete
    if (l - 1 >= l0) weight_vjp(l - 1);
    MW_TRY(a.status);
  }
  weight_vjp(l1 - 1);
  return a.status;
}

inline uint32_t __float_as_uint_host(float f) {
  uint32_t u;
  memcpy(&u, &f, sizeof(u));
  return u;
}

// entries of the product table per layer of a chained sweep
int chain_entries_per_layer(const Ctx& c, bool pair) { return 2 * (c.B / (pair ? 256 : 128)) + 3; }

// backprop's reverse pass as one launch: B_l (h_{l} -> g_z of layer l-1) and D_l read the same g_z
mw_status backprop_program(const Ctx& c, const void* const* params, const void* x, void* const* dW,
                           const __nv_bfloat16* x0p) {
  const Layout& lay = *c.lay;
  mw_net* n = c.n;
  const int L = n->L, d = c.dim;
  const std::vector<const void*> key = key_of(c, params, x, nullptr, dW);
  if (!program_ready(c, MW_PROG_BP_BWD, key)) {
    Adder a{c, program_begin(c, MW_PROG_BP_BWD, 1)};
    int prevB = -1, prevD = -1, cur = 0;
    for (int l = L - 1; l >= 0; --l) {
      const __nv_bfloat16* gz = c.at<__nv_bfloat16>(lay.hp[cur]);
      const __nv_bfloat16* xl = l == 0 ? x0p : c.at<__nv_bfloat16>(lay.stored_act[l]);
      int thisD = -1, thisB = -1;
      if (dW[l]) {
        TcGemm g = weight_vjp_product(c, gz, xl, (float*)dW[l]);
        thisD = a.add(g, prevB, g.split_k > 1 ? prevD : -1);
      }
      if (l > 0) {
        const __nv_bfloat16* Wp = nullptr;
        MW_TRY(weight_planes(c, l, params[l], false, &Wp));
        const mw_layer_desc& below = n->layers[l - 1];
        TcEpilogue e;
        e.mode = TC_EPI_BWD;
        e.act = below.act;
        e.slope = (float)below.slope;
        e.mask = c.at<uint32_t>(lay.mask[l - 1]);
        e.planes = c.at<__nv_bfloat16>(lay.hp[cur ^ 1]);
        e.n_planes = c.pr.pg2;
        e.plane_stride = c.bn;
        // writes the slot that held g_z of layer l+1: its weight vjp must have read it
        thisB = a.add(product(c, operand(gz, c.B, d, c.pr.pg2, false), operand(Wp, d, d, c.pr.pw, true),
                              c.B, d, d, e, 0), prevB, prevD);
      }
      prevB = thisB;
      if (thisD >= 0) prevD = thisD;
      cur ^= 1;
    }
    MW_TRY(a.status);
    state_of(c)->key[MW_PROG_BP_BWD][0] = key;
  }
  return tc_program_launch(state_of(c)->prog[MW_PROG_BP_BWD][0], c.st, c.s);
}

}  // namespace

bool tensor_supported(const mw_net* n) {
  if (n->layers[0].kind == MW_CONV1D) return conv1d_tensor_supported(n);
  if (n->layers[0].kind == MW_CONV2D)
    return n->layers[0].stride == 1 ? conv_tensor_supported(n) : sconv_tensor_supported(n);
  if (n->opts.prec != MW_F32 && n->opts.prec != MW_BF16_F32ACC) return false;
  if (n->opts.loss == MW_LOSS_XENT_MEAN) return false;
  const int d = n->layers[0].n_in;
  for (const auto& l : n->layers) {
    if (l.kind != MW_DENSE) return false;
    if (l.n_in != d || d % 64 != 0) return false;
    if (l.act == MW_ACT_LEAKY_RELU && !(l.slope != 0.0)) return false;
  }
  return true;
}

void tensor_layout(mw_net* n, bool backprop, Layout& lay, size_t start) {
  struct B2 {
    size_t cur;
    Region take(size_t bytes) {
      Region r; r.off = cur; r.bytes = bytes; cur = align_up(cur + bytes, 256); return r;
    }
  } b{start};
  if (!n->tc) {
    TensorState* t = new TensorState();
    t->cache = tc_cache_create();
    n->tc = t;
  }
  if (n->layers[0].kind == MW_CONV1D) {
    conv1d_tensor_layout(n, backprop, lay, start);
    return;
  }
  if (n->layers[0].kind == MW_CONV2D) {
    if (n->layers[0].stride == 1) conv_tensor_layout(n, backprop, lay, start);
    else sconv_tensor_layout(n, backprop, lay, start);
    return;
  }
  const Prec pr = prec_of(n);
  const int L = n->L;
  const size_t d = (size_t)n->layers[0].n_in;
  const size_t bn = (size_t)n->B * d, nn = d * d;
  const bool resident = n->opts.resident_inverse != 0;
  lay.z = b.take(4 * bn);                                   // fp32 network output
  for (int i = 0; i < 2; ++i) lay.cot[i] = b.take(4 * bn);  // fp32 cotangent scratch (loss top)
  // (two more x slots and two more g_z slots where the sweep runs as chains: see Ctx)
  const bool chains = !backprop && chain_sizes(n);
  for (int i = 0; i < (chains ? 5 : 3); ++i) lay.xp[i] = b.take(2 * (size_t)pr.px * bn);
  const int hpl = pr.ph > pr.pg2 ? pr.ph : pr.pg2;
  for (int i = 0; i < 2; ++i) lay.hp[i] = b.take(2 * (size_t)hpl * bn);
  for (int i = 0; i < (chains ? 4 : 2); ++i)
    lay.gzp[i] = b.take(2 * (size_t)(pr.pgw > pr.pg2 ? pr.pgw : pr.pg2) * bn);
  // K-split meeting places: slot 0 recompute / Phase I / Phase II, slot 1 vijp, slot 2 weight vjp
  {
    const int B = n->B, dd = (int)d;
    auto need = [&](int pa, int pb, int M, int N, int K) {
      return tc_split_scratch_bytes(pa, pb, M, N, 1, tc_auto_split(pa, pb, M, N, K, 1));
    };
    size_t s0 = need(pr.px, pr.pw, B, dd, dd);
    const size_t s0b = need(pr.pg2, pr.pw, B, dd, dd);
    if (s0b > s0) s0 = s0b;
    const size_t s1 = need(pr.ph, pr.ph, B, dd, dd);
    const size_t s2 = need(pr.pgw, pr.pxw, dd, dd, B);
    if (s0) lay.split[0] = b.take(s0);
    if (s1 && !backprop) lay.split[1] = b.take(s1);
    if (s2) lay.split[2] = b.take(s2);
  }
  if (use_programs(n)) {
    const int progs = 2;     // Phase I / Phase II, or backprop's forward / reverse pass
    // (table 0 also holds the chained forward sweep: up to kTcMaxProgram entries)
    for (int i = 0; i < progs; ++i) {
      const size_t entries = (i == 0 && !backprop) ? (size_t)kTcMaxProgram : 5 * (size_t)(L + 1);
      lay.prog_table[i] = b.take(tc_program_table_bytes((int)entries));
      lay.prog_done[i] = b.take(sizeof(unsigned int) * (entries + 1));
    }
  }
  if (n->opts.prec == MW_F32) {
    if (resident) {
      for (int l = 0; l < L; ++l) lay.w_planes[l] = b.take(2 * 3 * nn);
    } else {
      Region slot = b.take(2 * 3 * nn);
      for (int l = 0; l < L; ++l) lay.w_planes[l] = slot;
    }
  }
  if (n->opts.lu_param) {
    const size_t G = (size_t)lu_chunk(n);
    lay.lu_l = b.take(6 * nn * G);
    lay.lu_u = b.take(6 * nn * G);
    lay.lu_g = b.take(6 * nn * G);
    lay.lu_a = b.take(4 * nn * G);
    lay.lu_b = b.take(4 * nn * G);
    lay.lu_table = b.take(tc_program_table_bytes(kLuProgEntries));
    lay.lu_done = b.take(sizeof(unsigned int) * (kLuProgEntries + 1));
    if (!backprop) {
      lay.lu_t = b.take(6 * nn * G);
      lay.lu_s = b.take(6 * nn * G);
      for (int i = 0; i < 2; ++i) lay.lu_y[i] = b.take(6 * nn * G);
      lay.lu_diag = b.take(sizeof(float) * 2 * G * d * kLuBlock);
      for (int l = 0; l < L; ++l) lay.inv[l] = b.take(2 * (size_t)pr.ph * nn);
    }
    lay.total = b.cur;
    return;
  }
  if (!backprop) {
    if (use_programs(n)) {
      // the inverses stay where the last Newton-Schulz step wrote them (ns_r)
    } else if (resident) {
      for (int l = 0; l < L; ++l) lay.inv[l] = b.take(2 * (size_t)pr.ph * nn);
    } else {
      Region slot = b.take(2 * (size_t)pr.ph * nn);
      for (int l = 0; l < L; ++l) lay.inv[l] = slot;
    }
    // program path: every layer keeps its own Newton-Schulz iterate
    const size_t G = use_programs(n) ? (size_t)L : (size_t)ns_group(n);
    lay.ns_sumsq = b.take(sizeof(double) * gate_slots((int)d) * G);
    lay.ns_scale = b.take(sizeof(float) * (size_t)L);
    lay.ns_x = b.take(4 * nn * G);
    lay.ns_r = b.take(2 * 9 * nn * G);  // per group member: R planes [3] + two iterate plane sets
    if (n->opts.prec != MW_F32 && G > 1 && !use_programs(n)) lay.ns_w = b.take(2 * nn * G);
    lay.inv_scratch = b.take(12 * kMaxGroup + 64 + 8 * (size_t)kMaxGroup * kFrobBlocks);
  }
  lay.total = b.cur;
}

void tensor_destroy(mw_net* n) {
  if (n->tc) {
    TensorState* t = static_cast<TensorState*>(n->tc);
    for (int i = 0; i < MW_PROG_COUNT; ++i)
      for (int v = 0; v < kProgVariants; ++v)
        if (t->prog[i][v]) tc_program_destroy(t->prog[i][v]);
    for (int v = 0; v < 2; ++v)
      for (TcProgram* pr : t->sweep[v]) tc_program_destroy(pr);
    for (int v = 0; v < 2; ++v)
      for (TcProgram* pr : t->lu_prog[v])
        if (pr) tc_program_destroy(pr);
    tc_cache_destroy(t->cache);
    delete t;
    n->tc = nullptr;
  }
}

mw_status tensor_input_cotangent(mw_net* n, const void* const* params, const void* x,
                                 const void* target, void* g0, double* loss_out, void* ws,
                                 cudaStream_t s) {
  if (n->layers[0].kind == MW_CONV1D)
    return conv1d_tensor_input_cotangent(n, params, x, target, g0, loss_out, ws, s);
  if (n->layers[0].kind == MW_CONV2D)
    return n->layers[0].stride == 1 ? conv_tensor_input_cotangent(n, params, x, target, g0, loss_out, ws, s)
                                    : sconv_tensor_input_cotangent(n, params, x, target, g0, loss_out, ws, s);
  const Layout& lay = n->mwl;
  Ctx c = make_ctx(n, lay, ws, s);
  const int L = n->L, d = c.dim;
  MW_CUDA_OK(cudaMemsetAsync(at<char>(ws, lay.status), 0, 256, s));
  MW_TRY(clear_split_counters(c));
  const bool resident = n->opts.resident_inverse != 0;
  if (use_programs(n) && n->opts.lu_param) {
    // LU-parameterised layers: W and W^-1 come from the factors; each phase is then one launch
    MW_TRY(lu_prepare(c, params, true));
    MW_TRY(forward_program(c, params, x, false));             // Phase I
    MW_TRY(loss_and_top(c, target, loss_out, true));
    return phase2_program(c, params, g0, nullptr);            // Phase II
  }
  if (use_programs(n)) {
    // each phase is one launch, and the inverse steps of all layers ride along in both
    // a workspace that kept its inverses: refresh them (one step) instead of starting over
    const bool warm = n->opts.warm_inverse != 0 && n->warm_ws == ws;
    n->warm_ws = nullptr;
    NsFeed feed = make_feed(c, params, warm, warm ? n->inv_side : 0);
    if (feed.steps < 1) return MW_ERR_INVALID_ARG;
    MW_TRY(split_all_weights(c, params));
    if (!warm) MW_TRY(ns_prepare_all(c, params));
    // (a symmetric residual product on single CTAs leaves the pieces of its left-out tiles unwritten)
    MW_CUDA_OK(cudaMemsetAsync(c.at<char>(lay.ns_sumsq), 0, lay.ns_sumsq.bytes, s));
    MW_TRY(forward_program(c, params, x, false, &feed));      // Phase I
    MW_TRY(loss_and_top(c, target, loss_out, true));
    MW_TRY(phase2_program(c, params, g0, &feed));             // Phase II
    // the last update squares the last residual: gate on it so a diverging layer is reported.
    // From scratch the residual is spread over all directions and its rms singular value is
    // judged; a refresh must keep the LARGEST one small enough for its square to vanish in the
    // working precision (5e-4 squared for MW_F32, 4e-3 squared for the two-term bf16 chain)
    const double limit = warm ? (n->opts.prec == MW_F32 ? 5e-4 : 4e-3) : (n->opts.prec == MW_F32 ? 2e-3 : 2e-2);
    const NsStep lastst = feed.sched[feed.steps - 1];
    const int pw = c.pr.pw < lastst.pr ? c.pr.pw : lastst.pr;
    residual_gate_kernel<<<L, 256, 0, s>>>(ns_buffers(c).sumsq, (int64_t)gate_slots(d),
                                           (int64_t)tc_sumsq_slots(pw, lastst.pr, d, d, net_pair(c)), d, limit, c.st, 0,
                                           warm ? 1 : 0);
    MW_TRY(launch_ok());
    n->inv_side = (feed.side0 + feed.steps) & 1;
    if (n->opts.warm_inverse) n->warm_ws = ws;
    return MW_OK;
  }
  if (n->opts.lu_param) {
    MW_TRY(lu_prepare(c, params, true));      // W and W^-1 of every layer from its factors
  } else if (resident) {
    const int G = ns_group(n);
    for (int l = 0; l < L; l += G) MW_TRY(newton_schulz_group(c, l, (L - l) < G ? (L - l) : G, params));
  }
  MW_TRY(forward_pass(c, params, x, false));                 // Phase I
  MW_TRY(loss_and_top(c, target, loss_out, true));
  // Phase II: g_z planes ping-pong between hp[0] and hp[1]
  int cur = 0;
  for (int l = L - 1; l >= 0; --l) {
    const __nv_bfloat16* Wp = nullptr;
    MW_TRY(weight_planes(c, l, params[l], !resident, &Wp));
    TcEpilogue e;
    e.mode = TC_EPI_BWD;
    if (l == 0) {
      e.out_f32 = (float*)g0;
    } else {
      const mw_layer_desc& below = n->layers[l - 1];
      if (is_reseed(n, l)) {
        e.planes2 = c.at<__nv_bfloat16>(lay.reseed[l]);
        e.n_planes2 = c.pr.ph;
        e.plane_stride2 = c.bn;
      }
      e.act = below.act;
      e.slope = (float)below.slope;
      e.mask = c.at<uint32_t>(lay.mask[l - 1]);
      e.planes = c.at<__nv_bfloat16>(lay.hp[cur ^ 1]);
      e.n_planes = c.pr.pg2;
      e.plane_stride = c.bn;
      if (below.act == MW_ACT_RELU) {
        // the layer below is not submersive: keep the cotangent at its dead units (Section 5.1)
        MW_TRY(relu_index(c, l - 1));
        e.frag_off = c.at<uint32_t>(lay.frag_off[l - 1]);
        e.frag_rank = c.at<uint32_t>(lay.frag_rank[l - 1]);
        e.frag_vals = c.at<float>(lay.frag_vals[l - 1]);
      }
    }
    TcGemm g = product(c, operand(c.at<__nv_bfloat16>(lay.hp[cur]), c.B, d, c.pr.pg2, false),
                       operand(Wp, d, d, c.pr.pw, true), c.B, d, d, e, 0);
    MW_TRY(run(c, &g, 1));
    cur ^= 1;
  }
  return MW_OK;
}

mw_status tensor_forward_sweep(mw_net* n, const void* const* params, const void* x, const void* g0,
                               void* const* dW, void* ws, cudaStream_t s) {
  if (n->layers[0].kind == MW_CONV1D) return conv1d_tensor_forward_sweep(n, params, x, g0, dW, ws, s);
  if (n->layers[0].kind == MW_CONV2D)
    return n->layers[0].stride == 1 ? conv_tensor_forward_sweep(n, params, x, g0, dW, ws, s)
                                    : sconv_tensor_forward_sweep(n, params, x, g0, dW, ws, s);
  const Layout& lay = n->mwl;
  Ctx c = make_ctx(n, lay, ws, s);
  const int L = n->L, d = c.dim;
  const bool resident = n->opts.resident_inverse != 0;
  const __nv_bfloat16* x0p = nullptr;
  MW_TRY(input_planes(c, x, &x0p));
  MW_TRY(split_planes((const float*)g0, c.bn, c.at<__nv_bfloat16>(lay.hp[0]), c.pr.ph, c.bn, s));
  // Nets whose products all run in the pair form (bf16 storage, sizes multiples of 256): the sweep
  // as chains of products inside program launches, as many layers per launch as the table holds.
  if (use_programs(n) && chain_sizes(n) && g_sweep_chains) {
    TensorState* t = state_of(c);
    // The chains of one layer are (B / 256) x (d / 256) pair tiles per product; with few of them
    // most pairs wait on the chain's critical path, and tiles of 128 rows on single CTAs (four
    // times as many, each half as long) finish the sweep sooner.
    const bool pair = net_pair(c) && (g_sweep_chains == 2 || (c.B / 256) * (c.dim / 256) >= 32);
    const int per_layer = chain_entries_per_layer(c, pair);
    int chunk = (kTcMaxProgram - 4) / per_layer;
    // gradient buckets (mw_sweep_bucket_events): a launch per bucket, so that each bucket's event
    // can be recorded while the later layers still run
    if (n->bucket_layers > 0 && n->bucket_layers < chunk) chunk = n->bucket_layers;
    if (chunk >= 1) {
      const int nchunks = (L + chunk - 1) / chunk;
      std::vector<const void*> key = key_of(c, params, x, nullptr, dW);
      // the fused update (mw_forward_sweep_apply) changes the weight vjp's epilogue
      key.push_back(n->apply_params);
      key.push_back(reinterpret_cast<const void*>((uintptr_t)__float_as_uint_host(n->apply_lr)));
      const int v = n->inv_side & 1;       // the programs name the inverses' current home
      std::vector<TcProgram*>& progs = t->sweep[v];
      if (t->sweep_key[v] != key || (int)progs.size() != nchunks) {
        t->sweep_key[v].clear();
        while ((int)progs.size() < nchunks) progs.push_back(tc_program_create());
        while ((int)progs.size() > nchunks) { tc_program_destroy(progs.back()); progs.pop_back(); }
        for (int i = 0; i < nchunks; ++i) {
          const int l0 = i * chunk, l1 = l0 + chunk < L ? l0 + chunk : L;
          MW_TRY(sweep_chain_program(c, progs[(size_t)i], l0, l1, params, dW, x0p, pair));
        }
        t->sweep_key[v] = key;
      }
      for (int i = 0; i < nchunks; ++i) {
        MW_TRY(tc_program_launch(progs[(size_t)i], c.st, c.s));
        const int l1 = (i + 1) * chunk < L ? (i + 1) * chunk : L;
        // LU-parameterised layers: the gradients of W just formed become those of the factors
        if (n->opts.lu_param) MW_TRY(lu_map_gradients(c, params, dW, i * chunk, l1));
        record_buckets(n, l1, c.s);
      }
      return MW_OK;
    }
  }
  // otherwise one launch per layer (for nets of small products the whole sweep as one program
  // launch measured slower: its chains leave little for the waiting CTAs to do)
  auto xbuf = [&](int l) -> const __nv_bfloat16* {          // term planes of x_l
    return l == 0 ? x0p : c.at<__nv_bfloat16>(lay.xp[l % 3]);
  };
  // launch l: recompute x_{l+1} and vijp of layer l, with the weight vjp of layer l-1
  for (int l = 0; l <= L; ++l) {
    TcGemm g[3];
    int cnt = 0;
    if (l < L) {
      const bool more = l + 1 < L;
      const bool want_h = more && !is_reseed(n, l + 1);
      if (!resident) MW_TRY(newton_schulz_group(c, l, 1, params));   // W^-1 (and W planes) of this layer
      if (more) {
        const __nv_bfloat16* Wp = nullptr;
        MW_TRY(weight_planes(c, l, params[l], false, &Wp));
        g[cnt++] = recompute_product(c, l, xbuf(l), Wp);
      }
      if (dW[l] || want_h) g[cnt++] = vijp_product(c, l, want_h, dW[l] != nullptr);
    }
    if (l >= 1 && dW[l - 1])
      g[cnt++] = weight_vjp_product(c, c.at<__nv_bfloat16>(lay.gzp[(l - 1) & 1]), xbuf(l - 1),
                                    (float*)dW[l - 1], l - 1);
    if (cnt) MW_TRY(run(c, g, cnt));
    // LU-parameterised layer: the gradient of W just formed becomes the gradient of the factors
    if (n->opts.lu_param && l >= 1) MW_TRY(lu_map_gradients(c, params, dW, l - 1, l));
    record_buckets(n, l, c.s);      // launch l carries the weight vjp of layer l - 1
  }
  return MW_OK;
}

mw_status tensor_backprop(mw_net* n, const void* const* params, const void* x, const void* target,
                          void* const* dW, double* loss_out, void* ws, cudaStream_t s) {
  if (n->layers[0].kind == MW_CONV1D)
    return conv1d_tensor_backprop(n, params, x, target, dW, loss_out, ws, s);
  if (n->layers[0].kind == MW_CONV2D)
    return n->layers[0].stride == 1 ? conv_tensor_backprop(n, params, x, target, dW, loss_out, ws, s)
                                    : sconv_tensor_backprop(n, params, x, target, dW, loss_out, ws, s);
  const Layout& lay = n->bpl;
  Ctx c = make_ctx(n, lay, ws, s);
  const int L = n->L, d = c.dim;
  MW_CUDA_OK(cudaMemsetAsync(at<char>(ws, lay.status), 0, 256, s));
  MW_TRY(clear_split_counters(c));
  const bool programs = use_programs(n);
  if (programs) {
    if (n->opts.lu_param) MW_TRY(lu_prepare(c, params, false));
    else MW_TRY(split_all_weights(c, params));
    MW_TRY(forward_program(c, params, x, true));
  } else {
    if (n->opts.lu_param) MW_TRY(lu_prepare(c, params, false));
    MW_TRY(forward_pass(c, params, x, true));
  }
  MW_TRY(loss_and_top(c, target, loss_out, false));
  const __nv_bfloat16* x0p = nullptr;
  if (n->opts.prec == MW_F32) x0p = c.at<__nv_bfloat16>(lay.xp[0]);   // split by the forward pass
  else x0p = (const __nv_bfloat16*)x;
  if (programs) {
    MW_TRY(backprop_program(c, params, x, dW, x0p));
    if (n->opts.lu_param) MW_TRY(lu_map_gradients(c, params, dW, 0, L));
    return MW_OK;
  }
  int cur = 0;
  // one launch per layer: both vjps of layer l read the same g_z
  for (int l = L - 1; l >= 0; --l) {
    const __nv_bfloat16* gz = c.at<__nv_bfloat16>(lay.hp[cur]);
    const __nv_bfloat16* xl = l == 0 ? x0p : c.at<__nv_bfloat16>(lay.stored_act[l]);
    TcGemm g[2];
    int cnt = 0;
    if (l > 0) {
      const __nv_bfloat16* Wp = nullptr;
      // resident: the planes made by forward_pass are still there (MW_F32)
      MW_TRY(weight_planes(c, l, params[l], n->opts.resident_inverse == 0, &Wp));
      const mw_layer_desc& below = n->layers[l - 1];
      TcEpilogue e;
      e.mode = TC_EPI_BWD;
      e.act = below.act;
      e.slope = (float)below.slope;
      e.mask = c.at<uint32_t>(lay.mask[l - 1]);
      e.planes = c.at<__nv_bfloat16>(lay.hp[cur ^ 1]);
      e.n_planes = c.pr.pg2;
      e.plane_stride = c.bn;
      g[cnt++] = product(c, operand(gz, c.B, d, c.pr.pg2, false), operand(Wp, d, d, c.pr.pw, true),
                         c.B, d, d, e, 0);
    }
    if (dW[l]) {
      TcEpilogue e;
      e.mode = TC_EPI_PLAIN;
      e.out_f32 = (float*)dW[l];
      g[cnt++] = product(c, operand(gz, c.B, d, c.pr.pgw, true), operand(xl, c.B, d, c.pr.pxw, true),
                         d, d, c.B, e, 2);
    }
    if (cnt) MW_TRY(run(c, g, cnt));
    if (n->opts.lu_param) MW_TRY(lu_map_gradients(c, params, dW, l, l + 1));
    cur ^= 1;
  }
  return MW_OK;
}

}  // namespace mw
