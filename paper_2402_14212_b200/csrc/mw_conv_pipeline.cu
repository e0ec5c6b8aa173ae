// Tensor-core pipelines of the three calls for convolutional nets (MW_F32): a chain of stride-1,
// same-size, 64-channel convolutions with leaky-ReLU (or no) activation, optionally closed by a
// linear head on the flattened activation.
//
// Every convolution step is a product of the persistent tcgen05 kernel with a shifted-window A
// operand (mw_conv_tensor.cu); activations and cotangents travel as three bf16 term planes.
//   Phase I    x_{l+1} = phi(conv(x_l, w_l))              -> sign words + term planes   (Section 4.1)
//   Phase II   h_l = TransposeConv(g_z, w_l)              -> checkpoint (fp32) + next g_z planes
//   sweep      recompute x_{l+1}; vijp of the convolution: the g with TransposeConv(g, w_l) = h_l,
//              by the elimination relation of Lemma 1's proof outline used as a fixed-point
//              iteration on the whole centre tap W_c,
//                  g <- h W_c^-T - TransposeConv(g, w^),   w^[j] = W_c^-1 w[j] (0 at the centre),
//              started from g = h W_c^-T, early updates in fewer bf16 terms (their error is
//              contracted away by the later ones); the last update carries the activation's
//              vijp in its epilogue (Eq. "h_i"); then dw_l = weight vjp(x_l, g_z) (Eq. "g_i").
// The head (10 x 65536) and the loss run on CUDA cores.
#include "mw_conv_tensor.cuh"
#include "mw_tensor.cuh"

namespace mw {

namespace {

struct CCtx {
  mw_net* n;
  const Layout* lay;
  void* ws;
  cudaStream_t s;
  TcMapCache* cache;
  DeviceStatus* st;
  ConvGeom g;
  int Lc;            // convolution layers
  bool head;
  int64_t P;         // elements of one activation (pixels * 64)
  int64_t we;        // elements of one kernel
  template <typename T> T* at(const Region& r) const { return mw::at<T>(ws, r); }
};

CCtx make_cctx(mw_net* n, const Layout& lay, void* ws, cudaStream_t s) {
  CCtx c;
  c.n = n; c.lay = &lay; c.ws = ws; c.s = s;
  c.cache = static_cast<TensorState*>(n->tc)->cache;
  c.st = status_of(ws, lay);
  const mw_layer_desc& d = n->layers[0];
  c.g = ConvGeom{n->B, d.H, d.W, d.k, d.pad};
  c.head = n->layers[n->L - 1].kind == MW_HEAD_LINEAR;
  c.Lc = c.head ? n->L - 1 : n->L;
  c.P = c.g.pixels() * 64;
  c.we = (int64_t)d.k * d.k * 4096;
  return c;
}

// terms of the operands of update t (1-based) of `T`: the last two updates are fp32-accurate, the
// three before them carry two terms, earlier ones one.  An update's rounding error (4e-3, 1.5e-5,
// 1e-7 relative for 1, 2, 3 terms) is contracted by the later updates (0.14 each for the default
// kernels): two later updates take a two-term error to 3e-7, five take a one-term error there.
int update_terms(int t, int T) {
  const int left = T - t;
  return left < 2 ? 3 : (left < 5 ? 2 : 1);
}

// w^[tap] = Winv w[tap] for tap != centre, zero at the centre; one block per (tap, row, layer)
__global__ void __launch_bounds__(64)
fold_kernel(SmallBatch ws, const float* __restrict__ winv0, int centre, int64_t we,
            float* __restrict__ what0) {
  const int tap = blockIdx.x, c = blockIdx.y, cp = threadIdx.x;
  const float* w = static_cast<const float*>(ws.p[blockIdx.z]);
  const float* winv = winv0 + (int64_t)blockIdx.z * 4096;
  float* what = what0 + (int64_t)blockIdx.z * we;
  float a = 0.f;
  if (tap != centre)
    for (int m = 0; m < 64; ++m) a = fmaf(winv[c * 64 + m], w[((int64_t)tap * 64 + m) * 64 + cp], a);
  what[((int64_t)tap * 64 + c) * 64 + cp] = a;
}

// per-step preparation of layers [l0, l0 + G): kernel term planes, centre-tap inverses, folded
// kernels, G <= kSmallBatch layers per launch
mw_status prep_layers(const CCtx& c, int l0, int G, const void* const* params, bool inverse) {
  const Layout& lay = *c.lay;
  for (int g = 0; g < G; ++g)
    MW_TRY(split_planes((const float*)params[l0 + g], c.we, c.at<__nv_bfloat16>(lay.cw[l0 + g]), 3, c.we, c.s));
  if (!inverse) return MW_OK;
  const int centre = c.g.pad * c.g.k + c.g.pad;
  float* winv = c.at<float>(lay.cwinv_f32);      // [kSmallBatch][64*64]
  float* what = c.at<float>(lay.cwhat_f32);      // [kSmallBatch][k*k*64*64]
  SmallBatch ws{};
  for (int g = 0; g < G; ++g) ws.p[g] = params[l0 + g];
  MW_TRY(inverse_small_batch<float>(ws, G, (int64_t)centre * 4096, 64, winv, c.st, l0, c.s));
  fold_kernel<<<dim3(c.g.k * c.g.k, 64, G), 64, 0, c.s>>>(ws, winv, centre, c.we, what);
  MW_TRY(launch_ok());
  for (int g = 0; g < G; ++g) {
    MW_TRY(split_planes(winv + (int64_t)g * 4096, 4096, c.at<__nv_bfloat16>(lay.cwinv[l0 + g]), 3, 4096, c.s));
    MW_TRY(split_planes(what + (int64_t)g * c.we, c.we, c.at<__nv_bfloat16>(lay.cwhat[l0 + g]), 3, c.we, c.s));
  }
  return MW_OK;
}

mw_status prep_layer(const CCtx& c, int l, const void* const* params, bool inverse) {
  return prep_layers(c, l, 1, params, inverse);
}

// ---- the linear head (a few outputs over a very long row) on CUDA cores -------------------
// logits[b][o] = sum_k x[b][k] W[o][k]: one CTA per (o, b)
__global__ void __launch_bounds__(256)
head_forward_kernel(const float* __restrict__ x, const float* __restrict__ W, int64_t nf, int no,
                    float* __restrict__ logits) {
  __shared__ float red[256];
  const int o = blockIdx.x, b = blockIdx.y;
  const float4* xr = reinterpret_cast<const float4*>(x + (int64_t)b * nf);
  const float4* wr = reinterpret_cast<const float4*>(W + (int64_t)o * nf);
  float a = 0.f;
  for (int64_t i = threadIdx.x; i < nf / 4; i += 256) {
    const float4 u = xr[i], v = wr[i];
    a = fmaf(u.x, v.x, fmaf(u.y, v.y, fmaf(u.z, v.z, fmaf(u.w, v.w, a))));
  }
  red[threadIdx.x] = a;
  __syncthreads();
  for (int s = 128; s; s >>= 1) {
    if (threadIdx.x < s) red[threadIdx.x] += red[threadIdx.x + s];
    __syncthreads();
  }
  if (threadIdx.x == 0) logits[(int64_t)b * no + o] = red[0];
}

// h[b][k] = sum_o hl[b][o] W[o][k]
__global__ void __launch_bounds__(256)
head_backward_kernel(const float* __restrict__ hl, const float* __restrict__ W, int64_t nf, int no,
                     float* __restrict__ h) {
  const int b = blockIdx.y;
  const int64_t k = (int64_t)blockIdx.x * 256 + threadIdx.x;
  if (k >= nf) return;
  float a = 0.f;
  for (int o = 0; o < no; ++o) a = fmaf(hl[(int64_t)b * no + o], W[(int64_t)o * nf + k], a);
  h[(int64_t)b * nf + k] = a;
}

// dW[o][k] = sum_b hl[b][o] x[b][k]
__global__ void __launch_bounds__(256)
head_wgrad_kernel(const float* __restrict__ hl, const float* __restrict__ x, int64_t nf, int no, int B,
                  float* __restrict__ dW, const float* theta = nullptr, float lr = 0.f) {
  const int o = blockIdx.y;
  const int64_t k = (int64_t)blockIdx.x * 256 + threadIdx.x;
  if (k >= nf) return;
  float a = 0.f;
  for (int b = 0; b < B; ++b) a = fmaf(hl[(int64_t)b * no + o], x[(int64_t)b * nf + k], a);
  dW[(int64_t)o * nf + k] = theta ? fmaf(-lr, a, theta[(int64_t)o * nf + k]) : a;   // fused update
}

// Phase I (or backprop's forward).  x_{l+1} planes go to the stores (backprop) or rotate; the
// last convolution's output also lands in fp32 (lay.cxf) for the head / the loss.
mw_status conv_forward_pass(const CCtx& c, const void* const* params, const void* x, bool store_acts) {
  const Layout& lay = *c.lay;
  MW_TRY(split_planes((const float*)x, c.P, c.at<__nv_bfloat16>(lay.xp[0]), 3, c.P, c.s));
  const __nv_bfloat16* xin = c.at<__nv_bfloat16>(lay.xp[0]);
  for (int l0 = 0; l0 < c.Lc; l0 += kSmallBatch)
    MW_TRY(prep_layers(c, l0, (c.Lc - l0) < kSmallBatch ? (c.Lc - l0) : kSmallBatch, params,
                       !store_acts && c.n->opts.resident_inverse));
  for (int l = 0; l < c.Lc; ++l) {
    const mw_layer_desc& ld = c.n->layers[l];
    const bool last = l + 1 == c.Lc;
    __nv_bfloat16* xout = (store_acts && l + 1 < c.n->L) ? c.at<__nv_bfloat16>(lay.stored_act[l + 1])
                                                        : c.at<__nv_bfloat16>(lay.xp[(l + 1) % 3]);
    TcEpilogue e;
    e.mode = TC_EPI_FWD;
    e.mask = c.at<uint32_t>(lay.mask[l]);
    e.write_mask = 1;
    e.act = ld.act;
    e.slope = (float)ld.slope;
    if (!last || (store_acts && c.head)) { e.planes = xout; e.n_planes = 3; e.plane_stride = c.P; }
    if (last) e.out_f32 = c.at<float>(lay.cxf);
    TcGemm g = conv_forward_product(c.g, xin, 3, c.at<__nv_bfloat16>(lay.cw[l]), 3, e);
    MW_TRY(tc_gemm_group(c.cache, &g, 1, c.st, c.s));
    xin = xout;
  }
  return MW_OK;
}

// loss on top of the last convolution (through the head when there is one); leaves h wrt the
// last convolution's output in cot[0] (fp32) and the head's cotangent in h_last
mw_status conv_loss_top(const CCtx& c, const void* const* params, const void* target,
                        double* loss_out, bool keep_head_cotangent) {
  const Layout& lay = *c.lay;
  const int L = c.n->L;
  float* xf = c.at<float>(lay.cxf);
  float* h = c.at<float>(lay.cot[0]);
  if (c.head) {
    const mw_layer_desc& hd = c.n->layers[L - 1];
    float* logits = c.at<float>(lay.clogits);
    float* hl = logits + (int64_t)c.n->B * hd.n_out;
    if (hd.n_in % 4 != 0) return MW_ERR_UNSUPPORTED;
    head_forward_kernel<<<dim3(hd.n_out, c.n->B), 256, 0, c.s>>>(xf, (const float*)params[L - 1], hd.n_in,
                                                               hd.n_out, logits);
    MW_TRY(launch_ok());
    MW_TRY(loss_cotangent<float>(logits, target, c.n->B, hd.n_out, c.n->opts.loss, hl,
                                 c.at<double>(lay.partials), loss_out, c.s));
    if (keep_head_cotangent)
      MW_CUDA_OK(cudaMemcpyAsync(c.at<float>(lay.h_last), hl, sizeof(float) * c.n->B * hd.n_out,
                                 cudaMemcpyDeviceToDevice, c.s));
    head_backward_kernel<<<dim3((unsigned)((hd.n_in + 255) / 256), c.n->B), 256, 0, c.s>>>(
        hl, (const float*)params[L - 1], hd.n_in, hd.n_out, h);
    MW_TRY(launch_ok());
  } else {
    MW_TRY(loss_cotangent<float>(xf, target, c.g.pixels(), 64, c.n->opts.loss, h,
                                 c.at<double>(lay.partials), loss_out, c.s));
  }
  return MW_OK;
}

// g_z of the last convolution from h (fp32, cot[0]) as three term planes in hp[0]
mw_status conv_top_gz(const CCtx& c) {
  const Layout& lay = *c.lay;
  const mw_layer_desc& ld = c.n->layers[c.Lc - 1];
  const float* h = c.at<float>(lay.cot[0]);
  const float* src = h;
  if (ld.act != MW_ACT_NONE) {
    float* g = c.at<float>(lay.cot[1]);
    MW_TRY(scale_by_mask<float>(h, c.at<uint32_t>(lay.mask[c.Lc - 1]), c.g.pixels(), 64, ld.act, ld.slope,
                                g, c.s));
    src = g;
  }
  return split_planes(src, c.P, c.at<__nv_bfloat16>(lay.hp[0]), 3, c.P, c.s);
}

}  // namespace

bool conv_tensor_supported(const mw_net* n) {
  if (n->opts.prec != MW_F32) return false;
  const mw_layer_desc& d0 = n->layers[0];
  if (d0.kind != MW_CONV2D) return false;
  const int L = n->L;
  for (int l = 0; l < L; ++l) {
    const mw_layer_desc& d = n->layers[l];
    if (d.kind == MW_HEAD_LINEAR) {
      if (l != L - 1) return false;
      continue;
    }
    if (d.kind != MW_CONV2D) return false;
    if (d.C_in != 64 || d.C_out != 64 || d.H != d0.H || d.W != d0.W || d.k != d0.k || d.pad != d0.pad)
      return false;
    if (d.act == MW_ACT_RELU) return false;
    if (d.act == MW_ACT_LEAKY_RELU && !(d.slope != 0.0)) return false;
  }
  if (d0.W > 64 || 64 % d0.W != 0 || d0.H % (128 / d0.W) != 0 || (d0.H * d0.W) % 128 != 0) return false;
  if (d0.k * d0.k > 64 || !(d0.k & 1)) return false;
  if ((int64_t)n->B * d0.H * d0.W >= ((int64_t)1 << 31) / 64) return false;
  if (n->layers[L - 1].kind != MW_HEAD_LINEAR && n->opts.loss == MW_LOSS_XENT_MEAN) return false;
  return true;
}

void conv_tensor_layout(mw_net* n, bool backprop, Layout& lay, size_t start) {
  struct B2 {
    size_t cur;
    Region take(size_t bytes) {
      Region r; r.off = cur; r.bytes = bytes; cur = align_up(cur + bytes, 256); return r;
    }
  } b{start};
  const mw_layer_desc& d = n->layers[0];
  const int L = n->L;
  const bool head = n->layers[L - 1].kind == MW_HEAD_LINEAR;
  const int Lc = head ? L - 1 : L;
  const size_t P = (size_t)n->B * d.H * d.W * 64;
  const size_t we = (size_t)d.k * d.k * 4096;
  for (int i = 0; i < 2; ++i) lay.cot[i] = b.take(4 * P);
  lay.cxf = b.take(4 * P);
  for (int i = 0; i < 3; ++i) lay.xp[i] = b.take(2 * 3 * P);
  for (int i = 0; i < 2; ++i) lay.hp[i] = b.take(2 * 3 * P);
  lay.cw.resize(L); lay.cwhat.resize(L); lay.cwinv.resize(L);
  for (int l = 0; l < Lc; ++l) lay.cw[l] = b.take(2 * 3 * we);
  if (head) lay.clogits = b.take(4 * 2 * (size_t)n->B * n->layers[L - 1].n_out);
  lay.cpart = b.take(4 * (size_t)conv_wgrad_tensor_slices((int64_t)n->B * d.H * d.W, 64, d.k * d.k) * we);
  if (!backprop) {
    for (int i = 0; i < 2; ++i) lay.cg[i] = b.take(2 * 3 * P);
    lay.chpf = b.take(4 * P);
    for (int l = 0; l < Lc; ++l) {
      lay.cwhat[l] = b.take(2 * 3 * we);
      lay.cwinv[l] = b.take(2 * 3 * 4096);
    }
    lay.cwinv_f32 = b.take(4 * 4096 * (size_t)kSmallBatch);
    lay.cwhat_f32 = b.take(4 * we * (size_t)kSmallBatch);
  }
  lay.total = b.cur;
}

mw_status conv_tensor_input_cotangent(mw_net* n, const void* const* params, const void* x,
                                      const void* target, void* g0, double* loss_out, void* ws,
                                      cudaStream_t s) {
  const Layout& lay = n->mwl;
  CCtx c = make_cctx(n, lay, ws, s);
  MW_CUDA_OK(cudaMemsetAsync(at<char>(ws, lay.status), 0, 256, s));
  MW_TRY(conv_forward_pass(c, params, x, false));                  // Phase I (+ per-step prep)
  MW_TRY(conv_loss_top(c, params, target, loss_out, true));
  if (c.head && is_reseed(n, c.Lc))
    MW_CUDA_OK(cudaMemcpyAsync(c.at<float>(lay.reseed[c.Lc]), c.at<float>(lay.cot[0]), 4 * c.P,
                               cudaMemcpyDeviceToDevice, s));
  MW_TRY(conv_top_gz(c));
  int cur = 0;
  for (int l = c.Lc - 1; l >= 0; --l) {                            // Phase II
    TcEpilogue e;
    e.mode = TC_EPI_BWD;
    if (l == 0) {
      e.out_f32 = (float*)g0;
    } else {
      const mw_layer_desc& below = n->layers[l - 1];
      if (is_reseed(n, l)) e.out_f32 = c.at<float>(lay.reseed[l]);
      e.act = below.act;
      e.slope = (float)below.slope;
      e.mask = c.at<uint32_t>(lay.mask[l - 1]);
      e.planes = c.at<__nv_bfloat16>(lay.hp[cur ^ 1]);
      e.n_planes = 3;
      e.plane_stride = c.P;
    }
    TcGemm g = conv_transpose_product(c.g, c.at<__nv_bfloat16>(lay.hp[cur]), 3,
                                      c.at<__nv_bfloat16>(lay.cw[l]), 3, false, e);
    MW_TRY(tc_gemm_group(c.cache, &g, 1, c.st, s));
    cur ^= 1;
  }
  return MW_OK;
}

mw_status conv_tensor_forward_sweep(mw_net* n, const void* const* params, const void* x,
                                    const void* g0, void* const* dW, void* ws, cudaStream_t s) {
  const Layout& lay = n->mwl;
  CCtx c = make_cctx(n, lay, ws, s);
  const int L = n->L, Lc = c.Lc;
  const bool resident = n->opts.resident_inverse != 0;
  const int T = n->opts.conv_vijp_iters;
  MW_TRY(split_planes((const float*)x, c.P, c.at<__nv_bfloat16>(lay.xp[0]), 3, c.P, s));
  MW_TRY(split_planes((const float*)g0, c.P, c.at<__nv_bfloat16>(lay.hp[0]), 3, c.P, s));
  float* hpf = c.at<float>(lay.chpf);
  for (int l = 0; l < Lc; ++l) {
    const mw_layer_desc& ld = n->layers[l];
    uint32_t* words = c.at<uint32_t>(lay.mask[l]);
    const __nv_bfloat16* xin = c.at<__nv_bfloat16>(lay.xp[l % 3]);
    const __nv_bfloat16* hin = c.at<__nv_bfloat16>(lay.hp[l & 1]);
    __nv_bfloat16* hout = c.at<__nv_bfloat16>(lay.hp[(l + 1) & 1]);
    const bool more = l + 1 < Lc;
    const bool reseed_next = (more || c.head) && is_reseed(n, l + 1);
    const bool want_h = more && !reseed_next;
    if (!resident) MW_TRY(prep_layer(c, l, params, true));
    // recompute x_{l+1} (the last one in fp32, for the head's weight vjp)
    if (more || (c.head && dW[L - 1])) {
      TcEpilogue e;
      e.mode = TC_EPI_FWD;
      e.mask = words;
      e.write_mask = 0;
      e.act = ld.act;
      e.slope = (float)ld.slope;
      if (more) { e.planes = c.at<__nv_bfloat16>(lay.xp[(l + 1) % 3]); e.n_planes = 3; e.plane_stride = c.P; }
      else e.out_f32 = c.at<float>(lay.cxf);
      TcGemm g = conv_forward_product(c.g, xin, 3, c.at<__nv_bfloat16>(lay.cw[l]), 3, e);
      MW_TRY(tc_gemm_group(c.cache, &g, 1, c.st, s));
    }
    // vijp of the convolution, activation vijp in the last epilogue
    if (dW[l] || want_h) {
      auto final_epilogue = [&](TcEpilogue& e) {
        e.mode = TC_EPI_VIJP;
        e.act = ld.act;
        e.slope = (float)ld.slope;
        e.mask = words;
        if (want_h) { e.planes2 = hout; e.n_planes2 = 3; e.plane_stride2 = c.P; }
        if (dW[l]) { e.planes = c.at<__nv_bfloat16>(lay.cg[T & 1]); e.n_planes = 2; e.plane_stride = c.P; }
      };
      {
        // g^(0) = h W_c^-T, kept in fp32 as the constant of the iteration
        TcGemm p;
        p.A = pixel_operand(hin, c.g.pixels(), 3, c.P, false);
        p.B.base = c.at<__nv_bfloat16>(lay.cwinv[l]); p.B.rows = 64; p.B.cols = 64; p.B.planes = 3;
        p.B.plane_stride = 4096; p.B.mn_major = false;
        p.M = (int)c.g.pixels(); p.N = 64; p.K = 64;
        if (T == 0) {
          final_epilogue(p.epi);
        } else {
          p.epi.mode = TC_EPI_PLAIN;
          p.epi.out_f32 = hpf;
          p.epi.planes = c.at<__nv_bfloat16>(lay.cg[0]);
          p.epi.n_planes = update_terms(1, T);
          p.epi.plane_stride = c.P;
        }
        MW_TRY(tc_gemm_group(c.cache, &p, 1, c.st, s));
      }
      for (int t = 1; t <= T; ++t) {
        const int terms = update_terms(t, T);
        TcEpilogue e;
        if (t == T) {
          final_epilogue(e);
        } else {
          e.mode = TC_EPI_PLAIN;
          e.planes = c.at<__nv_bfloat16>(lay.cg[t & 1]);
          e.n_planes = update_terms(t + 1, T);
          e.plane_stride = c.P;
        }
        e.alpha = -1.f;
        e.addend = hpf;
        TcGemm p = conv_transpose_product(c.g, c.at<__nv_bfloat16>(lay.cg[(t - 1) & 1]), terms,
                                          c.at<__nv_bfloat16>(lay.cwhat[l]), terms, true, e);
        MW_TRY(tc_gemm_group(c.cache, &p, 1, c.st, s));
      }
    }
    if (reseed_next && more)   // the recursion restarts from the stored cotangent h_{l+1}
      MW_TRY(split_planes(c.at<float>(lay.reseed[l + 1]), c.P, hout, 3, c.P, s));
    // weight vjp
    if (dW[l])
      MW_TRY(conv_wgrad_tensor(c.cache, c.g, xin, c.at<__nv_bfloat16>(lay.cg[T & 1]), 2,
                               c.at<float>(lay.cpart), (float*)dW[l], c.st, s,
                               n->apply_params ? (const float*)n->apply_params[l] : nullptr, n->apply_lr));
  }
  if (c.head && dW[L - 1]) {
    // the head has no vijp: its output cotangent is the loss cotangent itself
    const mw_layer_desc& hd = n->layers[L - 1];
    head_wgrad_kernel<<<dim3((unsigned)((hd.n_in + 255) / 256), hd.n_out), 256, 0, s>>>(
        c.at<float>(lay.h_last), c.at<float>(lay.cxf), hd.n_in, hd.n_out, n->B, (float*)dW[L - 1],
        n->apply_params ? (const float*)n->apply_params[L - 1] : nullptr, n->apply_lr);
    MW_TRY(launch_ok());
  }
  return MW_OK;
}

mw_status conv_tensor_backprop(mw_net* n, const void* const* params, const void* x,
                               const void* target, void* const* dW, double* loss_out, void* ws,
                               cudaStream_t s) {
  const Layout& lay = n->bpl;
  CCtx c = make_cctx(n, lay, ws, s);
  const int L = n->L;
  MW_CUDA_OK(cudaMemsetAsync(at<char>(ws, lay.status), 0, 256, s));
  MW_TRY(conv_forward_pass(c, params, x, true));
  MW_TRY(conv_loss_top(c, params, target, loss_out, false));
  if (c.head && dW[L - 1]) {
    const mw_layer_desc& hd = n->layers[L - 1];
    const float* hl = c.at<float>(lay.clogits) + (int64_t)n->B * hd.n_out;
    head_wgrad_kernel<<<dim3((unsigned)((hd.n_in + 255) / 256), hd.n_out), 256, 0, s>>>(
        hl, c.at<float>(lay.cxf), hd.n_in, hd.n_out, n->B, (float*)dW[L - 1]);
    MW_TRY(launch_ok());
  }
  MW_TRY(conv_top_gz(c));
  int cur = 0;
  for (int l = c.Lc - 1; l >= 0; --l) {
    const __nv_bfloat16* gz = c.at<__nv_bfloat16>(lay.hp[cur]);
    const __nv_bfloat16* xl = l == 0 ? c.at<__nv_bfloat16>(lay.xp[0]) : c.at<__nv_bfloat16>(lay.stored_act[l]);
    if (dW[l])
      MW_TRY(conv_wgrad_tensor(c.cache, c.g, xl, gz, 2, c.at<float>(lay.cpart), (float*)dW[l], c.st, s));
    if (l > 0) {
      const mw_layer_desc& below = n->layers[l - 1];
      TcEpilogue e;
      e.mode = TC_EPI_BWD;
      e.act = below.act;
      e.slope = (float)below.slope;
      e.mask = c.at<uint32_t>(lay.mask[l - 1]);
      e.planes = c.at<__nv_bfloat16>(lay.hp[cur ^ 1]);
      e.n_planes = 3;
      e.plane_stride = c.P;
      TcGemm g = conv_transpose_product(c.g, gz, 3, c.at<__nv_bfloat16>(lay.cw[l]), 3, false, e);
      MW_TRY(tc_gemm_group(c.cache, &g, 1, c.st, s));
      cur ^= 1;
    }
  }
  return MW_OK;
}

}  // namespace mw
