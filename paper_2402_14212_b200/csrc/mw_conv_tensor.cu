// Convolution steps on the tensor cores (stride 1, same size, 64 channels, fp32 storage).
//
// Every step is a product of the persistent tcgen05 kernel (mw_tc_gemm.cu) whose A operand is the
// channel-last activation or cotangent read through a window shifted by the tap; one K block is
// one tap.  fp32 values travel as three bf16 term planes.
//   forward        x'[i',c'] = sum_{j,c} w[j,c,c'] x[i'+j-p, c]                  (Lemma 1)
//   TransposeConv  h[i,c]    = sum_{j,c'} w[j,c,c'] h'[i+p-j, c']                (Eq. "conv-vjp")
//   weight vjp     dw[j,c,c'] = sum_{b,i'} x[b,i'+j-p,c] g_z[b,i',c']            (Eq. "g_i")
//   vijp           g <- h W_c^-T - TransposeConv(g, w^),  w^[j] = W_c^-1 w[j], 0 at the centre
#include "mw_conv_tensor.cuh"

namespace mw {

namespace {

__global__ void __launch_bounds__(256)
slice_sum_f32_kernel(const float* __restrict__ part, int64_t n, int64_t stride, int slices,
                     float* __restrict__ out, const float* theta = nullptr, float lr = 0.f) {
  const int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x;
  if (i >= n) return;
  float a = 0.f;
  for (int z = 0; z < slices; ++z) a += part[(int64_t)z * stride + i];   // fixed order
  out[i] = theta ? fmaf(-lr, a, theta[i]) : a;
}

}  // namespace

__global__ void __launch_bounds__(256)
zero_above_diagonal_kernel(float* __restrict__ tap, int C) {
  const int i = blockIdx.x * 256 + threadIdx.x;
  if (i >= C * C) return;
  const int c = i / C, cp = i - c * C;
  if (c < cp) tap[i] = 0.f;
}

mw_status conv_zero_fixed_entries(float* w, int64_t offset, int C, cudaStream_t s) {
  zero_above_diagonal_kernel<<<(C * C + 255) / 256, 256, 0, s>>>(w + offset, C);
  return launch_ok();
}

mw_status conv_slice_sum(const float* part, int64_t n, int slices, float* out, const float* theta,
                         float lr, cudaStream_t s) {
  slice_sum_f32_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(part, n, n, slices, out, theta, lr);
  return launch_ok();
}

// Slices of the pixel sum.  A slice is at most 128 K blocks where the sum is long: the tensor
// core truncates its fp32 accumulator at every instruction, a bias that grows with the length of
// one accumulation (about 1e-4 relative after 1024 K blocks) and that the fixed-order sum of the
// slices, in round-to-nearest fp32, does not have.
int conv_wgrad_tensor_slices(int64_t pixels, int C, int taps) {
  const int64_t blocks = pixels / 64;
  // output tiles of one slice: 128 rows (tap, channel) x all C columns (two-term operands)
  const int tiles = ((taps * C + 127) / 128) * (C % 128 == 0 ? C / 128 : C / 64);
  const int sms = 148;
  // Among the powers of two that divide the K blocks (at most 128 K blocks per slice where the sum
  // is long enough, at least 4), the one with the shortest estimated time: waves of `sms` units,
  // each unit about 6 us of set-up and epilogue plus 0.8 us per K block.
  int best = 1;
  double best_t = 1e30;
  for (int s = 1; s <= 256; s <<= 1) {
    if (blocks % s != 0) break;
    const int64_t kb = blocks / s;
    if (s > 1 && kb < 4) break;
    const double waves = (double)(((int64_t)tiles * s + sms - 1) / sms);
    double t = waves * (6.0 + 0.8 * (double)kb);
    if (kb > 128) t *= 4.0;     // long accumulations lose accuracy (see above): strongly disfavoured
    if (t < best_t) { best_t = t; best = s; }
  }
  return best;
}

TcOperand pixel_operand(const void* planes, int64_t pixels, int terms, int64_t plane_stride, bool mn,
                        int channels) {
  TcOperand o;
  o.base = planes;
  o.rows = (int)pixels;
  o.cols = channels;
  o.planes = terms;
  o.plane_stride = plane_stride;
  o.mn_major = mn;
  return o;
}

TcGemm conv_forward_product(const ConvGeom& g, const __nv_bfloat16* x_planes, int xt,
                            const __nv_bfloat16* w_planes, int wt, const TcEpilogue& e) {
  TcGemm p;
  const int C = g.C;
  p.A = pixel_operand(x_planes, g.pixels(), xt, g.pixels() * C, false, C);
  // w[tap][ci][co]: K = (tap, ci) rows, N = co contiguous
  p.B.base = w_planes; p.B.rows = g.k * g.k * C; p.B.cols = C; p.B.planes = wt;
  p.B.plane_stride = g.kernel_elems(); p.B.mn_major = true;
  p.M = (int)g.out_pixels(); p.N = C; p.K = g.k * g.k * C;
  p.epi = e;
  p.conv.mode = TC_CONV_PIXELS; p.conv.H = g.H; p.conv.W = g.W; p.conv.k = g.k; p.conv.pad = g.pad;
  p.conv.C = C; p.conv.stride = g.stride; p.conv.Ho = g.Ho(); p.conv.Wo = g.Wo();
  p.conv.sgn = 1;
  if (g.stride != 1) {
    // window of output pixel i' starts at stride*i' + j - pad
    int n = 0;
    for (int j0 = 0; j0 < g.k; ++j0)
      for (int j1 = 0; j1 < g.k; ++j1, ++n) {
        p.conv.dy[n] = (signed char)(j0 - g.pad);
        p.conv.dx[n] = (signed char)(j1 - g.pad);
        p.conv.tb[n] = (signed char)n;
      }
    p.conv.ntaps = n;
  }
  return p;
}

bool conv_transpose_class_product(const ConvGeom& g, int py, int px, const __nv_bfloat16* g_planes,
                                  int gt, const __nv_bfloat16* w_planes, int wt, const TcEpilogue& e,
                                  TcGemm* out) {
  TcGemm p;
  const int C = g.C, s = g.stride, Ho = g.Ho(), Wo = g.Wo();
  p.A = pixel_operand(g_planes, g.out_pixels(), gt, g.out_pixels() * C, false, C);
  // w[tap][c][c']: for one tap N = c rows, K = c' contiguous
  p.B.base = w_planes; p.B.rows = g.k * g.k * C; p.B.cols = C; p.B.planes = wt;
  p.B.plane_stride = g.kernel_elems(); p.B.mn_major = false;
  p.conv.mode = TC_CONV_PIXELS; p.conv.H = Ho; p.conv.W = Wo; p.conv.C = C; p.conv.stride = 1;
  p.conv.Ho = Ho; p.conv.Wo = Wo; p.conv.k = g.k; p.conv.pad = g.pad; p.conv.b_tap_rows = 1;
  int n = 0;
  for (int j0 = 0; j0 < g.k; ++j0) {
    const int vy = py + g.pad - j0;
    if (((vy % s) + s) % s != 0) continue;
    for (int j1 = 0; j1 < g.k; ++j1) {
      const int vx = px + g.pad - j1;
      if (((vx % s) + s) % s != 0) continue;
      // h[s y + py] takes w[j] h'[(s y + py + pad - j) / s] = h'[y + vy / s]
      p.conv.dy[n] = (signed char)(vy >= 0 ? vy / s : -((-vy) / s));
      p.conv.dx[n] = (signed char)(vx >= 0 ? vx / s : -((-vx) / s));
      p.conv.tb[n] = (signed char)(j0 * g.k + j1);
      ++n;
    }
  }
  if (n == 0) return false;
  p.conv.ntaps = n;
  p.M = (int)g.out_pixels(); p.N = C; p.K = n * C;
  p.epi = e;
  p.epi.remap_s = s; p.epi.remap_ho = Ho; p.epi.remap_wo = Wo; p.epi.remap_py = py; p.epi.remap_px = px;
  *out = p;
  return true;
}

TcGemm conv_transpose_product(const ConvGeom& g, const __nv_bfloat16* g_planes, int gt,
                              const __nv_bfloat16* w_planes, int wt, bool skip_centre,
                              const TcEpilogue& e) {
  TcGemm p;
  p.A = pixel_operand(g_planes, g.pixels(), gt, g.pixels() * 64, false);
  // w[tap][c][c']: for one tap N = c rows, K = c' contiguous
  p.B.base = w_planes; p.B.rows = g.k * g.k * 64; p.B.cols = 64; p.B.planes = wt;
  p.B.plane_stride = (int64_t)g.k * g.k * 4096; p.B.mn_major = false;
  p.M = (int)g.pixels(); p.N = 64;
  p.K = (g.k * g.k - (skip_centre ? 1 : 0)) * 64;
  p.epi = e;
  p.conv.mode = TC_CONV_PIXELS; p.conv.H = g.H; p.conv.W = g.W; p.conv.k = g.k; p.conv.pad = g.pad;
  p.conv.sgn = -1; p.conv.b_tap_rows = 1;
  p.conv.skip_tap = skip_centre ? g.pad * g.k + g.pad : -1;
  return p;
}

mw_status conv_wgrad_tensor(TcMapCache* cache, const ConvGeom& g, const __nv_bfloat16* x_planes,
                            const __nv_bfloat16* gz_planes, int terms, float* partials, float* dw,
                            DeviceStatus* st, cudaStream_t s, const float* theta, float lr) {
  const int C = g.C;
  const int slices = conv_wgrad_tensor_slices(g.out_pixels(), C, g.k * g.k);
  const int rows = g.k * g.k * C;
  TcGemm p;
  p.A = pixel_operand(x_planes, g.pixels(), terms, g.pixels() * C, true, C);
  p.B = pixel_operand(gz_planes, g.out_pixels(), terms, g.out_pixels() * C, true, C);
  p.M = rows; p.N = C; p.K = (int)(g.out_pixels() / slices);
  p.batch = slices;
  p.epi.mode = TC_EPI_PLAIN;
  p.epi.out_f32 = slices > 1 ? partials : dw;
  p.epi.bs_f32 = (int64_t)rows * C;
  if (theta && slices == 1) { p.epi.alpha = -lr; p.epi.addend = theta; }
  p.conv.mode = TC_CONV_WGRAD; p.conv.H = g.H; p.conv.W = g.W; p.conv.k = g.k; p.conv.pad = g.pad;
  p.conv.C = C; p.conv.stride = g.stride; p.conv.Ho = g.Ho(); p.conv.Wo = g.Wo();
  MW_TRY(tc_gemm_group(cache, &p, 1, st, s));
  if (slices > 1) {
    const int64_t n = (int64_t)rows * C;
    slice_sum_f32_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(partials, n, n, slices, dw, theta, lr);
    MW_TRY(launch_ok());
  }
  return MW_OK;
}

}  // namespace mw

// ---------------------------------------------------------------------------------------
// C ABI: the three convolution products, exposed for unit parity tests
// ---------------------------------------------------------------------------------------
extern "C" mw_status mw_conv2d_strided_split_bf16(int32_t op, const float* a, const float* b, float* out,
                                                  int32_t images, int32_t H, int32_t W, int32_t C,
                                                  int32_t k, int32_t stride, int32_t pad, int32_t terms,
                                                  void* scratch, size_t scratch_bytes, void* stream) {
  using namespace mw;
  if (!a || !b || !out || !scratch) return MW_ERR_INVALID_ARG;
  if (op < 0 || op > 2 || terms < 1 || terms > 3 || images < 1 || H < 1 || W < 1 || k < 1 || C < 64 ||
      C % 64 != 0 || stride < 1 || pad < 0 || pad >= k || H + 2 * pad < k || W + 2 * pad < k)
    return MW_ERR_INVALID_ARG;
  ConvGeom g{images, H, W, k, pad, C, stride};
  const int64_t pin = g.pixels() * C, pout = g.out_pixels() * C;  // elements of the two pixel arrays
  const int64_t ew = g.kernel_elems();
  const int64_t ea = op == 1 ? pout : pin;
  const int64_t eb = op == 2 ? pout : ew;
  const int slices = conv_wgrad_tensor_slices(g.out_pixels(), C, k * k);
  const size_t sa = align_up((size_t)ea, 128), sb = align_up((size_t)eb, 128);
  const size_t need = 256 + 2 * (size_t)terms * (sa + sb) + (op == 2 ? (size_t)slices * ew * 4 : 0) + 512;
  if (((uintptr_t)scratch & 255u) || scratch_bytes < need) return MW_ERR_WORKSPACE;
  if (op == 1 && stride > 1 && (stride > 2 || H != stride * g.Ho() || W != stride * g.Wo()))
    return MW_ERR_UNSUPPORTED;
  cudaStream_t s = (cudaStream_t)stream;
  DeviceStatus* st = reinterpret_cast<DeviceStatus*>(scratch);
  MW_CUDA_OK(cudaMemsetAsync(st, 0, 256, s));
  __nv_bfloat16* pa = reinterpret_cast<__nv_bfloat16*>(static_cast<char*>(scratch) + 256);
  __nv_bfloat16* pb = pa + (size_t)terms * sa;
  float* partials = reinterpret_cast<float*>(pb + (size_t)terms * sb);
  MW_TRY(split_planes(a, ea, pa, terms, (int64_t)sa, s));
  MW_TRY(split_planes(b, eb, pb, terms, (int64_t)sb, s));
  mw_status rc = MW_OK;
  TcEpilogue e;
  e.mode = TC_EPI_PLAIN;
  e.out_f32 = out;
  if (op == 2) {
    // the planes here are spaced by the padded sizes: build the product with those strides
    const int rows = k * k * C;
    TcGemm p;
    p.A = pixel_operand(pa, g.pixels(), terms, (int64_t)sa, true, C);
    p.B = pixel_operand(pb, g.out_pixels(), terms, (int64_t)sb, true, C);
    p.M = rows; p.N = C; p.K = (int)(g.out_pixels() / slices); p.batch = slices;
    p.epi.mode = TC_EPI_PLAIN;
    p.epi.out_f32 = slices > 1 ? partials : out;
    p.epi.bs_f32 = (int64_t)rows * C;
    p.conv.mode = TC_CONV_WGRAD; p.conv.H = H; p.conv.W = W; p.conv.k = k; p.conv.pad = pad;
    p.conv.C = C; p.conv.stride = stride; p.conv.Ho = g.Ho(); p.conv.Wo = g.Wo();
    rc = tc_gemm_group(nullptr, &p, 1, st, s);
    if (rc == MW_OK && slices > 1) {
      const int64_t n = (int64_t)rows * C;
      slice_sum_f32_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(partials, n, n, slices, out);
      rc = launch_ok();
    }
  } else if (op == 0) {
    TcGemm p = conv_forward_product(g, pa, terms, pb, terms, e);
    p.A.plane_stride = (int64_t)sa;
    p.B.plane_stride = (int64_t)sb;
    rc = tc_gemm_group(nullptr, &p, 1, st, s);
  } else if (stride == 1) {
    if (2 * pad + 1 != k) return MW_ERR_UNSUPPORTED;
    TcGemm p = conv_transpose_product(g, pa, terms, pb, terms, false, e);
    p.A.plane_stride = (int64_t)sa;
    p.B.plane_stride = (int64_t)sb;
    rc = tc_gemm_group(nullptr, &p, 1, st, s);
  } else {
    TcGemm cls[4];
    int n = 0;
    for (int py = 0; py < stride; ++py)
      for (int px = 0; px < stride; ++px) {
        if (!conv_transpose_class_product(g, py, px, pa, terms, pb, terms, e, &cls[n])) return MW_ERR_UNSUPPORTED;
        cls[n].A.plane_stride = (int64_t)sa;
        cls[n].B.plane_stride = (int64_t)sb;
        ++n;
      }
    rc = tc_gemm_group(nullptr, cls, n, st, s);
  }
  MW_TRY(rc);
  DeviceStatus host;
  MW_CUDA_OK(cudaMemcpyAsync(&host, st, sizeof(host), cudaMemcpyDeviceToHost, s));
  MW_CUDA_OK(cudaStreamSynchronize(s));
  return host.code == 0 ? MW_OK : (mw_status)host.code;
}

extern "C" mw_status mw_conv2d_split_bf16(int32_t op, const float* a, const float* b, float* out,
                                          int32_t images, int32_t H, int32_t W, int32_t k,
                                          int32_t terms, void* scratch, size_t scratch_bytes,
                                          void* stream) {
  if (k < 1 || !(k & 1)) return MW_ERR_INVALID_ARG;
  return mw_conv2d_strided_split_bf16(op, a, b, out, images, H, W, 64, k, 1, k / 2, terms, scratch,
                                      scratch_bytes, stream);
}
