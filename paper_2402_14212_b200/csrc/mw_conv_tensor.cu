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
                     float* __restrict__ out) {
  const int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x;
  if (i >= n) return;
  float a = 0.f;
  for (int z = 0; z < slices; ++z) a += part[(int64_t)z * stride + i];   // fixed order
  out[i] = a;
}

}  // namespace

int conv_wgrad_tensor_slices(int64_t pixels) {
  const int64_t blocks = pixels / 64;
  for (int s = 32; s > 1; s >>= 1)
    if (blocks % s == 0 && blocks / s >= 4) return s;
  return 1;
}

TcOperand pixel_operand(const void* planes, int64_t pixels, int terms, int64_t plane_stride, bool mn) {
  TcOperand o;
  o.base = planes;
  o.rows = (int)pixels;
  o.cols = 64;
  o.planes = terms;
  o.plane_stride = plane_stride;
  o.mn_major = mn;
  return o;
}

TcGemm conv_forward_product(const ConvGeom& g, const __nv_bfloat16* x_planes, int xt,
                            const __nv_bfloat16* w_planes, int wt, const TcEpilogue& e) {
  TcGemm p;
  p.A = pixel_operand(x_planes, g.pixels(), xt, g.pixels() * 64, false);
  // w[tap][ci][co]: K = (tap, ci) rows, N = co contiguous
  p.B.base = w_planes; p.B.rows = g.k * g.k * 64; p.B.cols = 64; p.B.planes = wt;
  p.B.plane_stride = (int64_t)g.k * g.k * 4096; p.B.mn_major = true;
  p.M = (int)g.pixels(); p.N = 64; p.K = g.k * g.k * 64;
  p.epi = e;
  p.conv.mode = TC_CONV_PIXELS; p.conv.H = g.H; p.conv.W = g.W; p.conv.k = g.k; p.conv.pad = g.pad;
  p.conv.sgn = 1;
  return p;
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
                            DeviceStatus* st, cudaStream_t s) {
  const int slices = conv_wgrad_tensor_slices(g.pixels());
  const int rows = g.k * g.k * 64;
  TcGemm p;
  p.A = pixel_operand(x_planes, g.pixels(), terms, g.pixels() * 64, true);
  p.B = pixel_operand(gz_planes, g.pixels(), terms, g.pixels() * 64, true);
  p.M = rows; p.N = 64; p.K = (int)(g.pixels() / slices);
  p.batch = slices;
  p.epi.mode = TC_EPI_PLAIN;
  p.epi.out_f32 = slices > 1 ? partials : dw;
  p.epi.bs_f32 = (int64_t)rows * 64;
  p.conv.mode = TC_CONV_WGRAD; p.conv.H = g.H; p.conv.W = g.W; p.conv.k = g.k; p.conv.pad = g.pad;
  MW_TRY(tc_gemm_group(cache, &p, 1, st, s));
  if (slices > 1) {
    const int64_t n = (int64_t)rows * 64;
    slice_sum_f32_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(partials, n, n, slices, dw);
    MW_TRY(launch_ok());
  }
  return MW_OK;
}

}  // namespace mw

// ---------------------------------------------------------------------------------------
// C ABI: the three convolution products, exposed for unit parity tests
// ---------------------------------------------------------------------------------------
extern "C" mw_status mw_conv2d_split_bf16(int32_t op, const float* a, const float* b, float* out,
                                          int32_t images, int32_t H, int32_t W, int32_t k,
                                          int32_t terms, void* scratch, size_t scratch_bytes,
                                          void* stream) {
  using namespace mw;
  if (!a || !b || !out || !scratch) return MW_ERR_INVALID_ARG;
  if (op < 0 || op > 2 || terms < 1 || terms > 3 || images < 1 || H < 1 || W < 1 || k < 1 || !(k & 1))
    return MW_ERR_INVALID_ARG;
  ConvGeom g{images, H, W, k, k / 2};
  const int64_t px = g.pixels();
  const int64_t ea = px * 64;                                   // pixel array
  const int64_t ew = (int64_t)k * k * 4096;                     // kernel
  const int64_t eb = op == 2 ? ea : ew;
  const int slices = conv_wgrad_tensor_slices(px);
  const size_t need = 256 + 2 * (size_t)terms * (align_up((size_t)ea, 128) + align_up((size_t)eb, 128)) +
                      (op == 2 ? (size_t)slices * ew * 4 : 0) + 512;
  if (((uintptr_t)scratch & 255u) || scratch_bytes < need) return MW_ERR_WORKSPACE;
  cudaStream_t s = (cudaStream_t)stream;
  DeviceStatus* st = reinterpret_cast<DeviceStatus*>(scratch);
  MW_CUDA_OK(cudaMemsetAsync(st, 0, 256, s));
  __nv_bfloat16* pa = reinterpret_cast<__nv_bfloat16*>(static_cast<char*>(scratch) + 256);
  __nv_bfloat16* pb = pa + (size_t)terms * align_up((size_t)ea, 128);
  float* partials = reinterpret_cast<float*>(pb + (size_t)terms * align_up((size_t)eb, 128));
  MW_TRY(split_planes(a, ea, pa, terms, (int64_t)align_up((size_t)ea, 128), s));
  MW_TRY(split_planes(b, eb, pb, terms, (int64_t)align_up((size_t)eb, 128), s));
  mw_status rc;
  if (op == 2) {
    // planes are spaced by the padded size: rebuild the operands with that stride
    TcGemm p;
    p.A = pixel_operand(pa, px, terms, (int64_t)align_up((size_t)ea, 128), true);
    p.B = pixel_operand(pb, px, terms, (int64_t)align_up((size_t)eb, 128), true);
    const int rows = k * k * 64;
    p.M = rows; p.N = 64; p.K = (int)(px / slices); p.batch = slices;
    p.epi.mode = TC_EPI_PLAIN;
    p.epi.out_f32 = slices > 1 ? partials : out;
    p.epi.bs_f32 = (int64_t)rows * 64;
    p.conv.mode = TC_CONV_WGRAD; p.conv.H = H; p.conv.W = W; p.conv.k = k; p.conv.pad = k / 2;
    rc = tc_gemm_group(nullptr, &p, 1, st, s);
    if (rc == MW_OK && slices > 1) {
      const int64_t n = (int64_t)rows * 64;
      slice_sum_f32_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(partials, n, n, slices, out);
      rc = launch_ok();
    }
  } else {
    TcEpilogue e;
    e.mode = TC_EPI_PLAIN;
    e.out_f32 = out;
    TcGemm p = op == 0 ? conv_forward_product(g, pa, terms, pb, terms, e)
                       : conv_transpose_product(g, pa, terms, pb, terms, false, e);
    p.A.plane_stride = (int64_t)align_up((size_t)ea, 128);
    p.B.plane_stride = (int64_t)align_up((size_t)eb, 128);
    rc = tc_gemm_group(nullptr, &p, 1, st, s);
  }
  MW_TRY(rc);
  DeviceStatus host;
  MW_CUDA_OK(cudaMemcpyAsync(&host, st, sizeof(host), cudaMemcpyDeviceToHost, s));
  MW_CUDA_OK(cudaStreamSynchronize(s));
  return host.code == 0 ? MW_OK : (mw_status)host.code;
}
