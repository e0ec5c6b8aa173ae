// Convolution steps as products of the persistent tcgen05 kernel (internal; see mw_conv_tensor.cu).
#pragma once
#include "mw_tc_gemm.cuh"

namespace mw {

// C -> C channels (a multiple of 64), k x k kernel, H x W input, (H + 2 pad - k)/stride + 1 output
struct ConvGeom {
  int images, H, W, k, pad;
  int C = 64, stride = 1;
  int Ho() const { return (H + 2 * pad - k) / stride + 1; }
  int Wo() const { return (W + 2 * pad - k) / stride + 1; }
  int64_t pixels() const { return (int64_t)images * H * W; }
  int64_t out_pixels() const { return (int64_t)images * Ho() * Wo(); }
  int64_t kernel_elems() const { return (int64_t)k * k * C * C; }
};

// term planes of a channel-last pixel array [pixels][channels] as an operand
TcOperand pixel_operand(const void* planes, int64_t pixels, int terms, int64_t plane_stride, bool mn,
                        int channels = 64);

// x' = conv(x, w): rows = output pixels, N = c_out.  w planes: [terms][k*k][C][C]
TcGemm conv_forward_product(const ConvGeom& g, const __nv_bfloat16* x_planes, int xt,
                            const __nv_bfloat16* w_planes, int wt, const TcEpilogue& e);
// h = TransposeConv(g, w) of a stride-1 layer (optionally without the centre tap)
TcGemm conv_transpose_product(const ConvGeom& g, const __nv_bfloat16* g_planes, int gt,
                              const __nv_bfloat16* w_planes, int wt, bool skip_centre,
                              const TcEpilogue& e);
// One parity class of a strided TransposeConv (Eq. "conv-vjp": the dilated cotangent is zero
// off the stride grid, so input pixel (stride*y + py, stride*x + px) only sees the taps j with
// py + pad - j0 and px + pad - j1 multiples of the stride): rows = the pixels of the class, one
// per output pixel (H = stride*Ho and W = stride*Wo are required), scattered to their places by the
// epilogue.  The stride*stride classes together give h.  Returns false when the class has no tap.
bool conv_transpose_class_product(const ConvGeom& g, int py, int px, const __nv_bfloat16* g_planes,
                                  int gt, const __nv_bfloat16* w_planes, int wt, const TcEpilogue& e,
                                  TcGemm* out);
// dw[k*k][C][C] = sum over output pixels; `partials` holds conv_wgrad_tensor_slices(out pixels)
// copies of dw
int conv_wgrad_tensor_slices(int64_t pixels, int C = 64, int taps = 9);
// Constrained parameterisation (Section "Constrained Convolutions"): the entries of the C x C tap
// at w + offset that Lemma 1 (ii) fixes (c < c') are not parameters; after a fused update they are
// put back to zero.
mw_status conv_zero_fixed_entries(float* w, int64_t offset, int C, cudaStream_t s);
// out[i] = sum over the slices (in order) of part[z*n + i]; with `theta`: theta[i] - lr * that sum
mw_status conv_slice_sum(const float* part, int64_t n, int slices, float* out, const float* theta,
                         float lr, cudaStream_t s);
// With `theta` given the result is theta - lr * dw instead (fused parameter update).
mw_status conv_wgrad_tensor(TcMapCache* cache, const ConvGeom& g, const __nv_bfloat16* x_planes,
                            const __nv_bfloat16* gz_planes, int terms, float* partials, float* dw,
                            DeviceStatus* st, cudaStream_t s, const float* theta = nullptr,
                            float lr = 0.f);

}  // namespace mw
