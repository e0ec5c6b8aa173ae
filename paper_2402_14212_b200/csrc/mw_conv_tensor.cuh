// Convolution steps as products of the persistent tcgen05 kernel (internal; see mw_conv_tensor.cu).
#pragma once
#include "mw_tc_gemm.cuh"

namespace mw {

struct ConvGeom {
  int images, H, W, k, pad;
  int64_t pixels() const { return (int64_t)images * H * W; }
};

// term planes of a channel-last pixel array [pixels][64] as an operand
TcOperand pixel_operand(const void* planes, int64_t pixels, int terms, int64_t plane_stride, bool mn);

// x' = conv(x, w): rows = pixels, N = c_out.  w planes: [terms][k*k][64][64]
TcGemm conv_forward_product(const ConvGeom& g, const __nv_bfloat16* x_planes, int xt,
                            const __nv_bfloat16* w_planes, int wt, const TcEpilogue& e);
// h = TransposeConv(g, w) (optionally without the centre tap)
TcGemm conv_transpose_product(const ConvGeom& g, const __nv_bfloat16* g_planes, int gt,
                              const __nv_bfloat16* w_planes, int wt, bool skip_centre,
                              const TcEpilogue& e);
// dw[k*k][64][64] = sum over pixels; `partials` holds conv_wgrad_tensor_slices(pixels) copies of dw
int conv_wgrad_tensor_slices(int64_t pixels);
mw_status conv_wgrad_tensor(TcMapCache* cache, const ConvGeom& g, const __nv_bfloat16* x_planes,
                            const __nv_bfloat16* gz_planes, int terms, float* partials, float* dw,
                            DeviceStatus* st, cudaStream_t s);

}  // namespace mw
