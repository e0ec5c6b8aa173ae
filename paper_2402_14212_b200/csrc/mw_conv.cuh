// Convolution steps on CUDA cores (internal declarations; see mw_conv.cu).
#pragma once
#include "mw_common.cuh"

namespace mw {

// out = mode ? base - acc : acc;  acc[m][n] = sum_{tap,ci} in[pixel m shifted by sgn*(tap-p)][ci] *
// (wtrans ? w[tap][n][ci] : w[tap][ci][n]).  sgn = +1: forward convolution; sgn = -1 with
// wtrans = 1: TransposeConv.
template <typename T>
mw_status conv_igemm(const T* in, const T* w, T* out, const T* base, int Bn, int H, int W, int Ci,
                     int Co, int k, int pad, int sgn, int wtrans, int mode, cudaStream_t s);

// dw[tap][c][c'] = sum over pixels; scratch holds conv_wgrad_slices(pixels) partial copies of dw.
int conv_wgrad_slices(int64_t pixels);
template <typename T>
mw_status conv_wgrad(const T* x, const T* gz, T* dw, T* scratch, int Bn, int H, int W, int Ci,
                     int Co, int k, int pad, cudaStream_t s);

template <typename T>
mw_status zero_array(T* p, int64_t n, cudaStream_t s);

}  // namespace mw
