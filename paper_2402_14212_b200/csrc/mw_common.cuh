// Shared declarations of the Moonwalk CUDA library (internal; the public ABI is moonwalk.h).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "moonwalk.h"

namespace mw {

// Device status block at the start of every workspace (256 bytes reserved).
//   word 0: first error code recorded by a kernel (mw_status value), 0 = none
//   words 1..4: kernel-specific detail of that first error
struct DeviceStatus {
  unsigned int code;
  unsigned int detail[4];
};

__device__ __forceinline__ void record_error(DeviceStatus* st, unsigned int code, unsigned int d0,
                                             unsigned int d1, unsigned int d2, unsigned int d3) {
  if (st == nullptr) return;
  if (atomicCAS(&st->code, 0u, code) == 0u) {
    st->detail[0] = d0;
    st->detail[1] = d1;
    st->detail[2] = d2;
    st->detail[3] = d3;
  }
}

#define MW_CUDA_OK(expr)                          \
  do {                                            \
    cudaError_t e__ = (expr);                     \
    if (e__ != cudaSuccess) return MW_ERR_CUDA;   \
  } while (0)

#define MW_TRY(expr)                 \
  do {                               \
    mw_status s__ = (expr);          \
    if (s__ != MW_OK) return s__;    \
  } while (0)

// Kernel launches enqueued by this library since load (host-side count, for the benchmark's
// "gpu_launches" figure).  launch_ok(k) is called after k launches.
extern long long g_launch_count;
inline mw_status launch_ok(int k = 1) {
  g_launch_count += k;
  return cudaGetLastError() == cudaSuccess ? MW_OK : MW_ERR_CUDA;
}

static inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
static inline int ceil_div(int64_t a, int64_t b) { return (int)((a + b - 1) / b); }

// ---- scalar type helpers ---------------------------------------------------------------
template <typename T>
__device__ __forceinline__ float to_f32(T v) { return (float)v; }
template <>
__device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

template <typename T>
__device__ __forceinline__ T from_f64(double v) { return (T)v; }
template <>
__device__ __forceinline__ __nv_bfloat16 from_f64<__nv_bfloat16>(double v) { return __float2bfloat16_rn((float)v); }

// strict positivity: 0, -0.0 and NaN are "not positive"
template <typename T>
__device__ __forceinline__ bool is_pos(T v) { return v > (T)0; }
template <>
__device__ __forceinline__ bool is_pos<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v) > 0.f; }

// ---- elementwise / residual-store kernels (mw_elementwise.cu) ----------------------------
// x_out = phi(z) and sign words; T = double/float (z), TX = storage of x_out.
template <typename T, typename TX>
mw_status act_forward_pack(const T* z, int64_t rows, int cols, int act, double slope, TX* x_out,
                           uint32_t* words, bool write_words, cudaStream_t s);
template <typename T>
mw_status pack_sign_bits(const T* z, int64_t rows, int cols, uint32_t* words, cudaStream_t s);
// g_z = h * phi'(mask)
template <typename T>
mw_status scale_by_mask(const T* h, const uint32_t* words, int64_t rows, int cols, int act,
                        double slope, T* gz, cudaStream_t s);
// activation vijp; for ReLU restores dead units from fragments and zeroes g_z there
template <typename T>
mw_status activation_vijp(const T* gz, const uint32_t* words, int64_t rows, int cols, int act,
                          double slope, const uint32_t* off, const T* vals, T* h_out, T* gz_out,
                          cudaStream_t s);
// ReLU fragments: cnt/off (exclusive scan over rows) and ordered compaction
mw_status fragment_offsets(const uint32_t* words, int64_t rows, int cols, uint32_t* cnt,
                           uint32_t* off, uint32_t* total, void* scratch, size_t scratch_bytes,
                           cudaStream_t s);
// the same index built by one CTA, plus rank[r][c/64] = dead units of row r before column
// 64*(c/64) (cols % 64 == 0; meant for a few thousand rows)
mw_status fragment_index(const uint32_t* words, int rows, int cols, uint32_t* cnt, uint32_t* off,
                         uint32_t* rank, uint32_t* total, cudaStream_t s);
template <typename T>
mw_status fragment_compact(const T* h, const uint32_t* words, int64_t rows, int cols,
                           const uint32_t* off, T* vals, cudaStream_t s);
// loss and its cotangent; partial sums land in `partials` (>= 1024 doubles), J in loss_out
template <typename T>
mw_status loss_cotangent(const T* y, const void* target, int64_t rows, int cols, int loss, T* h,
                         double* partials, double* loss_out, cudaStream_t s);
template <typename TI, typename TO>
mw_status convert_array(const TI* in, TO* out, int64_t n, cudaStream_t s);

// ---- CUDA-core GEMM and small inverse (mw_gemm_simt.cu) ----------------------------------
// C[M][N] = alpha * op(A) op(B) + beta * C ; op(A) is [M][K]: A row-major [M][lda] (ta = 0) or
// A row-major [K][lda] read transposed (ta = 1); op(B) is [K][N]: B row-major [K][ldb] (tb = 0)
// or B row-major [N][ldb] read transposed (tb = 1).
template <typename T>
mw_status gemm_simt(int ta, int tb, int M, int N, int K, double alpha, const T* A, int lda,
                    const T* B, int ldb, double beta, T* C, int ldc, cudaStream_t s);
// Gauss-Jordan inverse with partial pivoting of one n x n matrix, n <= 64, one CTA, fp64 inside.
template <typename T>
mw_status inverse_small(const T* W, int n, T* Winv, DeviceStatus* st, int layer, cudaStream_t s);
// the same for up to kSmallBatch matrices at once (one CTA each): matrix b = Ws.p[b] + offset
constexpr int kSmallBatch = 32;
struct SmallBatch { const void* p[kSmallBatch]; };
template <typename T>
mw_status inverse_small_batch(const SmallBatch& Ws, int count, int64_t offset, int n, T* Winv,
                              DeviceStatus* st, int layer0, cudaStream_t s);
// X <- X (2I - W X) style Newton-Schulz on CUDA cores (any n); scratch >= 2 n^2 elements.
template <typename T>
mw_status inverse_newton_simt(const T* W, int n, int iters, T* X, T* scratch, DeviceStatus* st,
                              int layer, double tol, cudaStream_t s);

}  // namespace mw
