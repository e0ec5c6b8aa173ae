// Tensor-core product core for sm_100a: TMA-staged operand tiles, tcgen05.mma with the
// accumulator in tensor memory, fused epilogues.  Internal interface.
//
// Every dense step of the Moonwalk path is one call of tc_gemm():
//   Phase I / recompute   z   = x W^T         (A = x K-major,  B = W K-major)
//   Phase II              h'  = g_z W         (A = g_z K-major, B = W MN-major)
//   dense vijp            g_z = h W^-1        (A = h K-major,  B = W^-1 MN-major)       Eq. "h_i"
//   weight vjp            dW  = g_z^T x       (A = g_z MN-major, B = x MN-major)        Eq. "g_i"
//   Newton-Schulz         R = I - W X, X' = X + X R
//
// An operand is a stack of 1..3 bf16 "term planes" whose sum is the value (term t holds the
// bf16 rounding of what the earlier terms left over).  A product of an a-term and a b-term
// operand accumulates, in fp32, the cross products (i, j) with i + j < max(a, b): 1 product for
// plain bf16, 3 for ~16-bit operands, 6 for fp32-accurate operands.
#pragma once
#include <cuda.h>

#include "mw_common.cuh"

namespace mw {

struct TcOperand {
  const void* base = nullptr;   // bf16 planes, each [rows][cols] row-major
  int rows = 0, cols = 0;       // K-major: rows = M or N, cols = K.  MN-major: rows = K, cols = M or N
  int planes = 1;
  int64_t plane_stride = 0;     // elements between planes
  bool mn_major = false;
  int batch_planes = 0;         // batched launch: planes between consecutive batch items (0 = planes)
};

enum TcEpiMode : int {
  TC_EPI_PLAIN = 0,    // v = alpha*acc (+ addend);  out_f32 and/or planes
  TC_EPI_RESID = 1,    // v = (row == col) - acc;    planes; sum of squares -> sumsq
  TC_EPI_FWD = 2,      // z = acc; sign word written (write_mask) or read; x = phi(z) -> planes (+ out_f32)
  TC_EPI_BWD = 3,      // h = acc -> out_f32 (optional); g = h * phi'(mask) -> planes
  TC_EPI_VIJP = 4,     // g = acc; leaky: h = g or g/slope -> planes2 ; g -> planes (for the weight vjp)
};

struct TcEpilogue {
  int mode = TC_EPI_PLAIN;
  float alpha = 1.f;
  const float* addend = nullptr;       // [M][N] fp32
  float* out_f32 = nullptr;            // [M][N] fp32
  __nv_bfloat16* planes = nullptr;     // primary split output, n_planes x [M][N]
  int n_planes = 0;
  int64_t plane_stride = 0;
  __nv_bfloat16* planes2 = nullptr;    // secondary split output (TC_EPI_VIJP: h)
  int n_planes2 = 0;
  int64_t plane_stride2 = 0;
  uint32_t* mask = nullptr;            // sign words [M][N/32]
  int write_mask = 0;
  int act = MW_ACT_NONE;
  float slope = 1.f;
  double* sumsq = nullptr;             // TC_EPI_RESID: atomically accumulated ||v||_F^2
  // batched launch (grid.z): element strides between consecutive batch items
  int64_t bs_f32 = 0;                  // addend and out_f32
  int64_t bs_planes = 0, bs_planes2 = 0;
  int64_t bs_mask = 0;                 // words
  int64_t bs_sumsq = 0;                // doubles
};

// Cache of encoded tensor maps (host side), owned by the caller of tc_gemm.
struct TcMapCache;
TcMapCache* tc_cache_create();
void tc_cache_destroy(TcMapCache*);

// D[M][N] = sum over term pairs of A_i B_j^T-style products; see TcOperand for layouts.
// Requirements: N % 64 == 0; K % 64 == 0 for K-major operands; inner dimensions % 64 == 0;
// all bases 16-byte aligned (256 recommended).
// batch > 1 runs `batch` independent products of the same shape in one launch (grid.z): batch
// item b reads planes b*batch_planes + t of each operand and offsets the epilogue pointers by
// b times the bs_* strides.
mw_status tc_gemm(TcMapCache* cache, const TcOperand& A, const TcOperand& B, int M, int N, int K,
                  const TcEpilogue& epi, DeviceStatus* st, cudaStream_t s, int batch = 1);

// Per-launch timing of the product kernel (CUDA events around every launch while enabled).
void tc_profile_begin();
mw_status tc_profile_end(double* total_ms, long long* launches, double* flops, double* mma_flops);

// fp32 [n] -> `planes` bf16 term planes (plane p at out + p*plane_stride)
mw_status split_planes(const float* in, int64_t n, __nv_bfloat16* out, int planes,
                       int64_t plane_stride, cudaStream_t s);
// batched: item b reads in + b*in_stride and writes out + b*out_stride
mw_status split_planes_batched(const float* in, int64_t n, int batch, int64_t in_stride,
                               __nv_bfloat16* out, int planes, int64_t plane_stride,
                               int64_t out_stride, cudaStream_t s);

}  // namespace mw
