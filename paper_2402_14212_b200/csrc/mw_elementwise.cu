// Elementwise and residual-store kernels of the Moonwalk library (stand-alone forms).
//
//  * sign-bit pack (Section "Residual Impact": Phase I keeps one bit per activation),
//  * activation forward / vjp scaling / vijp (Eq. "h_i" restricted to the activation),
//  * ReLU fragment store: count, exclusive scan, ordered compaction and restore
//    (Section 5.1 applied to ReLU: keep exactly the cotangent elements that the vijp cannot
//    reconstruct, i.e. those at dead units),
//  * losses and their cotangents.
//
// All are HBM-bound: every tensor is touched once, with 128-bit accesses on the float paths
// when the row length allows (cols % 128 == 0), one warp per 128-column segment.
#include <type_traits>

#include "mw_common.cuh"

namespace mw {

static constexpr int kThreads = 256;

__device__ __forceinline__ unsigned lanemask_lt() {
  unsigned m;
  asm("mov.u32 %0, %%lanemask_lt;" : "=r"(m));
  return m;
}

// derivative / forward factor of the negative branch
__host__ __device__ __forceinline__ double neg_factor(int act, double slope) {
  return act == MW_ACT_LEAKY_RELU ? slope : (act == MW_ACT_RELU ? 0.0 : 1.0);
}

// ---------------------------------------------------------------------------------------
// generic (any type, any cols): one warp per (row, 32-column word), ballot builds the word
// ---------------------------------------------------------------------------------------
template <typename T, typename TX, bool WRITE_X, bool WRITE_WORDS, bool READ_WORDS>
__global__ void __launch_bounds__(kThreads)
act_forward_kernel(const T* __restrict__ z, int64_t rows, int cols, int wpr, int act, double slope,
                   TX* __restrict__ x_out, uint32_t* __restrict__ words) {
  const int lane = threadIdx.x & 31;
  const int64_t warp0 = ((int64_t)blockIdx.x * kThreads + threadIdx.x) >> 5;
  const int64_t nwarps = ((int64_t)gridDim.x * kThreads) >> 5;
  const int64_t total = rows * wpr;
  const double nf = neg_factor(act, slope);
  for (int64_t t = warp0; t < total; t += nwarps) {
    const int64_t r = t / wpr;
    const int w = (int)(t - r * wpr);
    const int c = w * 32 + lane;
    const bool in = c < cols;
    T v = z[in ? r * cols + c : 0];
    bool pos;
    if (READ_WORDS) {
      pos = (words[t] >> lane) & 1u;
    } else {
      pos = in && is_pos(v);
      if (act == MW_ACT_NONE) pos = in;
    }
    if (WRITE_WORDS) {
      unsigned b = __ballot_sync(0xffffffffu, pos);
      if (lane == 0) words[t] = b;
    }
    if constexpr (WRITE_X) {
      if (in) {
        T o = pos ? v : (T)((T)nf * v);
        x_out[r * cols + c] = from_f64<TX>((double)o);
      }
    }
  }
}

// float, cols % 128 == 0: one warp per 128 columns, float4 per lane, nibble merge by shuffles
template <typename TX, bool WRITE_X, bool WRITE_WORDS, bool READ_WORDS>
__global__ void __launch_bounds__(kThreads)
act_forward_vec4_kernel(const float* __restrict__ z, int64_t nseg, int act, float nf,
                        TX* __restrict__ x_out, uint32_t* __restrict__ words) {
  const int lane = threadIdx.x & 31;
  const int64_t warp0 = ((int64_t)blockIdx.x * kThreads + threadIdx.x) >> 5;
  const int64_t nwarps = ((int64_t)gridDim.x * kThreads) >> 5;
  for (int64_t sgm = warp0; sgm < nseg; sgm += nwarps) {
    const int64_t e0 = sgm * 128 + lane * 4;
    float4 v = *reinterpret_cast<const float4*>(z + e0);
    unsigned nib;
    if (READ_WORDS) {
      unsigned wv = words[sgm * 4 + (lane >> 3)];
      nib = (wv >> (4 * (lane & 7))) & 0xFu;
    } else {
      nib = (v.x > 0.f ? 1u : 0u) | (v.y > 0.f ? 2u : 0u) | (v.z > 0.f ? 4u : 0u) |
            (v.w > 0.f ? 8u : 0u);
      if (act == MW_ACT_NONE) nib = 0xFu;
    }
    if (WRITE_WORDS) {
      unsigned part = nib << (4 * (lane & 7));
      part |= __shfl_xor_sync(0xffffffffu, part, 1);
      part |= __shfl_xor_sync(0xffffffffu, part, 2);
      part |= __shfl_xor_sync(0xffffffffu, part, 4);
      if ((lane & 7) == 0) words[sgm * 4 + (lane >> 3)] = part;
    }
    if (WRITE_X) {
      float o0 = (nib & 1u) ? v.x : nf * v.x;
      float o1 = (nib & 2u) ? v.y : nf * v.y;
      float o2 = (nib & 4u) ? v.z : nf * v.z;
      float o3 = (nib & 8u) ? v.w : nf * v.w;
      if (sizeof(TX) == 4) {
        *reinterpret_cast<float4*>(reinterpret_cast<float*>(x_out) + e0) = make_float4(o0, o1, o2, o3);
      } else {
        __nv_bfloat162 lo = __floats2bfloat162_rn(o0, o1);
        __nv_bfloat162 hi = __floats2bfloat162_rn(o2, o3);
        uint2 pk;
        pk.x = *reinterpret_cast<unsigned*>(&lo);
        pk.y = *reinterpret_cast<unsigned*>(&hi);
        *reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(x_out) + e0) = pk;
      }
    }
  }
}

static int grid_for(int64_t warps_needed) {
  int64_t blocks = (warps_needed * 32 + kThreads - 1) / kThreads;
  const int64_t cap = 148 * 16;
  if (blocks > cap) blocks = cap;
  if (blocks < 1) blocks = 1;
  return (int)blocks;
}

template <typename T>
static bool vec_ok(const void* p, const void* q, int cols) {
  return sizeof(T) == 4 && cols % 128 == 0 && ((uintptr_t)p % 16 == 0) && ((uintptr_t)q % 16 == 0);
}

template <typename T, typename TX>
mw_status act_forward_pack(const T* z, int64_t rows, int cols, int act, double slope, TX* x_out,
                           uint32_t* words, bool write_words, cudaStream_t s) {
  if (rows == 0 || cols == 0) return MW_OK;
  const int wpr = (cols + 31) / 32;
  if (vec_ok<T>(z, x_out, cols) && (sizeof(TX) == 4 || sizeof(TX) == 2)) {
    const int64_t nseg = rows * (cols / 128);
    const float nf = (float)neg_factor(act, slope);
    if (write_words)
      act_forward_vec4_kernel<TX, true, true, false><<<grid_for(nseg), kThreads, 0, s>>>(
          (const float*)z, nseg, act, nf, x_out, words);
    else
      act_forward_vec4_kernel<TX, true, false, true><<<grid_for(nseg), kThreads, 0, s>>>(
          (const float*)z, nseg, act, nf, x_out, words);
  } else {
    const int64_t total = rows * wpr;
    if (write_words)
      act_forward_kernel<T, TX, true, true, false><<<grid_for(total), kThreads, 0, s>>>(
          z, rows, cols, wpr, act, slope, x_out, words);
    else
      act_forward_kernel<T, TX, true, false, true><<<grid_for(total), kThreads, 0, s>>>(
          z, rows, cols, wpr, act, slope, x_out, words);
  }
  return launch_ok();
}

template <typename T>
mw_status pack_sign_bits(const T* z, int64_t rows, int cols, uint32_t* words, cudaStream_t s) {
  if (rows == 0 || cols == 0) return MW_OK;
  const int wpr = (cols + 31) / 32;
  if (vec_ok<T>(z, z, cols)) {
    const int64_t nseg = rows * (cols / 128);
    act_forward_vec4_kernel<float, false, true, false><<<grid_for(nseg), kThreads, 0, s>>>(
        (const float*)z, nseg, MW_ACT_RELU, 0.f, (float*)nullptr, words);
  } else {
    act_forward_kernel<T, T, false, true, false><<<grid_for(rows * wpr), kThreads, 0, s>>>(
        z, rows, cols, wpr, MW_ACT_RELU, 0.0, (T*)nullptr, words);
  }
  return launch_ok();
}

// ---------------------------------------------------------------------------------------
// g_z = h * phi'(mask)  and leaky vijp  h = g_z / phi'(mask)   (same kernel, factor differs)
// ---------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(kThreads)
mask_scale_kernel(const T* __restrict__ in, const uint32_t* __restrict__ words, int64_t rows,
                  int cols, int wpr, T neg, T* __restrict__ out) {
  const int lane = threadIdx.x & 31;
  const int64_t warp0 = ((int64_t)blockIdx.x * kThreads + threadIdx.x) >> 5;
  const int64_t nwarps = ((int64_t)gridDim.x * kThreads) >> 5;
  const int64_t total = rows * wpr;
  for (int64_t t = warp0; t < total; t += nwarps) {
    const int64_t r = t / wpr;
    const int c = (int)(t - r * wpr) * 32 + lane;
    if (c < cols) {
      const bool pos = (words[t] >> lane) & 1u;
      T v = in[r * cols + c];
      out[r * cols + c] = pos ? v : v * neg;
    }
  }
}

__global__ void __launch_bounds__(kThreads)
mask_scale_vec4_kernel(const float* __restrict__ in, const uint32_t* __restrict__ words,
                       int64_t nseg, float neg, bool divide, float* __restrict__ out) {
  const int lane = threadIdx.x & 31;
  const int64_t warp0 = ((int64_t)blockIdx.x * kThreads + threadIdx.x) >> 5;
  const int64_t nwarps = ((int64_t)gridDim.x * kThreads) >> 5;
  for (int64_t sgm = warp0; sgm < nseg; sgm += nwarps) {
    const int64_t e0 = sgm * 128 + lane * 4;
    float4 v = *reinterpret_cast<const float4*>(in + e0);
    const unsigned nib = (words[sgm * 4 + (lane >> 3)] >> (4 * (lane & 7))) & 0xFu;
    if (divide) {
      if (!(nib & 1u)) v.x = v.x / neg;
      if (!(nib & 2u)) v.y = v.y / neg;
      if (!(nib & 4u)) v.z = v.z / neg;
      if (!(nib & 8u)) v.w = v.w / neg;
    } else {
      if (!(nib & 1u)) v.x *= neg;
      if (!(nib & 2u)) v.y *= neg;
      if (!(nib & 4u)) v.z *= neg;
      if (!(nib & 8u)) v.w *= neg;
    }
    *reinterpret_cast<float4*>(out + e0) = v;
  }
}

template <typename T>
__global__ void __launch_bounds__(kThreads)
mask_divide_kernel(const T* __restrict__ in, const uint32_t* __restrict__ words, int64_t rows,
                   int cols, int wpr, T neg, T* __restrict__ out) {
  const int lane = threadIdx.x & 31;
  const int64_t warp0 = ((int64_t)blockIdx.x * kThreads + threadIdx.x) >> 5;
  const int64_t nwarps = ((int64_t)gridDim.x * kThreads) >> 5;
  const int64_t total = rows * wpr;
  for (int64_t t = warp0; t < total; t += nwarps) {
    const int64_t r = t / wpr;
    const int c = (int)(t - r * wpr) * 32 + lane;
    if (c < cols) {
      const bool pos = (words[t] >> lane) & 1u;
      T v = in[r * cols + c];
      out[r * cols + c] = pos ? v : v / neg;
    }
  }
}

template <typename T>
mw_status scale_by_mask(const T* h, const uint32_t* words, int64_t rows, int cols, int act,
                        double slope, T* gz, cudaStream_t s) {
  if (rows == 0 || cols == 0) return MW_OK;
  const int wpr = (cols + 31) / 32;
  const double nf = neg_factor(act, slope);
  if (vec_ok<T>(h, gz, cols)) {
    const int64_t nseg = rows * (cols / 128);
    mask_scale_vec4_kernel<<<grid_for(nseg), kThreads, 0, s>>>((const float*)h, words, nseg,
                                                                (float)nf, false, (float*)gz);
  } else {
    mask_scale_kernel<T><<<grid_for(rows * wpr), kThreads, 0, s>>>(h, words, rows, cols, wpr,
                                                                    (T)nf, gz);
  }
  return launch_ok();
}

// ---------------------------------------------------------------------------------------
// ReLU fragments
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads)
dead_count_kernel(const uint32_t* __restrict__ words, int64_t rows, int cols, int wpr,
                  uint32_t* __restrict__ cnt) {
  const int lane = threadIdx.x & 31;
  const int64_t warp0 = ((int64_t)blockIdx.x * kThreads + threadIdx.x) >> 5;
  const int64_t nwarps = ((int64_t)gridDim.x * kThreads) >> 5;
  for (int64_t r = warp0; r < rows; r += nwarps) {
    unsigned live = 0;
    for (int w = lane; w < wpr; w += 32) live += __popc(words[r * wpr + w]);
    for (int o = 16; o; o >>= 1) live += __shfl_xor_sync(0xffffffffu, live, o);
    if (lane == 0) cnt[r] = (unsigned)cols - live;
  }
}

// single CTA, chunked exclusive scan with a running carry (deterministic, integer exact)
__device__ __forceinline__ void block_exclusive_scan(const uint32_t* cnt, int64_t rows,
                                                     uint32_t* off, uint32_t* total) {
  __shared__ uint32_t warp_sums[32];
  __shared__ uint32_t carry_s;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  if (tid == 0) carry_s = 0;
  __syncthreads();
  for (int64_t base = 0; base < rows; base += 1024) {
    const int64_t i = base + tid;
    uint32_t v = i < rows ? cnt[i] : 0u;
    uint32_t incl = v;
    for (int o = 1; o < 32; o <<= 1) {
      uint32_t n = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += n;
    }
    if (lane == 31) warp_sums[wid] = incl;
    __syncthreads();
    if (wid == 0) {
      uint32_t ws = warp_sums[lane];
      uint32_t wi = ws;
      for (int o = 1; o < 32; o <<= 1) {
        uint32_t n = __shfl_up_sync(0xffffffffu, wi, o);
        if (lane >= o) wi += n;
      }
      warp_sums[lane] = wi - ws;  // exclusive prefix of warp sums
    }
    __syncthreads();
    const uint32_t carry = carry_s;
    if (i < rows) off[i] = carry + warp_sums[wid] + incl - v;
    __syncthreads();
    if (tid == 1023) carry_s = carry + warp_sums[31] + incl;
    __syncthreads();
  }
  if (tid == 0 && total) *total = carry_s;
}

__global__ void __launch_bounds__(1024)
exclusive_scan_kernel(const uint32_t* __restrict__ cnt, int64_t rows, uint32_t* __restrict__ off,
                      uint32_t* __restrict__ total) {
  block_exclusive_scan(cnt, rows, off, total);
}

// One CTA builds the whole index of a ReLU layer's fragment stream from its sign words:
// cnt[r] dead units of row r, rank[r][t] dead units of row r before column 64 t, off = exclusive
// scan of cnt over rows.  cols % 64 == 0.
__global__ void __launch_bounds__(1024)
fragment_index_kernel(const uint32_t* __restrict__ words, int rows, int cols, uint32_t* cnt,
                      uint32_t* __restrict__ off, uint32_t* __restrict__ rank,
                      uint32_t* __restrict__ total) {
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  const int wpr = cols >> 5, tiles = cols >> 6;
  for (int r = wid; r < rows; r += 32) {
    uint32_t carry = 0;
    for (int t0 = 0; t0 < tiles; t0 += 32) {
      const int t = t0 + lane;
      uint32_t d = 0;
      if (t < tiles) {
        const uint2 w = *reinterpret_cast<const uint2*>(words + (int64_t)r * wpr + 2 * t);
        d = 64u - __popc(w.x) - __popc(w.y);
      }
      uint32_t incl = d;
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t n = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += n;
      }
      if (t < tiles) rank[(int64_t)r * tiles + t] = carry + incl - d;
      carry += __shfl_sync(0xffffffffu, incl, 31);
    }
    if (lane == 0) cnt[r] = carry;
  }
  __syncthreads();
  block_exclusive_scan(cnt, rows, off, total);
}

mw_status fragment_offsets(const uint32_t* words, int64_t rows, int cols, uint32_t* cnt,
                           uint32_t* off, uint32_t* total, void* scratch, size_t scratch_bytes,
                           cudaStream_t s) {
  (void)scratch;
  (void)scratch_bytes;
  if (rows == 0) return MW_OK;
  const int wpr = (cols + 31) / 32;
  dead_count_kernel<<<grid_for(rows), kThreads, 0, s>>>(words, rows, cols, wpr, cnt);
  exclusive_scan_kernel<<<1, 1024, 0, s>>>(cnt, rows, off, total);
  return launch_ok(2);
}

mw_status fragment_index(const uint32_t* words, int rows, int cols, uint32_t* cnt, uint32_t* off,
                         uint32_t* rank, uint32_t* total, cudaStream_t s) {
  if (rows == 0) return MW_OK;
  if (cols % 64 != 0) return MW_ERR_UNSUPPORTED;
  fragment_index_kernel<<<1, 1024, 0, s>>>(words, rows, cols, cnt, off, rank, total);
  return launch_ok();
}

// one warp per row; MODE 0: compact h at dead units into vals; MODE 1: restore (activation vijp
// of ReLU): h_out = live ? gz : vals[...], gz_out = live ? gz : 0
template <typename T, int MODE>
__global__ void __launch_bounds__(kThreads)
fragment_row_kernel(const T* __restrict__ src, const uint32_t* __restrict__ words, int64_t rows,
                    int cols, int wpr, const uint32_t* __restrict__ off, T* __restrict__ vals,
                    T* __restrict__ h_out, T* __restrict__ gz_out) {
  const int lane = threadIdx.x & 31;
  const int64_t warp0 = ((int64_t)blockIdx.x * kThreads + threadIdx.x) >> 5;
  const int64_t nwarps = ((int64_t)gridDim.x * kThreads) >> 5;
  for (int64_t r = warp0; r < rows; r += nwarps) {
    uint32_t base = off[r];
    for (int w = 0; w < wpr; ++w) {
      const int c = w * 32 + lane;
      const unsigned word = words[r * wpr + w];
      const unsigned valid = (w * 32 + 32 <= cols) ? 0xffffffffu : ((1u << (cols - w * 32)) - 1u);
      const unsigned dead = ~word & valid;
      const bool mine = (dead >> lane) & 1u;
      const uint32_t pos = base + __popc(dead & lanemask_lt());
      if (MODE == 0) {
        if (mine) vals[pos] = src[r * cols + c];
      } else if (c < cols) {
        T g = src[r * cols + c];
        h_out[r * cols + c] = mine ? vals[pos] : g;
        if (gz_out) gz_out[r * cols + c] = mine ? (T)0 : g;
      }
      base += __popc(dead);
    }
  }
}

// float rows of a multiple of 128 columns: one warp per row, 128 columns (four sign words, one
// float4 per lane) per step, so that a warp keeps several 512-byte requests in flight; a lane's
// position in the stream = row offset + dead units of the earlier segments and words + dead bits
// below its nibble
template <int MODE>
__global__ void __launch_bounds__(kThreads)
fragment_row_vec4_kernel(const float* __restrict__ src, const uint32_t* __restrict__ words,
                         int64_t rows, int cols, const uint32_t* __restrict__ off,
                         float* __restrict__ vals, float* __restrict__ h_out,
                         float* __restrict__ gz_out) {
  const int lane = threadIdx.x & 31;
  const int64_t warp0 = ((int64_t)blockIdx.x * kThreads + threadIdx.x) >> 5;
  const int64_t nwarps = ((int64_t)gridDim.x * kThreads) >> 5;
  const int nseg = cols >> 7, wpr = cols >> 5;
  const int wi = lane >> 3;
  const unsigned sh = 4u * (unsigned)(lane & 7);
  for (int64_t r = warp0; r < rows; r += nwarps) {
    uint32_t base = off[r];
#pragma unroll 4
    for (int seg = 0; seg < nseg; ++seg) {
      const int64_t e0 = r * cols + seg * 128 + lane * 4;
      float4 v = *reinterpret_cast<const float4*>(src + e0);
      const unsigned dead_w = ~words[r * wpr + seg * 4 + wi];
      const unsigned c0 = __popc(__shfl_sync(0xffffffffu, dead_w, 0));
      const unsigned c1 = __popc(__shfl_sync(0xffffffffu, dead_w, 8));
      const unsigned c2 = __popc(__shfl_sync(0xffffffffu, dead_w, 16));
      const unsigned c3 = __popc(__shfl_sync(0xffffffffu, dead_w, 24));
      const unsigned before = (wi > 0 ? c0 : 0u) + (wi > 1 ? c1 : 0u) + (wi > 2 ? c2 : 0u) +
                              __popc(dead_w & ((1u << sh) - 1u));
      const unsigned nib = (dead_w >> sh) & 0xFu;
      uint32_t pos = base + before;
      if (MODE == 0) {
        if (nib & 1u) vals[pos++] = v.x;
        if (nib & 2u) vals[pos++] = v.y;
        if (nib & 4u) vals[pos++] = v.z;
        if (nib & 8u) vals[pos++] = v.w;
      } else {
        float4 h = v;
        if (nib & 1u) { h.x = vals[pos++]; v.x = 0.f; }
        if (nib & 2u) { h.y = vals[pos++]; v.y = 0.f; }
        if (nib & 4u) { h.z = vals[pos++]; v.z = 0.f; }
        if (nib & 8u) { h.w = vals[pos++]; v.w = 0.f; }
        *reinterpret_cast<float4*>(h_out + e0) = h;
        if (gz_out) *reinterpret_cast<float4*>(gz_out + e0) = v;
      }
      base += c0 + c1 + c2 + c3;
    }
  }
}

template <typename T>
mw_status fragment_compact(const T* h, const uint32_t* words, int64_t rows, int cols,
                           const uint32_t* off, T* vals, cudaStream_t s) {
  if (rows == 0 || cols == 0) return MW_OK;
  const int wpr = (cols + 31) / 32;
  if (vec_ok<T>(h, h, cols)) {
    fragment_row_vec4_kernel<0><<<grid_for(rows), kThreads, 0, s>>>(
        (const float*)h, words, rows, cols, off, (float*)vals, nullptr, nullptr);
    return launch_ok();
  }
  fragment_row_kernel<T, 0><<<grid_for(rows), kThreads, 0, s>>>(h, words, rows, cols, wpr, off,
                                                                vals, nullptr, nullptr);
  return launch_ok();
}

template <typename T>
mw_status activation_vijp(const T* gz, const uint32_t* words, int64_t rows, int cols, int act,
                          double slope, const uint32_t* off, const T* vals, T* h_out, T* gz_out,
                          cudaStream_t s) {
  if (rows == 0 || cols == 0) return MW_OK;
  const int wpr = (cols + 31) / 32;
  if (act == MW_ACT_RELU) {
    if (!off || !vals) return MW_ERR_INVALID_ARG;
    if (vec_ok<T>(gz, h_out, cols) && (!gz_out || ((uintptr_t)gz_out % 16 == 0)))
      fragment_row_vec4_kernel<1><<<grid_for(rows), kThreads, 0, s>>>(
          (const float*)gz, words, rows, cols, off, (float*)const_cast<T*>(vals), (float*)h_out,
          (float*)gz_out);
    else
      fragment_row_kernel<T, 1><<<grid_for(rows), kThreads, 0, s>>>(
          gz, words, rows, cols, wpr, off, const_cast<T*>(vals), h_out, gz_out);
  } else if (act == MW_ACT_LEAKY_RELU) {
    if (vec_ok<T>(gz, h_out, cols)) {
      const int64_t nseg = rows * (cols / 128);
      mask_scale_vec4_kernel<<<grid_for(nseg), kThreads, 0, s>>>(
          (const float*)gz, words, nseg, (float)slope, true, (float*)h_out);
    } else {
      mask_divide_kernel<T><<<grid_for(rows * wpr), kThreads, 0, s>>>(gz, words, rows, cols, wpr,
                                                                       (T)slope, h_out);
    }
    if (gz_out && gz_out != gz)
      MW_CUDA_OK(cudaMemcpyAsync(gz_out, gz, sizeof(T) * rows * cols, cudaMemcpyDeviceToDevice, s));
  } else {
    if (h_out != gz)
      MW_CUDA_OK(cudaMemcpyAsync(h_out, gz, sizeof(T) * rows * cols, cudaMemcpyDeviceToDevice, s));
    if (gz_out && gz_out != gz)
      MW_CUDA_OK(cudaMemcpyAsync(gz_out, gz, sizeof(T) * rows * cols, cudaMemcpyDeviceToDevice, s));
  }
  return launch_ok();
}

// ---------------------------------------------------------------------------------------
// losses
// ---------------------------------------------------------------------------------------
static constexpr int kLossBlocks = 512;

template <typename T>
__global__ void __launch_bounds__(kThreads)
sq_loss_kernel(const T* __restrict__ y, const T* __restrict__ t, int64_t n, T scale,
               T* __restrict__ h, double* __restrict__ partials) {
  __shared__ double red[kThreads];
  double acc = 0.0;
  for (int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x; i < n;
       i += (int64_t)gridDim.x * kThreads) {
    T d = y[i] - t[i];
    h[i] = scale * d;
    acc += (double)d * (double)d;
  }
  red[threadIdx.x] = acc;
  __syncthreads();
  for (int o = kThreads / 2; o; o >>= 1) {
    if (threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o];
    __syncthreads();
  }
  if (threadIdx.x == 0) partials[blockIdx.x] = red[0];
}

// one warp per row: softmax cross-entropy with integer labels
template <typename T>
__global__ void __launch_bounds__(kThreads)
xent_kernel(const T* __restrict__ y, const int32_t* __restrict__ label, int64_t rows, int cols,
            T* __restrict__ h, double* __restrict__ row_loss) {
  const int lane = threadIdx.x & 31;
  const int64_t warp0 = ((int64_t)blockIdx.x * kThreads + threadIdx.x) >> 5;
  const int64_t nwarps = ((int64_t)gridDim.x * kThreads) >> 5;
  for (int64_t r = warp0; r < rows; r += nwarps) {
    double mx = -1e300;
    for (int c = lane; c < cols; c += 32) mx = fmax(mx, (double)y[r * cols + c]);
    for (int o = 16; o; o >>= 1) mx = fmax(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    double se = 0.0;
    for (int c = lane; c < cols; c += 32) se += exp((double)y[r * cols + c] - mx);
    for (int o = 16; o; o >>= 1) se += __shfl_xor_sync(0xffffffffu, se, o);
    const int lab = label[r];
    for (int c = lane; c < cols; c += 32) {
      double p = exp((double)y[r * cols + c] - mx) / se;
      h[r * cols + c] = (T)((p - (c == lab ? 1.0 : 0.0)) / (double)rows);
    }
    if (lane == 0) row_loss[r] = -(((double)y[r * cols + lab] - mx) - log(se));
  }
}

__global__ void final_sum_kernel(const double* __restrict__ partials, int64_t n, double scale,
                                 double* __restrict__ out) {
  // one thread, fixed order: deterministic
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    double a = 0.0;
    for (int64_t i = 0; i < n; ++i) a += partials[i];
    *out = a * scale;
  }
}

template <typename T>
mw_status loss_cotangent(const T* y, const void* target, int64_t rows, int cols, int loss, T* h,
                         double* partials, double* loss_out, cudaStream_t s) {
  const int64_t n = rows * cols;
  if (n == 0) return MW_OK;
  if (loss == MW_LOSS_HALF_SSE || loss == MW_LOSS_MSE_MEAN) {
    const double scale = loss == MW_LOSS_HALF_SSE ? 1.0 : 2.0 / (double)n;
    int blocks = (int)((n + kThreads - 1) / kThreads);
    if (blocks > kLossBlocks) blocks = kLossBlocks;
    sq_loss_kernel<T><<<blocks, kThreads, 0, s>>>(y, (const T*)target, n, (T)scale, h, partials);
    if (loss_out) {
      final_sum_kernel<<<1, 32, 0, s>>>(partials, blocks,
                                        loss == MW_LOSS_HALF_SSE ? 0.5 : 1.0 / (double)n, loss_out);
      ++g_launch_count;
    }
  } else if (loss == MW_LOSS_XENT_MEAN) {
    if (rows > 1 << 20) return MW_ERR_UNSUPPORTED;
    xent_kernel<T><<<grid_for(rows), kThreads, 0, s>>>(y, (const int32_t*)target, rows, cols, h,
                                                       partials);
    if (loss_out) {
      final_sum_kernel<<<1, 32, 0, s>>>(partials, rows, 1.0 / (double)rows, loss_out);
      ++g_launch_count;
    }
  } else {
    return MW_ERR_INVALID_ARG;
  }
  return launch_ok();
}

template <typename TI, typename TO>
__global__ void __launch_bounds__(kThreads)
convert_kernel(const TI* __restrict__ in, TO* __restrict__ out, int64_t n) {
  for (int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x; i < n;
       i += (int64_t)gridDim.x * kThreads) {
    if constexpr (std::is_same<TI, double>::value) {
      out[i] = from_f64<TO>(in[i]);
    } else {
      out[i] = from_f64<TO>((double)to_f32(in[i]));
    }
  }
}

template <typename TI, typename TO>
mw_status convert_array(const TI* in, TO* out, int64_t n, cudaStream_t s) {
  if (n == 0) return MW_OK;
  int64_t blocks = (n + kThreads - 1) / kThreads;
  if (blocks > 148 * 16) blocks = 148 * 16;
  convert_kernel<TI, TO><<<(int)blocks, kThreads, 0, s>>>(in, out, n);
  return launch_ok();
}

// explicit instantiations
#define MW_INST_T(T)                                                                              \
  template mw_status pack_sign_bits<T>(const T*, int64_t, int, uint32_t*, cudaStream_t);         \
  template mw_status scale_by_mask<T>(const T*, const uint32_t*, int64_t, int, int, double, T*,  \
                                      cudaStream_t);                                             \
  template mw_status activation_vijp<T>(const T*, const uint32_t*, int64_t, int, int, double,    \
                                        const uint32_t*, const T*, T*, T*, cudaStream_t);        \
  template mw_status fragment_compact<T>(const T*, const uint32_t*, int64_t, int,                \
                                         const uint32_t*, T*, cudaStream_t);                     \
  template mw_status loss_cotangent<T>(const T*, const void*, int64_t, int, int, T*, double*,    \
                                       double*, cudaStream_t);
MW_INST_T(float)
MW_INST_T(double)
template mw_status pack_sign_bits<__nv_bfloat16>(const __nv_bfloat16*, int64_t, int, uint32_t*,
                                                 cudaStream_t);
template mw_status act_forward_pack<float, float>(const float*, int64_t, int, int, double, float*,
                                                  uint32_t*, bool, cudaStream_t);
template mw_status act_forward_pack<float, __nv_bfloat16>(const float*, int64_t, int, int, double,
                                                          __nv_bfloat16*, uint32_t*, bool,
                                                          cudaStream_t);
template mw_status act_forward_pack<double, double>(const double*, int64_t, int, int, double,
                                                    double*, uint32_t*, bool, cudaStream_t);
template mw_status convert_array<float, __nv_bfloat16>(const float*, __nv_bfloat16*, int64_t,
                                                       cudaStream_t);
template mw_status convert_array<__nv_bfloat16, float>(const __nv_bfloat16*, float*, int64_t,
                                                       cudaStream_t);
template mw_status convert_array<float, float>(const float*, float*, int64_t, cudaStream_t);
template mw_status convert_array<double, double>(const double*, double*, int64_t, cudaStream_t);

}  // namespace mw
