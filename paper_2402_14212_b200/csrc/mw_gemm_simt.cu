// CUDA-core products and inverses: the exact-arithmetic backend (fp64 nets, odd sizes, and the
// A/B check of the tensor-core path).  Dense-layer steps of the Moonwalk sweep expressed with it:
//   recompute   z   = x W^T            (Algorithm 1, line x_i <- f_i)
//   dense vijp  g_z = h W^-1           (Eq. "h_i" for a square invertible layer)
//   weight vjp  dW  = g_z^T x          (Eq. "g_i")
#include "mw_common.cuh"

namespace mw {

// ---------------------------------------------------------------------------------------
// C = alpha * op(A) op(B) + beta * C, 64x64 tile, 16-deep slices, 4x4 outputs per thread
// ---------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256)
gemm_simt_kernel(int ta, int tb, int M, int N, int K, T alpha, const T* __restrict__ A, int lda,
                 const T* __restrict__ B, int ldb, T beta, T* __restrict__ C, int ldc) {
  __shared__ T As[16][64 + 1];
  __shared__ T Bs[16][64 + 1];
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  const int m0 = blockIdx.y * 64, n0 = blockIdx.x * 64;
  T acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = (T)0;
  for (int k0 = 0; k0 < K; k0 += 16) {
    for (int e = threadIdx.x; e < 64 * 16; e += 256) {
      int kk, mm;
      if (ta) { mm = e & 63; kk = e >> 6; } else { kk = e & 15; mm = e >> 4; }
      const int gm = m0 + mm, gk = k0 + kk;
      T v = (T)0;
      if (gm < M && gk < K) v = ta ? A[(int64_t)gk * lda + gm] : A[(int64_t)gm * lda + gk];
      As[kk][mm] = v;
    }
    for (int e = threadIdx.x; e < 64 * 16; e += 256) {
      int kk, nn;
      if (tb) { kk = e & 15; nn = e >> 4; } else { nn = e & 63; kk = e >> 6; }
      const int gn = n0 + nn, gk = k0 + kk;
      T v = (T)0;
      if (gn < N && gk < K) v = tb ? B[(int64_t)gn * ldb + gk] : B[(int64_t)gk * ldb + gn];
      Bs[kk][nn] = v;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < 16; ++kk) {
      T a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = As[kk][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) b[j] = Bs[kk][tx * 4 + j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fma(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int gm = m0 + ty * 4 + i;
    if (gm >= M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int gn = n0 + tx * 4 + j;
      if (gn >= N) continue;
      T* p = C + (int64_t)gm * ldc + gn;
      T v = alpha * acc[i][j];
      if (beta != (T)0) v += beta * (*p);
      *p = v;
    }
  }
}

template <typename T>
mw_status gemm_simt(int ta, int tb, int M, int N, int K, double alpha, const T* A, int lda,
                    const T* B, int ldb, double beta, T* C, int ldc, cudaStream_t s) {
  if (M == 0 || N == 0) return MW_OK;
  dim3 grid(ceil_div(N, 64), ceil_div(M, 64));
  if (grid.y > 65535) return MW_ERR_UNSUPPORTED;
  gemm_simt_kernel<T><<<grid, 256, 0, s>>>(ta, tb, M, N, K, (T)alpha, A, lda, B, ldb, (T)beta, C,
                                           ldc);
  return launch_ok();
}

// ---------------------------------------------------------------------------------------
// Gauss-Jordan with partial pivoting, one CTA, n <= 64, double arithmetic in shared memory
// ---------------------------------------------------------------------------------------
template <typename T>
__device__ __forceinline__ void inverse_small_body(const T* __restrict__ W, int n, T* __restrict__ Winv,
                                                   DeviceStatus* st, int layer) {
  extern __shared__ double aug[];  // [n][2n]
  __shared__ int piv_s;
  __shared__ double pval_s;
  const int w2 = 2 * n;
  for (int e = threadIdx.x; e < n * w2; e += blockDim.x) {
    const int i = e / w2, j = e - i * w2;
    aug[e] = j < n ? (double)W[i * n + j] : (j - n == i ? 1.0 : 0.0);
  }
  __syncthreads();
  for (int k = 0; k < n; ++k) {
    if (threadIdx.x == 0) {
      int p = k;
      double best = fabs(aug[k * w2 + k]);
      for (int i = k + 1; i < n; ++i) {
        double v = fabs(aug[i * w2 + k]);
        if (v > best) { best = v; p = i; }
      }
      piv_s = p;
      pval_s = aug[p * w2 + k];
    }
    __syncthreads();
    const int p = piv_s;
    const double pv = pval_s;
    if (!(fabs(pv) > 1e-300)) {
      if (threadIdx.x == 0) record_error(st, MW_ERR_NOT_SUBMERSIVE, (unsigned)layer, (unsigned)k, 1u, 0u);
      return;
    }
    for (int j = threadIdx.x; j < w2; j += blockDim.x) {
      double a = aug[k * w2 + j], b = aug[p * w2 + j];
      aug[p * w2 + j] = a;
      aug[k * w2 + j] = b / pv;
    }
    __syncthreads();
    // eliminate column k from every other row; factors read before any write of column k
    for (int i = threadIdx.x >> 5; i < n; i += (blockDim.x >> 5)) {
      if (i == k) continue;
      const double f = aug[i * w2 + k];
      __syncwarp();
      for (int j = threadIdx.x & 31; j < w2; j += 32) aug[i * w2 + j] -= f * aug[k * w2 + j];
    }
    __syncthreads();
  }
  for (int e = threadIdx.x; e < n * n; e += blockDim.x) {
    const int i = e / n, j = e - i * n;
    Winv[e] = (T)aug[i * w2 + n + j];
  }
}

template <typename T>
__global__ void __launch_bounds__(256)
inverse_small_kernel(const T* __restrict__ W, int n, T* __restrict__ Winv, DeviceStatus* st,
                     int layer) {
  inverse_small_body<T>(W, n, Winv, st, layer);
}

// one CTA per matrix: matrix b is Ws.p[b] + offset, its inverse lands at Winv + b*n*n
template <typename T>
__global__ void __launch_bounds__(256)
inverse_small_batch_kernel(SmallBatch Ws, int64_t offset, int n, T* __restrict__ Winv,
                           DeviceStatus* st, int layer0) {
  inverse_small_body<T>(static_cast<const T*>(Ws.p[blockIdx.x]) + offset, n,
                        Winv + (int64_t)blockIdx.x * n * n, st, layer0 + (int)blockIdx.x);
}

template <typename T>
mw_status inverse_small(const T* W, int n, T* Winv, DeviceStatus* st, int layer, cudaStream_t s) {
  if (n < 1 || n > 64) return MW_ERR_UNSUPPORTED;
  const size_t smem = sizeof(double) * n * 2 * n;
  static bool attr_done = false;
  if (!attr_done) {
    MW_CUDA_OK(cudaFuncSetAttribute(inverse_small_kernel<T>,
                                    cudaFuncAttributeMaxDynamicSharedMemorySize, 65536));
    attr_done = true;
  }
  inverse_small_kernel<T><<<1, 256, smem, s>>>(W, n, Winv, st, layer);
  return launch_ok();
}

template <typename T>
mw_status inverse_small_batch(const SmallBatch& Ws, int count, int64_t offset, int n, T* Winv,
                              DeviceStatus* st, int layer0, cudaStream_t s) {
  if (n < 1 || n > 64 || count < 1 || count > kSmallBatch) return MW_ERR_UNSUPPORTED;
  const size_t smem = sizeof(double) * n * 2 * n;
  static bool attr_done = false;
  if (!attr_done) {
    MW_CUDA_OK(cudaFuncSetAttribute(inverse_small_batch_kernel<T>,
                                    cudaFuncAttributeMaxDynamicSharedMemorySize, 65536));
    attr_done = true;
  }
  inverse_small_batch_kernel<T><<<count, 256, smem, s>>>(Ws, offset, n, Winv, st, layer0);
  return launch_ok();
}
template mw_status inverse_small_batch<float>(const SmallBatch&, int, int64_t, int, float*,
                                              DeviceStatus*, int, cudaStream_t);

// ---------------------------------------------------------------------------------------
// Newton-Schulz on CUDA cores: X <- 2X - X (W X), X_0 = (n / ||W||_F^2) W^T
// ---------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(1024)
frob_scale_kernel(const T* __restrict__ W, int64_t n2, int n, double* __restrict__ c_out) {
  __shared__ double red[1024];
  double a = 0.0;
  for (int64_t i = threadIdx.x; i < n2; i += 1024) a += (double)W[i] * (double)W[i];
  red[threadIdx.x] = a;
  __syncthreads();
  for (int o = 512; o; o >>= 1) {
    if (threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o];
    __syncthreads();
  }
  if (threadIdx.x == 0) *c_out = red[0] > 0.0 ? (double)n / red[0] : 0.0;
}

template <typename T>
__global__ void __launch_bounds__(256)
scaled_transpose_kernel(const T* __restrict__ W, int n, const double* __restrict__ c, T* __restrict__ X) {
  __shared__ T tile[32][33];
  const int bx = blockIdx.x * 32, by = blockIdx.y * 32;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  for (int r = ty; r < 32; r += 8)
    if (by + r < n && bx + tx < n) tile[r][tx] = W[(int64_t)(by + r) * n + bx + tx];
  __syncthreads();
  const T cc = (T)(*c);
  for (int r = ty; r < 32; r += 8)
    if (bx + r < n && by + tx < n) X[(int64_t)(bx + r) * n + by + tx] = cc * tile[tx][r];
}

// ||I - P||_F^2 with P = W X; records NOT_SUBMERSIVE if above tol^2 * n
template <typename T>
__global__ void __launch_bounds__(1024)
residual_check_kernel(const T* __restrict__ P, int n, double tol, DeviceStatus* st, int layer) {
  __shared__ double red[1024];
  double a = 0.0;
  const int64_t n2 = (int64_t)n * n;
  for (int64_t i = threadIdx.x; i < n2; i += 1024) {
    const int r = (int)(i / n), c = (int)(i - (int64_t)r * n);
    double d = (r == c ? 1.0 : 0.0) - (double)P[i];
    a += d * d;
  }
  red[threadIdx.x] = a;
  __syncthreads();
  for (int o = 512; o; o >>= 1) {
    if (threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o];
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    const double r2 = red[0];
    if (!(r2 <= tol * tol * (double)n))
      record_error(st, MW_ERR_NOT_SUBMERSIVE, (unsigned)layer, __float_as_uint((float)sqrt(r2)), 2u, 0u);
  }
}

template <typename T>
mw_status inverse_newton_simt(const T* W, int n, int iters, T* X, T* scratch, DeviceStatus* st,
                              int layer, double tol, cudaStream_t s) {
  // scratch: P [n*n], Xn [n*n], then one double (the scale) at the end, 8-byte aligned
  T* P = scratch;
  T* Xn = scratch + (size_t)n * n;
  double* c = reinterpret_cast<double*>(align_up((size_t)(uintptr_t)(Xn + (size_t)n * n), 8));
  frob_scale_kernel<T><<<1, 1024, 0, s>>>(W, (int64_t)n * n, n, c);
  dim3 tg(ceil_div(n, 32), ceil_div(n, 32));
  scaled_transpose_kernel<T><<<tg, 256, 0, s>>>(W, n, c, X);
  g_launch_count += 2;
  const size_t bytes = sizeof(T) * (size_t)n * n;
  for (int it = 0; it < iters; ++it) {
    MW_TRY(gemm_simt<T>(0, 0, n, n, n, 1.0, W, n, X, n, 0.0, P, n, s));         // P = W X
    MW_CUDA_OK(cudaMemcpyAsync(Xn, X, bytes, cudaMemcpyDeviceToDevice, s));
    MW_TRY(gemm_simt<T>(0, 0, n, n, n, -1.0, X, n, P, n, 2.0, Xn, n, s));       // Xn = 2X - X P
    MW_CUDA_OK(cudaMemcpyAsync(X, Xn, bytes, cudaMemcpyDeviceToDevice, s));
  }
  MW_TRY(gemm_simt<T>(0, 0, n, n, n, 1.0, W, n, X, n, 0.0, P, n, s));
  residual_check_kernel<T><<<1, 1024, 0, s>>>(P, n, tol, st, layer);
  return launch_ok();
}

template mw_status gemm_simt<float>(int, int, int, int, int, double, const float*, int,
                                    const float*, int, double, float*, int, cudaStream_t);
template mw_status gemm_simt<double>(int, int, int, int, int, double, const double*, int,
                                     const double*, int, double, double*, int, cudaStream_t);
template mw_status inverse_small<float>(const float*, int, float*, DeviceStatus*, int, cudaStream_t);
template mw_status inverse_small<double>(const double*, int, double*, DeviceStatus*, int,
                                         cudaStream_t);
template mw_status inverse_newton_simt<float>(const float*, int, int, float*, float*,
                                              DeviceStatus*, int, double, cudaStream_t);
template mw_status inverse_newton_simt<double>(const double*, int, int, double*, double*,
                                               DeviceStatus*, int, double, cudaStream_t);

}  // namespace mw
