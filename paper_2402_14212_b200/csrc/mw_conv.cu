// Convolution steps of the Moonwalk sweep on CUDA cores (channel-last, stride 1, same size).
//
//   forward        x'[i',c'] = sum_{j,c} w[j,c,c'] x[i'+j-p, c]                  (Lemma 1)
//   TransposeConv  h[i,c]    = sum_{j,c'} w[j,c,c'] h'[i+p-j, c']                (Eq. "conv-vjp")
//   weight vjp     dw[j,c,c'] = sum_{b,i'} x[b,i'+j-p,c] g_z[b,i',c']            (Eq. "g_i")
//   vijp           the g with TransposeConv(g, w) = h, by the elimination relation of Lemma 1's
//                  proof outline used as a fixed-point iteration on the whole centre tap:
//                  g <- h W_c^-T - TransposeConv(g, w^),  w^[j] = W_c^-1 w[j] (j != centre), 0 at centre
//
// All four are written as implicit products over (pixel, tap*channel) so one tiled kernel serves
// them; the gather for the shifted pixel happens while the A tile is staged in shared memory.
#include "mw_common.cuh"
#include "mw_conv.cuh"

namespace mw {

// out[m][n] = (mode ? base[m][n] - acc : acc),  acc = sum_{tap,ci} in[shift(m,tap)][ci] * wsel
// m = (b, y, x) flattened; shift: (y + sgn*(j0-p), x + sgn*(j1-p)); wsel = wtrans ? w[tap][n][ci]
// : w[tap][ci][n].
template <typename T>
__global__ void __launch_bounds__(256)
conv_igemm_kernel(const T* __restrict__ in, const T* __restrict__ w, T* __restrict__ out,
                  const T* __restrict__ base, int Bn, int H, int W, int Ci, int Co, int k, int pad,
                  int sgn, int wtrans, int mode) {
  __shared__ T As[16][64 + 1];
  __shared__ T Bs[16][64 + 1];
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  const int64_t M = (int64_t)Bn * H * W;
  const int64_t m0 = (int64_t)blockIdx.y * 64;
  const int n0 = blockIdx.x * 64;
  const int K = k * k * Ci;
  T acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = (T)0;
  for (int k0 = 0; k0 < K; k0 += 16) {
    for (int e = threadIdx.x; e < 64 * 16; e += 256) {
      const int kk = e & 15, mm = e >> 4;
      const int64_t gm = m0 + mm;
      const int gk = k0 + kk;
      T v = (T)0;
      if (gm < M && gk < K) {
        const int tap = gk / Ci, ci = gk - tap * Ci;
        const int j0 = tap / k, j1 = tap - j0 * k;
        const int x = (int)(gm % W);
        const int y = (int)((gm / W) % H);
        const int64_t b = gm / ((int64_t)W * H);
        const int yy = y + sgn * (j0 - pad), xx = x + sgn * (j1 - pad);
        if (yy >= 0 && yy < H && xx >= 0 && xx < W)
          v = in[((b * H + yy) * W + xx) * Ci + ci];
      }
      As[kk][mm] = v;
    }
    for (int e = threadIdx.x; e < 64 * 16; e += 256) {
      const int nn = e & 63, kk = e >> 6;
      const int gn = n0 + nn, gk = k0 + kk;
      T v = (T)0;
      if (gn < Co && gk < K) {
        const int tap = gk / Ci, ci = gk - tap * Ci;
        v = wtrans ? w[((int64_t)tap * Co + gn) * Ci + ci] : w[((int64_t)tap * Ci + ci) * Co + gn];
      }
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
    const int64_t gm = m0 + ty * 4 + i;
    if (gm >= M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int gn = n0 + tx * 4 + j;
      if (gn >= Co) continue;
      const int64_t o = gm * Co + gn;
      out[o] = mode ? base[o] - acc[i][j] : acc[i][j];
    }
  }
}

template <typename T>
mw_status conv_igemm(const T* in, const T* w, T* out, const T* base, int Bn, int H, int W, int Ci,
                     int Co, int k, int pad, int sgn, int wtrans, int mode, cudaStream_t s) {
  const int64_t M = (int64_t)Bn * H * W;
  if (M == 0) return MW_OK;
  dim3 grid(ceil_div(Co, 64), ceil_div(M, 64));
  if (grid.y > 65535) {
    // fold the pixel tiles over x when there are too many for gridDim.y
    return MW_ERR_UNSUPPORTED;
  }
  conv_igemm_kernel<T><<<grid, 256, 0, s>>>(in, w, out, base, Bn, H, W, Ci, Co, k, pad, sgn,
                                            wtrans, mode);
  return launch_ok();
}

// part[z][(tap,c)][c'] = sum over the z-th slice of pixels of x[shift(m,tap)][c] * gz[m][c']
template <typename T>
__global__ void __launch_bounds__(256)
conv_wgrad_kernel(const T* __restrict__ x, const T* __restrict__ gz, T* __restrict__ part, int Bn,
                  int H, int W, int Ci, int Co, int k, int pad, int64_t slice) {
  __shared__ T As[16][64 + 1];  // [pixel kk][row (tap,c)]
  __shared__ T Bs[16][64 + 1];  // [pixel kk][c']
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  const int64_t Mpix = (int64_t)Bn * H * W;
  const int R = k * k * Ci;
  const int r0 = blockIdx.y * 64, n0 = blockIdx.x * 64;
  const int64_t p_begin = (int64_t)blockIdx.z * slice;
  int64_t p_end = p_begin + slice;
  if (p_end > Mpix) p_end = Mpix;
  T acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = (T)0;
  for (int64_t p0 = p_begin; p0 < p_end; p0 += 16) {
    for (int e = threadIdx.x; e < 64 * 16; e += 256) {
      const int rr = e & 63, kk = e >> 6;
      const int gr = r0 + rr;
      const int64_t gm = p0 + kk;
      T v = (T)0;
      if (gr < R && gm < p_end) {
        const int tap = gr / Ci, ci = gr - tap * Ci;
        const int j0 = tap / k, j1 = tap - j0 * k;
        const int xx0 = (int)(gm % W);
        const int yy0 = (int)((gm / W) % H);
        const int64_t b = gm / ((int64_t)W * H);
        const int yy = yy0 + j0 - pad, xx = xx0 + j1 - pad;
        if (yy >= 0 && yy < H && xx >= 0 && xx < W) v = x[((b * H + yy) * W + xx) * Ci + ci];
      }
      As[kk][rr] = v;
    }
    for (int e = threadIdx.x; e < 64 * 16; e += 256) {
      const int nn = e & 63, kk = e >> 6;
      const int gn = n0 + nn;
      const int64_t gm = p0 + kk;
      Bs[kk][nn] = (gn < Co && gm < p_end) ? gz[gm * Co + gn] : (T)0;
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
  T* dst = part + (int64_t)blockIdx.z * R * Co;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int gr = r0 + ty * 4 + i;
    if (gr >= R) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int gn = n0 + tx * 4 + j;
      if (gn < Co) dst[(int64_t)gr * Co + gn] = acc[i][j];
    }
  }
}

template <typename T>
__global__ void __launch_bounds__(256)
slice_sum_kernel(const T* __restrict__ part, int64_t n, int slices, T* __restrict__ out) {
  const int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x;
  if (i >= n) return;
  double a = 0.0;
  for (int z = 0; z < slices; ++z) a += (double)part[(int64_t)z * n + i];  // fixed order
  out[i] = (T)a;
}

int conv_wgrad_slices(int64_t pixels) {
  int64_t s = (pixels + 2047) / 2048;
  if (s < 1) s = 1;
  if (s > 128) s = 128;
  return (int)s;
}

template <typename T>
mw_status conv_wgrad(const T* x, const T* gz, T* dw, T* scratch, int Bn, int H, int W, int Ci,
                     int Co, int k, int pad, cudaStream_t s) {
  const int64_t Mpix = (int64_t)Bn * H * W;
  const int R = k * k * Ci;
  const int slices = conv_wgrad_slices(Mpix);
  const int64_t slice = ((Mpix + slices - 1) / slices + 15) / 16 * 16;
  dim3 grid(ceil_div(Co, 64), ceil_div(R, 64), slices);
  conv_wgrad_kernel<T><<<grid, 256, 0, s>>>(x, gz, scratch, Bn, H, W, Ci, Co, k, pad, slice);
  const int64_t n = (int64_t)R * Co;
  slice_sum_kernel<T><<<ceil_div(n, 256), 256, 0, s>>>(scratch, n, slices, dw);
  return launch_ok(2);
}

// zero one k*k tap [Ci][Co] block
template <typename T>
__global__ void zero_kernel(T* p, int64_t n) {
  const int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x;
  if (i < n) p[i] = (T)0;
}

template <typename T>
mw_status zero_array(T* p, int64_t n, cudaStream_t s) {
  if (n == 0) return MW_OK;
  zero_kernel<T><<<ceil_div(n, 256), 256, 0, s>>>(p, n);
  return launch_ok();
}

template mw_status conv_igemm<float>(const float*, const float*, float*, const float*, int, int,
                                     int, int, int, int, int, int, int, int, cudaStream_t);
template mw_status conv_igemm<double>(const double*, const double*, double*, const double*, int,
                                      int, int, int, int, int, int, int, int, int, cudaStream_t);
template mw_status conv_wgrad<float>(const float*, const float*, float*, float*, int, int, int, int,
                                     int, int, int, cudaStream_t);
template mw_status conv_wgrad<double>(const double*, const double*, double*, double*, int, int, int,
                                      int, int, int, int, cudaStream_t);
template mw_status zero_array<float>(float*, int64_t, cudaStream_t);
template mw_status zero_array<double>(double*, int64_t, cudaStream_t);

}  // namespace mw
