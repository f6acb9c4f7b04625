// Small kernels beside the fused step: standalone de-bias (Alg. 1 line 8) and the invariant scan
// (column-stochastic mixing conserves sum_i w_i and sum_i x_i, counting messages in transit).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace sgp {

// Z[i, :] = X[i, :] * (1 / W[i]).  grid.y = node, grid.x strides over the row.
template <int VEC>
__global__ void __launch_bounds__(256) sgp_debias_kernel(const float *__restrict__ X, const float *__restrict__ W,
                                                          float *__restrict__ Z, int64_t d, int64_t ld) {
  const int row = blockIdx.y;
  const float inv = 1.0f / W[row];
  const int64_t base = static_cast<int64_t>(row) * ld;
  if (VEC == 4) {
    const int64_t nvec = d >> 2;
    const float4 *x4 = reinterpret_cast<const float4 *>(X + base);
    float4 *z4 = reinterpret_cast<float4 *>(Z + base);
    for (int64_t v = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; v < nvec;
         v += static_cast<int64_t>(gridDim.x) * blockDim.x) {
      float4 a = __ldcs(x4 + v);
      a.x *= inv; a.y *= inv; a.z *= inv; a.w *= inv;
      __stcs(z4 + v, a);
    }
    // ragged end of the row (d not a multiple of 4)
    if (blockIdx.x == 0) {
      const int64_t c = (nvec << 2) + threadIdx.x;
      if (c < d) Z[base + c] = X[base + c] * inv;
    }
  } else {
    for (int64_t c = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; c < d;
         c += static_cast<int64_t>(gridDim.x) * blockDim.x)
      Z[base + c] = X[base + c] * inv;
  }
}

__device__ __forceinline__ double warp_sum(double v) {
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// out[0] += sum of finite entries of A (rows x d, pitch ld); out[1] += number of non-finite entries.
__global__ void __launch_bounds__(256) sgp_scan_kernel(const float *__restrict__ A, int rows, int64_t d, int64_t ld,
                                                        double *out) {
  double s = 0.0, bad = 0.0;
  const int64_t total = static_cast<int64_t>(rows) * d;
  for (int64_t t = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; t < total;
       t += static_cast<int64_t>(gridDim.x) * blockDim.x) {
    const int64_t r = t / d, c = t - r * d;
    const float v = A[r * ld + c];
    if (isfinite(v)) s += static_cast<double>(v);
    else bad += 1.0;
  }
  s = warp_sum(s);
  bad = warp_sum(bad);
  if ((threadIdx.x & 31) == 0) {
    atomicAdd(out + 0, s);
    if (bad != 0.0) atomicAdd(out + 1, bad);
  }
}

// out[2] += sum_i W_i (+ ring weights); out[3] = min_i W_i (single CTA; n <= 256, ring of tau*n).
__global__ void __launch_bounds__(256) sgp_weight_scan_kernel(const float *__restrict__ W, int n,
                                                               const float *__restrict__ ring_w, int ring_len,
                                                               double *out) {
  __shared__ double s_sum[8];
  __shared__ float s_min[8];
  double s = 0.0;
  float mn = 3.4e38f;
  for (int i = threadIdx.x; i < n; i += blockDim.x) {
    s += static_cast<double>(W[i]);
    mn = fminf(mn, W[i]);
  }
  for (int i = threadIdx.x; i < ring_len; i += blockDim.x) s += static_cast<double>(ring_w[i]);
  s = warp_sum(s);
  for (int o = 16; o > 0; o >>= 1) mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
  if ((threadIdx.x & 31) == 0) {
    s_sum[threadIdx.x >> 5] = s;
    s_min[threadIdx.x >> 5] = mn;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    double t = 0.0;
    float m = 3.4e38f;
    for (int w = 0; w < static_cast<int>(blockDim.x >> 5); ++w) {
      t += s_sum[w];
      m = fminf(m, s_min[w]);
    }
    out[2] = t;
    out[3] = static_cast<double>(m);
  }
}

// Parameter deviation (Sec. 6.1 "Parameter deviations", Fig. 2): out[i] += sum over this CTA's columns of
// (A[i][c] - mean_j A[j][c])^2.  A CTA stages n rows x tile_cols columns in shared memory, forms the
// column means, then every warp reduces whole rows.  One read of A, nothing else.
__global__ void __launch_bounds__(256) sgp_deviation_kernel(const float *__restrict__ A, int n, int64_t d, int64_t ld,
                                                             int tile_cols, double *out) {
  extern __shared__ float dev_smem[];
  float *tile = dev_smem;                         // n x tile_cols
  float *mean = tile + static_cast<size_t>(n) * tile_cols;
  float *acc = mean + tile_cols;                  // n partial sums of this CTA
  for (int i = threadIdx.x; i < n; i += blockDim.x) acc[i] = 0.f;
  const int64_t ntiles = (d + tile_cols - 1) / tile_cols;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
  const float inv_n = 1.0f / static_cast<float>(n);
  for (int64_t t = blockIdx.x; t < ntiles; t += gridDim.x) {
    const int64_t col0 = t * tile_cols;
    const int valid = static_cast<int>(min(static_cast<int64_t>(tile_cols), d - col0));
    __syncthreads();
    for (int r = warp; r < n; r += nwarps)
      for (int c = lane; c < valid; c += 32) tile[r * tile_cols + c] = __ldcs(A + static_cast<int64_t>(r) * ld + col0 + c);
    __syncthreads();
    for (int c = threadIdx.x; c < valid; c += blockDim.x) {
      float s = 0.f;
      for (int r = 0; r < n; ++r) s += tile[r * tile_cols + c];
      mean[c] = s * inv_n;
    }
    __syncthreads();
    for (int r = warp; r < n; r += nwarps) {
      float q = 0.f;
      for (int c = lane; c < valid; c += 32) {
        const float e = tile[r * tile_cols + c] - mean[c];
        q = fmaf(e, e, q);
      }
      for (int o = 16; o > 0; o >>= 1) q += __shfl_xor_sync(0xffffffffu, q, o);
      if (lane == 0) acc[r] += q;                 // row r belongs to this warp only: no race
    }
  }
  __syncthreads();
  for (int i = threadIdx.x; i < n; i += blockDim.x) atomicAdd(out + i, static_cast<double>(acc[i]));
}

}  // namespace sgp
