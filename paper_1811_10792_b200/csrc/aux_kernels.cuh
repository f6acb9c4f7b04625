// Small kernels beside the fused step: standalone de-bias (Alg. 1 line 8), the invariant checks of
// column-stochastic mixing (Sec. 2: 1^T P = 1^T, so sum_i w_i and every column sum of X are conserved, counting
// the messages in transit of the delay model), and the standalone parameter-deviation pass (Sec. 6.1, Fig. 2).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "step_common.cuh"

namespace sgp {

// Z[i, :] = X[i, :] * (1 / W[i]).  grid.y = node, grid.x strides over the row.  A weight that is not positive
// gives zeros and a status bit, never inf.
template <int VEC>
__global__ void __launch_bounds__(256) sgp_debias_kernel(const float *__restrict__ X, const float *__restrict__ W,
                                                          float *__restrict__ Z, int64_t d, int64_t ld, int biased,
                                                          unsigned *status) {
  const int row = blockIdx.y;
  float inv = 1.0f;
  if (!biased) {
    const float w = W[row];
    inv = w > 0.0f ? 1.0f / w : 0.0f;
    if (!(w > 0.0f) && blockIdx.x == 0 && threadIdx.x == 0) atomicOr(status, kStatusZeroWeight);
  }
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
__device__ __forceinline__ double warp_max(double v) {
  for (int o = 16; o > 0; o >>= 1) v = fmax(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
// Non-negative doubles order like their bit patterns, so a 64-bit integer atomicMax keeps the largest.
__device__ __forceinline__ void atomic_max_nonneg(double *addr, double v) {
  atomicMax(reinterpret_cast<unsigned long long *>(addr), static_cast<unsigned long long>(__double_as_longlong(v)));
}

// Device-side layout of the invariant statistics (doubles).
enum : int { kStatTotal = 0, kStatNonFinite = 1, kStatSumW = 2, kStatMinW = 3, kStatMaxDrift = 4, kStatMaxRelDrift = 5, kStatCount = 6 };

// Per-column sums in fp64.  One thread owns one column and walks down the rows of A (rows x d, pitch ld) and of
// every ring slot (ring_rows = tau * n rows of the same pitch), so that a warp reads 128 contiguous bytes per row
// and no index needs a division.  For column c:
//     s = sum_r A[r, c] + sum_r ring[r, c]          a = the same sum of absolute values
// out (optional) receives s; with ref given the drift |s - ref[c]| and the relative drift |s - ref[c]| / a are
// max-reduced (warp shuffles, one atomic per warp) into stats.  Non-finite entries are counted and left out.
__global__ void __launch_bounds__(256) sgp_colsum_kernel(const float *__restrict__ A, int rows, int64_t d, int64_t ld,
                                                          const float *__restrict__ ring, int ring_rows,
                                                          double *__restrict__ out, const double *__restrict__ ref,
                                                          double *stats) {
  double total = 0.0, bad = 0.0, max_drift = 0.0, max_rel = 0.0;
  for (int64_t c = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; c < d;
       c += static_cast<int64_t>(gridDim.x) * blockDim.x) {
    double s = 0.0, a = 0.0;
    const float *col = A + c;
    int r = 0;
    for (; r + 8 <= rows; r += 8) {
      float v[8];
#pragma unroll
      for (int q = 0; q < 8; ++q) v[q] = __ldcs(col + static_cast<int64_t>(r + q) * ld);
#pragma unroll
      for (int q = 0; q < 8; ++q) {
        if (isfinite(v[q])) { s += static_cast<double>(v[q]); a += static_cast<double>(fabsf(v[q])); }
        else bad += 1.0;
      }
    }
    for (; r < rows; ++r) {
      const float v = __ldcs(col + static_cast<int64_t>(r) * ld);
      if (isfinite(v)) { s += static_cast<double>(v); a += static_cast<double>(fabsf(v)); }
      else bad += 1.0;
    }
    if (ring != nullptr) {
      const float *rc = ring + c;
      for (int q = 0; q < ring_rows; ++q) {
        const float v = __ldcs(rc + static_cast<int64_t>(q) * ld);
        if (isfinite(v)) { s += static_cast<double>(v); a += static_cast<double>(fabsf(v)); }
        else bad += 1.0;
      }
    }
    total += s;
    if (out != nullptr) out[c] = s;
    if (ref != nullptr) {
      const double want = ref[c];
      const double drift = fabs(s - want);
      const double scale = fmax(a, fabs(want));
      max_drift = fmax(max_drift, drift);
      if (drift > 0.0) max_rel = fmax(max_rel, scale > 0.0 ? drift / scale : 1.0);
    }
  }
  total = warp_sum(total);
  bad = warp_sum(bad);
  max_drift = warp_max(max_drift);
  max_rel = warp_max(max_rel);
  if ((threadIdx.x & 31) == 0) {
    atomicAdd(stats + kStatTotal, total);
    if (bad != 0.0) atomicAdd(stats + kStatNonFinite, bad);
    if (max_drift > 0.0) atomic_max_nonneg(stats + kStatMaxDrift, max_drift);
    if (max_rel > 0.0) atomic_max_nonneg(stats + kStatMaxRelDrift, max_rel);
  }
}

// Debug pre-pass of a checked step: expect[c] = sum_i h_ic + sum over every ring slot, where h = x^(k+1/2) is
// recomputed from X, G and the optimiser state exactly as the step will (nothing is written back).  By
// column-stochasticity this is what sum_i X'[i, c] plus the ring must be after the step (Sec. 2; delay model).
template <int UPD>
__global__ void __launch_bounds__(256) sgp_expected_colsum_kernel(const float *__restrict__ X, const float *__restrict__ G,
                                                                   const float *__restrict__ M, const float *__restrict__ V,
                                                                   int n, int64_t d, int64_t ld, UpdateScalars us,
                                                                   const float *__restrict__ ring, int ring_rows,
                                                                   double *__restrict__ expect) {
  for (int64_t c = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; c < d;
       c += static_cast<int64_t>(gridDim.x) * blockDim.x) {
    double s = 0.0;
    for (int r = 0; r < n; ++r) {
      const int64_t o = static_cast<int64_t>(r) * ld + c;
      float u = UpdTraits<UPD>::kHasM ? M[o] : 0.f;
      float v = UpdTraits<UPD>::kHasV ? V[o] : 0.f;
      s += static_cast<double>(local_update<UPD, float>(X[o], G[o], u, v, us));
    }
    if (ring != nullptr)
      for (int q = 0; q < ring_rows; ++q) s += static_cast<double>(ring[static_cast<int64_t>(q) * ld + c]);
    expect[c] = s;
  }
}

// stats[kStatSumW] = sum_i W_i (+ ring weights); stats[kStatMinW] = min_i W_i (NaN counts as -1) (single CTA).
__global__ void __launch_bounds__(256) sgp_weight_scan_kernel(const float *__restrict__ W, int n,
                                                               const float *__restrict__ ring_w, int ring_len,
                                                               double *stats) {
  __shared__ double s_sum[8];
  __shared__ float s_min[8];
  double s = 0.0;
  float mn = 3.4e38f;
  for (int i = threadIdx.x; i < n; i += blockDim.x) {
    const float w = W[i];
    s += static_cast<double>(w);
    mn = fminf(mn, w == w ? w : -1.0f);
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
    stats[kStatSumW] = t;
    stats[kStatMinW] = static_cast<double>(m);
  }
}

// Turns the statistics into bits of the device status word (one thread).  check_weights: the weight statistics
// were gathered in this pass; check_columns: a column-sum reference was compared.
// sum_before (may be null): the weight sum taken just before the step.  One step of column-stochastic mixing keeps
// the sum to a few roundings (1e-5 n is forty times what n = 256 weights can lose in one step, and a single lost
// message is a hundred times more), whereas against n itself the fp32 sum has walked 1e-4 n away after ~1e4 steps.
__global__ void sgp_check_finalize_kernel(const double *stats, int n, int check_weights, int check_columns,
                                          double rel_tol, unsigned *status, const double *sum_before) {
  unsigned bits = 0;
  if (stats[kStatNonFinite] > 0.0) bits |= kStatusNonFinite;
  if (check_weights) {
    if (!(stats[kStatMinW] > 0.0)) bits |= kStatusZeroWeight;
    const double want = sum_before != nullptr ? *sum_before : static_cast<double>(n);
    const double tol = (sum_before != nullptr ? 1e-5 : 1e-4) * static_cast<double>(n);
    if (!(fabs(stats[kStatSumW] - want) <= tol)) bits |= kStatusWeightSum;
  }
  if (check_columns && !(stats[kStatMaxRelDrift] <= rel_tol)) bits |= kStatusColumnSum;
  if (bits) atomicOr(status, bits);
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
