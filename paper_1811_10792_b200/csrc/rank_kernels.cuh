// One node per GPU (the paper's own setting, App. C): the SGP iteration split at the point where data must cross
// between nodes.  A node's step is
//     update   h_i = x_i - lr * s_i                     (Alg. 1 line 4 / Alg. 3 lines 4-5), published UNWEIGHTED in a
//              message slot in this GPU's memory together with w_i                  (Alg. 1 line 5: the "send")
//     mix      x_i' = sum_j p_ij h_j ,  w_i' = sum_j p_ij w_j ,  z_i = x_i' / w_i'  (Alg. 1 lines 6-8)
// where the mix reads the in-neighbours' slots straight out of THEIR GPU's memory with plain 128-bit loads over
// NVLink (peer pointers; no staging copy, no landing buffer, every reader issues its own loads): the pull and the mix are one kernel.
// With a delay tau >= 1 (Alg. 2) the messages consumed at step k were published at step k - tau, so nothing the
// kernel reads is still being written and update + pull + mix fuse into ONE kernel per step.
//
// Receiver-side weights: p_ij is applied by the receiver, so every out-neighbour reads the same unweighted slot.
// Summation order is the compiled schedule's CSR order (ascending sender, fp32 FMA chain), exactly as in the
// all-nodes-on-one-GPU kernels: results are bit-identical to those.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "step_common.cuh"

namespace sgp {

constexpr int kMaxRankPeers = 32;     // in-neighbours (self included) one mix can take
constexpr int kRankThreads = 256;

// The sources of one mix in CSR order.  src[e] points at a message slot (a row of ld floats followed, at
// [w_offset], by the sender's weight): the sender's own GPU memory for e != self_pos, this GPU's for e == self_pos.
struct RankSources {
  const float *src[kMaxRankPeers];
  float weight[kMaxRankPeers];
  int count;
  int self_pos;      // entry that is this node itself; -1 when the list holds only (delayed) peers
};

struct RankParams {
  float *x;          // numerator row (d floats)
  float *w;          // push-sum weight (1 float, device)
  float *m;          // momentum / Adam first moment row or null
  float *v;          // Adam second moment row or null
  const float *g;    // gradient row
  float *z;          // de-biased row or null
  float *msg;        // this node's message slot for this step (written by update / the fused kernel)
  int64_t d;
  int64_t w_offset;  // index of the weight inside a slot
  float self_weight; // p_ii of this step (fused kernel)
  int biased;
  UpdateScalars us;
  unsigned *ticket;  // last-CTA-commits protocol for w in the fused kernel
  unsigned *status;
};

// h = local update; publishes (h, w) in the message slot; momentum written back.  x is left alone: the mix
// overwrites it.
template <int VEC, int UPD>
__global__ void __launch_bounds__(kRankThreads) sgp_rank_update_kernel(const __grid_constant__ RankParams p) {
  using V = typename VecT<VEC>::type;
  constexpr bool HAS_M = UpdTraits<UPD>::kHasM;
  constexpr bool HAS_V = UpdTraits<UPD>::kHasV;
  if (blockIdx.x == 0 && threadIdx.x == 0) p.msg[p.w_offset] = *p.w;
  const int64_t nvec = VEC == 4 ? (p.d >> 2) : p.d;
  const int64_t stride = static_cast<int64_t>(gridDim.x) * kRankThreads;
  for (int64_t i = static_cast<int64_t>(blockIdx.x) * kRankThreads + threadIdx.x; i < nvec; i += stride) {
    V u = HAS_M ? ld_inplace(reinterpret_cast<const V *>(p.m) + i) : vzero<V>();
    V v2 = HAS_V ? ld_inplace(reinterpret_cast<const V *>(p.v) + i) : vzero<V>();
    const V h = local_update<UPD, V>(ld_stream(reinterpret_cast<const V *>(p.x) + i), ld_stream(reinterpret_cast<const V *>(p.g) + i), u, v2, p.us);
    if (HAS_M) st_stream(reinterpret_cast<V *>(p.m) + i, u);
    if (HAS_V) st_stream(reinterpret_cast<V *>(p.v) + i, v2);
    reinterpret_cast<V *>(p.msg)[i] = h;        // default policy: the out-neighbours (and this node's own mix) read it next
  }
  if (VEC == 4 && blockIdx.x == 0) {            // ragged end of the row
    const int64_t c = (nvec << 2) + threadIdx.x;
    if (c < p.d) {
      float u = HAS_M ? p.m[c] : 0.f, v2 = HAS_V ? p.v[c] : 0.f;
      const float h = local_update<UPD, float>(p.x[c], p.g[c], u, v2, p.us);
      if (HAS_M) p.m[c] = u;
      if (HAS_V) p.v[c] = v2;
      p.msg[c] = h;
    }
  }
}

// w' = sum_e weight[e] * (weight published in source e), in list order.
__device__ __forceinline__ float rank_mix_weight(const RankSources &s, int64_t w_offset) {
  float acc = 0.f;
  for (int e = 0; e < s.count; ++e) acc = fmaf(s.weight[e], __ldcg(s.src[e] + w_offset), acc);
  return acc;
}

template <typename V>
__device__ __forceinline__ V rank_gather(const RankSources &s, int64_t i) {
  V acc = vzero<V>();
  for (int e = 0; e < s.count; ++e) acc = vfma(s.weight[e], ld_stream(reinterpret_cast<const V *>(s.src[e]) + i), acc);
  return acc;
}

// Pull + mix + de-bias (tau = 0): x' = sum over the sources (self included, CSR order), z = x' / w'.
template <int VEC, bool HAS_Z>
__global__ void __launch_bounds__(kRankThreads) sgp_rank_mix_kernel(const __grid_constant__ RankParams p,
                                                                     const __grid_constant__ RankSources s) {
  using V = typename VecT<VEC>::type;
  const float w_new = rank_mix_weight(s, p.w_offset);
  const float inv = p.biased ? 1.0f : (w_new > 0.0f ? 1.0f / w_new : 0.0f);
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    if (!(w_new > 0.0f)) atomicOr(p.status, kStatusZeroWeight);
    *p.w = w_new;          // nobody reads *p.w in this launch: the old weight travels in the message slot
  }
  const int64_t nvec = VEC == 4 ? (p.d >> 2) : p.d;
  const int64_t stride = static_cast<int64_t>(gridDim.x) * kRankThreads;
  for (int64_t i = static_cast<int64_t>(blockIdx.x) * kRankThreads + threadIdx.x; i < nvec; i += stride) {
    const V acc = rank_gather<V>(s, i);
    st_stream(reinterpret_cast<V *>(p.x) + i, acc);
    if (HAS_Z) st_stream(reinterpret_cast<V *>(p.z) + i, vmul(inv, acc));
  }
  if (VEC == 4 && blockIdx.x == 0) {
    const int64_t c = (nvec << 2) + threadIdx.x;
    if (c < p.d) {
      const float acc = rank_gather<float>(s, c);
      p.x[c] = acc;
      if (HAS_Z) p.z[c] = inv * acc;
    }
  }
}

// Overlap SGP (tau >= 1), ONE kernel per step: update, publish (h, w) for the out-neighbours to read tau steps
// from now, and mix with what the in-neighbours published tau steps ago (their slots are complete: no wait):
//     x' = p_ii h + sum_{j != i} p_ij^(k-tau) h_j^(k-tau)      (Alg. 2 lines 7, 21; delay model)
template <int VEC, int UPD, bool HAS_Z>
__global__ void __launch_bounds__(kRankThreads) sgp_rank_overlap_kernel(const __grid_constant__ RankParams p,
                                                                         const __grid_constant__ RankSources s) {
  using V = typename VecT<VEC>::type;
  constexpr bool HAS_M = UpdTraits<UPD>::kHasM;
  constexpr bool HAS_V = UpdTraits<UPD>::kHasV;
  __shared__ float s_inv;
  if (threadIdx.x == 0) {
    const float w_old = __ldcg(p.w);
    const float w_new = fmaf(p.self_weight, w_old, 0.f) + rank_mix_weight(s, p.w_offset);
    s_inv = p.biased ? 1.0f : (w_new > 0.0f ? 1.0f / w_new : 0.0f);
    // every CTA takes a ticket after its read of the old weight; the last one commits the new weight
    __threadfence();
    const unsigned ticket = atomicAdd(p.ticket, 1u);
    if (ticket == gridDim.x - 1) {
      if (!(w_new > 0.0f)) atomicOr(p.status, kStatusZeroWeight);
      p.msg[p.w_offset] = w_old;
      *p.w = w_new;
      *p.ticket = 0u;
    }
  }
  __syncthreads();
  const float inv = s_inv;
  const int64_t nvec = VEC == 4 ? (p.d >> 2) : p.d;
  const int64_t stride = static_cast<int64_t>(gridDim.x) * kRankThreads;
  for (int64_t i = static_cast<int64_t>(blockIdx.x) * kRankThreads + threadIdx.x; i < nvec; i += stride) {
    V u = HAS_M ? ld_inplace(reinterpret_cast<const V *>(p.m) + i) : vzero<V>();
    V v2 = HAS_V ? ld_inplace(reinterpret_cast<const V *>(p.v) + i) : vzero<V>();
    const V h = local_update<UPD, V>(ld_inplace(reinterpret_cast<const V *>(p.x) + i), ld_stream(reinterpret_cast<const V *>(p.g) + i), u, v2, p.us);
    const V late = rank_gather<V>(s, i);
    if (HAS_M) st_stream(reinterpret_cast<V *>(p.m) + i, u);
    if (HAS_V) st_stream(reinterpret_cast<V *>(p.v) + i, v2);
    reinterpret_cast<V *>(p.msg)[i] = h;
    const V acc = vadd(vfma(p.self_weight, h, vzero<V>()), late);
    st_stream(reinterpret_cast<V *>(p.x) + i, acc);
    if (HAS_Z) st_stream(reinterpret_cast<V *>(p.z) + i, vmul(inv, acc));
  }
  if (VEC == 4 && blockIdx.x == 0) {
    const int64_t c = (nvec << 2) + threadIdx.x;
    if (c < p.d) {
      float u = HAS_M ? p.m[c] : 0.f, v2 = HAS_V ? p.v[c] : 0.f;
      const float h = local_update<UPD, float>(p.x[c], p.g[c], u, v2, p.us);
      const float late = rank_gather<float>(s, c);
      if (HAS_M) p.m[c] = u;
      if (HAS_V) p.v[c] = v2;
      p.msg[c] = h;
      const float acc = fmaf(p.self_weight, h, 0.f) + late;
      p.x[c] = acc;
      if (HAS_Z) p.z[c] = inv * acc;
    }
  }
}

}  // namespace sgp
