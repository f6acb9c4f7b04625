// Fused SGP step for rows that do NOT start on 16-byte boundaries (a dense pitch ld = d with d not a multiple of 4, or
// arrays that are all offset by the same odd number of floats): the register-staged scheme of step_regs_kernel.cuh
// with per-row PEELING.  A CTA still owns all n rows of a tile of columns [col0, col0 + T) -- ownership is not shifted,
// so nothing a neighbouring CTA rewrites in place is ever read -- but inside the tile every row is cut at ITS OWN
// 16-byte boundaries: up to three head elements, then aligned 128-bit vectors, then up to three tail elements.  Head
// and tail travel as masked "partial vectors" (scalar loads and stores of the elements the tile owns), everything else
// as 128-bit accesses.  The half steps x^(k+1/2) go to a shared tile in column order (row pitch T + 8, each row
// shifted so that its vectors land 16-byte aligned); the gather reads a sender's values with two aligned 128-bit reads
// and a select, because a sender's row is cut at other columns than the receiver's.  Same local update, same CSR order, same fp32
// FMA chain per element as the other step kernels: bit-identical results (Alg. 1 lines 4-8, Alg. 3 lines 4-5, Alg. 2).
#pragma once
#include "step_common.cuh"

namespace sgp {

constexpr int kPeelItems = 4;       // (row, vector slot) items a thread keeps in flight
constexpr int kPeelRowPad = 8;      // floats of slack per row of the shared tile (shift of up to 3 plus a partial vector)
constexpr int kPeelTilePad = 16;    // floats of slack after the last row (masked-out lanes of the gather may read there)

__device__ __forceinline__ float4 peel_load(const float *ptr, unsigned mask, bool streaming) {
  if (mask == 0xFu) {
    return streaming ? __ldcs(reinterpret_cast<const float4 *>(ptr)) : __ldcg(reinterpret_cast<const float4 *>(ptr));
  }
  float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
  if (mask & 1u) v.x = streaming ? __ldcs(ptr + 0) : __ldcg(ptr + 0);
  if (mask & 2u) v.y = streaming ? __ldcs(ptr + 1) : __ldcg(ptr + 1);
  if (mask & 4u) v.z = streaming ? __ldcs(ptr + 2) : __ldcg(ptr + 2);
  if (mask & 8u) v.w = streaming ? __ldcs(ptr + 3) : __ldcg(ptr + 3);
  return v;
}

__device__ __forceinline__ void peel_store(float *ptr, float4 v, unsigned mask) {
  if (mask == 0xFu) {
    __stcs(reinterpret_cast<float4 *>(ptr), v);
    return;
  }
  if (mask & 1u) __stcs(ptr + 0, v.x);
  if (mask & 2u) __stcs(ptr + 1, v.y);
  if (mask & 4u) __stcs(ptr + 2, v.z);
  if (mask & 8u) __stcs(ptr + 3, v.w);
}

// One (row, slot) item of a tile.  Slot k of a row whose first owned element sits `phase` floats after a 16-byte
// boundary covers the columns rel0 .. rel0 + 3 relative to the tile, rel0 = 4 k - phase: with phase > 0 slot 0 is the
// partial head (its first `phase` elements belong to the previous tile) and slot tv the partial tail.
struct PeelItem {
  int row;
  int rel0;        // first column of the vector relative to the tile's first column (-3 .. T - 1)
  unsigned mask;   // which of its four elements the tile owns
};

// Floats between the last 16-byte boundary and the row's first element of a tile (the same for every tile and array).
__device__ __forceinline__ int peel_phase(const StepParams &p, int row) {
  return (p.peel_phase0 + row * p.peel_phase_step) & 3;
}

__device__ __forceinline__ PeelItem peel_item(const StepParams &p, int item, int tile_items, int tv, int valid_cols) {
  PeelItem it;
  int k;
  if (item < tile_items) {
    it.row = item >> p.log2_tile_vecs;
    k = item & (tv - 1);
  } else {
    it.row = item - tile_items;          // the extra slot of every row: its partial tail
    k = tv;
  }
  it.rel0 = 4 * k - peel_phase(p, it.row);
  const int lo = max(0, -it.rel0);
  const int hi = min(4, valid_cols - it.rel0);
  it.mask = (it.row < p.n && hi > lo) ? ((0xFu << lo) & (0xFu >> (4 - hi))) : 0u;
  return it;
}

// Index of column `rel` of `row` in the shared tile: rows are shifted so that rel0 of every slot is a multiple of 4.
__device__ __forceinline__ int peel_smem_index(const StepParams &p, int row, int pitch, int rel) {
  return row * pitch + 4 + peel_phase(p, row) + rel;
}

template <int UPD, bool HAS_Z, bool HAS_RING>
__global__ void __launch_bounds__(kThreads, 2)
sgp_step_peel_kernel(const __grid_constant__ StepParams p, const __grid_constant__ ConstTable ct) {
  constexpr bool HAS_M = UpdTraits<UPD>::kHasM;
  constexpr bool HAS_V = UpdTraits<UPD>::kHasV;
  extern __shared__ __align__(128) unsigned char smem_raw[];
  const int n = p.n;
  const int tv = 1 << p.log2_tile_vecs;
  const int tile_cols = tv * 4;
  const int pitch = tile_cols + kPeelRowPad;
  const int tile_floats = n * pitch + kPeelTilePad;
  float *H0 = reinterpret_cast<float *>(smem_raw);
  float *H1 = p.single_buffer ? H0 : H0 + tile_floats;
  float *scratch = H0 + (p.single_buffer ? 1 : 2) * tile_floats;
  const CtaTables tab = cta_prologue<HAS_RING>(p, ct, scratch, kThreads);

  const int64_t ld = p.ld;
  const int64_t ncols = p.col_end - p.col_begin;
  const int64_t ntiles = (ncols + tile_cols - 1) / tile_cols;
  const int tile_items = n * tv;
  const int total_items = tile_items + n;                 // one extra (tail) slot per row
  int buf = 0;

  for (int64_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
    const int64_t col0 = p.col_begin + tile * tile_cols;
    const int valid_cols = static_cast<int>(min(static_cast<int64_t>(tile_cols), p.col_end - col0));
    float *H = buf ? H1 : H0;
    // ---- phase 1: local update; half steps into the shared tile
    for (int base = 0; base < total_items; base += kThreads * kPeelItems) {
      PeelItem it[kPeelItems];
      float4 x[kPeelItems], g[kPeelItems], u[kPeelItems], vv[kPeelItems];
      int64_t off[kPeelItems];
#pragma unroll
      for (int q = 0; q < kPeelItems; ++q) {
        const int item = base + q * kThreads + threadIdx.x;
        it[q] = peel_item(p, min(item, total_items - 1), tile_items, tv, valid_cols);
        if (item >= total_items) it[q].mask = 0u;
        off[q] = static_cast<int64_t>(it[q].row) * ld + col0 + it[q].rel0;
        if (it[q].mask && !SGP_BOUNDS_OK(p, it[q].row < n && col0 + it[q].rel0 + 4 > 0 && col0 + it[q].rel0 < ld)) it[q].mask = 0u;
      }
#pragma unroll
      for (int q = 0; q < kPeelItems; ++q) {
        if (it[q].mask) {
          x[q] = peel_load(p.X + off[q], it[q].mask, false);
          g[q] = peel_load(p.G + off[q], it[q].mask, true);
          if (HAS_M) u[q] = peel_load(p.M + off[q], it[q].mask, false);
          if (HAS_V) vv[q] = peel_load(p.V + off[q], it[q].mask, false);
        }
      }
#pragma unroll
      for (int q = 0; q < kPeelItems; ++q) {
        if (it[q].mask) {
          const float4 h = local_update<UPD, float4>(x[q], g[q], u[q], vv[q], p);
          if (HAS_M) peel_store(p.M + off[q], u[q], it[q].mask);
          if (HAS_V) peel_store(p.V + off[q], vv[q], it[q].mask);
          // masked-out lanes carry zeros: they land in the row's slack and are never read for an owned element
          *reinterpret_cast<float4 *>(H + peel_smem_index(p, it[q].row, pitch, it[q].rel0)) = h;
        }
      }
    }
    __syncthreads();
    // ---- phase 2: gather-mix over the step's in-neighbour lists, ring exchange, de-bias
    for (int base = 0; base < total_items; base += kThreads * kPeelItems) {
      PeelItem me[kPeelItems];
      float4 ring[kPeelItems];
#pragma unroll
      for (int q = 0; q < kPeelItems; ++q) {
        const int item = base + q * kThreads + threadIdx.x;
        me[q] = peel_item(p, min(item, total_items - 1), tile_items, tv, valid_cols);
        if (item >= total_items) me[q].mask = 0u;
        if (HAS_RING && me[q].mask)
          ring[q] = peel_load(p.ring_x + static_cast<int64_t>(me[q].row) * ld + col0 + me[q].rel0, me[q].mask, false);
      }
#pragma unroll
      for (int q = 0; q < kPeelItems; ++q) {
        if (!me[q].mask) continue;
        const int64_t o = static_cast<int64_t>(me[q].row) * ld + col0 + me[q].rel0;
        // my slot sits 16-byte aligned in my row of the tile; in a sender's row the same columns start `s` floats
        // after a 16-byte boundary, s = difference of the two rows' shifts: two aligned reads and a select
        const int my_shift = peel_phase(p, me[q].row);
        const int my_index = 4 + my_shift + me[q].rel0;                 // a multiple of 4
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f), offd = make_float4(0.f, 0.f, 0.f, 0.f);
        const int e1 = tab.rowptr[me[q].row + 1];
        for (int e = tab.rowptr[me[q].row]; e < e1; ++e) {
          const int j = tab.col[e];
          if (!SGP_BOUNDS_OK(p, j >= 0 && j < n)) continue;
          const float pv = tab.val[e];
          const int delta = peel_phase(p, j) - my_shift;                  // -3 .. 3
          const int s = delta & 3;
          const float4 *src = reinterpret_cast<const float4 *>(H + j * pitch + my_index + (delta < 0 ? -4 : 0));
          const float4 lo4 = src[0];
          float4 h4 = lo4;
          if (s != 0) {
            const float4 hi4 = src[1];
            h4 = s == 1 ? make_float4(lo4.y, lo4.z, lo4.w, hi4.x)
                        : (s == 2 ? make_float4(lo4.z, lo4.w, hi4.x, hi4.y) : make_float4(lo4.w, hi4.x, hi4.y, hi4.z));
          }
          if (HAS_RING && j != me[q].row) offd = vfma(pv, h4, offd);
          else acc = vfma(pv, h4, acc);
        }
        if (HAS_RING) {
          acc = vadd(acc, ring[q]);
          peel_store(p.ring_x + o, offd, me[q].mask);
        }
        peel_store(p.X + o, acc, me[q].mask);
        if (HAS_Z) peel_store(p.Z + o, vmul(tab.inv_w[me[q].row], acc), me[q].mask);
      }
    }
    buf ^= 1;
    if (p.single_buffer) __syncthreads();   // the only tile is about to be overwritten
  }
}

using PeelKernel = void (*)(const StepParams, const ConstTable);
PeelKernel peel_kernel(int upd, bool has_z, bool has_ring);

}  // namespace sgp
