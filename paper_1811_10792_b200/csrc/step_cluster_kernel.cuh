// Fused SGP step for many nodes (n > 128): a thread-block CLUSTER of 2 or 4 CTAs owns a column tile together.
//
// The mix of Alg. 1 line 6 needs x^(k+1/2) of every in-neighbour for the tile's columns, so all n rows of the tile
// must sit in shared memory at once.  With one CTA that caps the row segments at 256 bytes for n = 256, and short
// segments are what keeps HBM below its streaming rate.  Here every CTA of the cluster holds a slice of the rows
// (rows_per_cta = a power of two >= n / cluster size) at FOUR times the tile width, and the gather reads
// neighbour rows out of the sibling CTAs' shared memory (distributed shared memory, plain ld through
// map_shared_rank).  Two cluster barriers per tile: after the half steps are written, and
// before the tile is overwritten.  Nothing else differs from the register-staged kernel: same local update, same
// CSR order, same FMA chain, bit-identical results.
#pragma once
#include <cooperative_groups.h>

#include "step_common.cuh"

namespace sgp {

__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }

struct ClusterGeometry {
  int log2_rows_per_cta;   // rows of the tile one CTA holds
  int cluster_size;        // CTAs per cluster (2 or 4)
};

template <int UPD, bool HAS_Z, bool HAS_RING>
__global__ void __launch_bounds__(kThreads, 2)
sgp_step_cluster_kernel(const __grid_constant__ StepParams p, const __grid_constant__ ConstTable ct,
                        const __grid_constant__ ClusterGeometry geo) {
  using V = float4;
  constexpr int VEC = 4;
  constexpr bool HAS_M = UpdTraits<UPD>::kHasM;
  constexpr bool HAS_V = UpdTraits<UPD>::kHasV;
  constexpr int kItemsPerThread = UpdTraits<UPD>::kItems;
  namespace cg = cooperative_groups;
  cg::cluster_group cluster = cg::this_cluster();
  extern __shared__ __align__(128) unsigned char smem_raw[];
  const int n = p.n;
  const int tv = 1 << p.log2_tile_vecs;
  const int rows_per_cta = 1 << geo.log2_rows_per_cta;
  const int cta_rank = static_cast<int>(cluster.block_rank());
  const int row0 = cta_rank << geo.log2_rows_per_cta;                  // first row this CTA holds
  const int my_rows = max(0, min(rows_per_cta, n - row0));
  const int tile_items = my_rows * tv;
  V *H = reinterpret_cast<V *>(smem_raw);                              // rows_per_cta x tv vectors
  float *scratch = reinterpret_cast<float *>(H + static_cast<size_t>(rows_per_cta) * tv);
  const CtaTables tab = cta_prologue<HAS_RING>(p, ct, scratch, kThreads);

  const int64_t ld = p.ld;
  const int64_t ncols = p.col_end - p.col_begin;
  const int64_t tile_cols = static_cast<int64_t>(tv) * VEC;
  const int64_t ntiles = (ncols + tile_cols - 1) / tile_cols;
  const int64_t cluster_id = blockIdx.x / geo.cluster_size;
  const int64_t num_clusters = gridDim.x / geo.cluster_size;
  const int batches = max(1, (tile_items + kThreads * kItemsPerThread - 1) / (kThreads * kItemsPerThread));
  const int q_max = ((tile_items + batches - 1) / batches + kThreads - 1) / kThreads;
  const int batch_items = max(1, q_max * kThreads);

  for (int64_t tile = cluster_id; tile < ntiles; tile += num_clusters) {
    const int64_t col0 = p.col_begin + tile * tile_cols;
    // ---- phase 1: local update of this CTA's rows
    for (int base = 0; base < tile_items; base += batch_items) {
      V x[kItemsPerThread], g[kItemsPerThread], u[kItemsPerThread], vv[kItemsPerThread];
      bool ok[kItemsPerThread];
      int64_t off[kItemsPerThread];
#pragma unroll
      for (int q = 0; q < kItemsPerThread; ++q) {
        const int item = base + q * kThreads + threadIdx.x;
        const int row = row0 + (item >> p.log2_tile_vecs);
        const int c = item & (tv - 1);
        const int64_t col = col0 + static_cast<int64_t>(c) * VEC;
        ok[q] = (q < q_max) && (item < tile_items) && (col < p.col_end);
        off[q] = static_cast<int64_t>(row) * ld + col;
        if (ok[q]) ok[q] = SGP_BOUNDS_OK(p, row < n && col >= 0 && col + VEC <= ld);
      }
#pragma unroll
      for (int q = 0; q < kItemsPerThread; ++q) {
        if (ok[q]) {
          x[q] = ld_inplace(reinterpret_cast<const V *>(p.X + off[q]));
          g[q] = ld_stream(reinterpret_cast<const V *>(p.G + off[q]));
          if (HAS_M) u[q] = ld_inplace(reinterpret_cast<const V *>(p.M + off[q]));
          if (HAS_V) vv[q] = ld_inplace(reinterpret_cast<const V *>(p.V + off[q]));
        }
      }
#pragma unroll
      for (int q = 0; q < kItemsPerThread; ++q) {
        const int item = base + q * kThreads + threadIdx.x;
        if (ok[q]) {
          const V h = local_update<UPD, V>(x[q], g[q], u[q], vv[q], p);
          if (HAS_M) st_stream(reinterpret_cast<V *>(p.M + off[q]), u[q]);
          if (HAS_V) st_stream(reinterpret_cast<V *>(p.V + off[q]), vv[q]);
          H[item] = h;
        } else if (q < q_max && item < tile_items) {
          H[item] = vzero<V>();
        }
      }
    }
    cluster_arrive();          // every CTA's slice of the half steps is written ...
    cluster_wait();            // ... and visible to its siblings
    // ---- phase 2: gather-mix; neighbour rows come from whichever CTA of the cluster holds them
    for (int base = 0; base < tile_items; base += batch_items) {
      V ring_in[kItemsPerThread];
      if (HAS_RING) {
#pragma unroll
        for (int q = 0; q < kItemsPerThread; ++q) {
          const int item = base + q * kThreads + threadIdx.x;
          const int row = row0 + (item >> p.log2_tile_vecs);
          const int c = item & (tv - 1);
          const int64_t col = col0 + static_cast<int64_t>(c) * VEC;
          if (q < q_max && item < tile_items && col < p.col_end)
            ring_in[q] = ld_inplace(reinterpret_cast<const V *>(p.ring_x + static_cast<int64_t>(row) * ld + col));
        }
      }
#pragma unroll
      for (int q = 0; q < kItemsPerThread; ++q) {
        const int item = base + q * kThreads + threadIdx.x;
        const int row = row0 + (item >> p.log2_tile_vecs);
        const int c = item & (tv - 1);
        const int64_t col = col0 + static_cast<int64_t>(c) * VEC;
        if (q < q_max && item < tile_items && col < p.col_end) {
          const int64_t o = static_cast<int64_t>(row) * ld + col;
          V acc = vzero<V>(), offd = vzero<V>();
          const int e1 = tab.rowptr[row + 1];
          for (int e = tab.rowptr[row]; e < e1; ++e) {
            const int j = tab.col[e];
            if (!SGP_BOUNDS_OK(p, j >= 0 && j < n)) continue;
            const float pv = tab.val[e];
            const V *Hj = cluster.map_shared_rank(H, static_cast<unsigned>(j >> geo.log2_rows_per_cta));   // the sibling that holds row j
            const V hj = Hj[((j & (rows_per_cta - 1)) << p.log2_tile_vecs) + c];
            if (HAS_RING && j != row) offd = vfma(pv, hj, offd);
            else acc = vfma(pv, hj, acc);
          }
          if (HAS_RING) {
            acc = vadd(acc, ring_in[q]);
            st_stream(reinterpret_cast<V *>(p.ring_x + o), offd);
          }
          st_stream(reinterpret_cast<V *>(p.X + o), acc);
          if (HAS_Z) st_stream(reinterpret_cast<V *>(p.Z + o), vmul(tab.inv_w[row], acc));
        }
      }
    }
    cluster_arrive();          // this CTA is done reading its siblings' tiles ...
    cluster_wait();            // ... and nobody still reads this CTA's: the tile may be overwritten (or the CTA may exit)
  }
}

using ClusterKernel = void (*)(const StepParams, const ConstTable, const ClusterGeometry);
ClusterKernel cluster_kernel(int upd, bool has_z, bool has_ring);

}  // namespace sgp
