// Bulk-copy (TMA) pipelined fused SGP step kernel for sm_100a (Alg. 1 lines 4-8 with the update of Alg. 3,
// Alg. 2 with the delayed-message ring).
#pragma once
#include "step_common.cuh"

namespace sgp {

// ------------------------------------------------------------------------------------------------
// Bulk-copy (TMA) pipelined kernel.  A producer warp streams whole column tiles -- every node's row
// segment of X, G (and M, ring) -- into a ring of shared-memory stages with cp.async.bulk, completion
// counted on an mbarrier per stage; eight consumer warps update, exchange through the stage itself
// (x^(k+1/2) overwrites the X tile in place), gather-mix and store with 128-bit streaming stores.
// Loads therefore stay in flight while the consumers compute and store.  Every CTA fetches its own tiles; no cluster.
// Every wait is bounded: on expiry the CTA records a status bit and leaves.
// ------------------------------------------------------------------------------------------------
constexpr int kTmaConsumers = 256;
constexpr int kTmaThreads = kTmaConsumers + 32;

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t *bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ uint64_t global_timer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// Waits for the phase with the given parity; gives up after limit_ns (wall clock of the device).
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t *bar, uint32_t parity, uint64_t limit_ns) {
  if (mbar_try_wait(bar, parity)) return true;
  const uint64_t t0 = global_timer_ns();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 256; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (global_timer_ns() - t0 > limit_ns) return false;
  }
}
// One contiguous global -> shared copy of `bytes` (multiple of 16, both addresses 16-byte aligned).
__device__ __forceinline__ void bulk_copy_g2s(void *dst_smem, const void *src_gmem, uint32_t bytes, uint64_t *bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_u32(dst_smem)),
               "l"(__cvta_generic_to_global(src_gmem)), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}
// Tiled 2-D tensor copy global -> shared: box of (tile columns x all n rows) at column x, row y.
__device__ __forceinline__ void tma_load_2d(void *dst_smem, const CUtensorMap *map, int x, int y, uint64_t *bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(
          smem_u32(dst_smem)),
      "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(smem_u32(bar))
      : "memory");
}
// Tensor maps of the arrays a launch streams in (only those the launch uses are encoded).
struct alignas(64) TmaMaps {
  CUtensorMap x, g, m, v, r;
};
__device__ __forceinline__ uint64_t l2_evict_first_policy() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ void bulk_copy_g2s_hint(void *dst_smem, const void *src_gmem, uint32_t bytes, uint64_t *bar,
                                                   uint64_t policy) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(
          smem_u32(dst_smem)),
      "l"(__cvta_generic_to_global(src_gmem)), "r"(bytes), "r"(smem_u32(bar)), "l"(policy)
      : "memory");
}
__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void consumer_barrier() { asm volatile("bar.sync 1, %0;" ::"n"(kTmaConsumers) : "memory"); }
// Barrier over the consumer threads that also ANDs a flag, so that all of them take the same decision.
__device__ __forceinline__ bool consumer_all(bool flag) {
  uint32_t out;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.u32 q, %1, 0;\n\t"
      "bar.red.and.pred p, 1, %2, q;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(out)
      : "r"(static_cast<uint32_t>(flag)), "n"(kTmaConsumers)
      : "memory");
  return out != 0;
}

template <int UPD, bool HAS_Z, bool HAS_RING, bool DIAG>
__global__ void __launch_bounds__(kTmaThreads, 2)
sgp_step_tma_kernel(const __grid_constant__ StepParams p, const __grid_constant__ ConstTable ct,
                    const __grid_constant__ TmaMaps maps, const int stages, const int use_tensor_maps) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  constexpr bool HAS_M = UpdTraits<UPD>::kHasM;
  constexpr bool HAS_V = UpdTraits<UPD>::kHasV;
  // stage layout: [X][G][M if any][V if any][ring if any], each n x tile columns
  constexpr int kIdxM = 2, kIdxV = 2 + (HAS_M ? 1 : 0), kIdxR = kIdxV + (HAS_V ? 1 : 0);
  constexpr int kArrays = kIdxR + (HAS_RING ? 1 : 0);
  constexpr int kMaxStages = 8;
  const int n = p.n;
  const int tv = 1 << p.log2_tile_vecs;
  const int tile_items = n * tv;                       // float4 items per array per stage
  const size_t stage_bytes = static_cast<size_t>(kArrays) * tile_items * sizeof(float4);
  uint64_t *full_bar = reinterpret_cast<uint64_t *>(smem_raw + stages * stage_bytes);
  uint64_t *empty_bar = full_bar + kMaxStages;
  float4 *partial = reinterpret_cast<float4 *>(empty_bar + kMaxStages);   // uniform_parts x tv vectors
  float *scratch = reinterpret_cast<float *>(partial + p.uniform_parts * tv);
  __shared__ int s_abort;

  const CtaTables tab = cta_prologue<HAS_RING>(p, ct, scratch, kTmaThreads);
  // Fused diagnostics (a separate instantiation): scratch after the weights and, when it was copied, the table.
  constexpr int kDiagArrays = HAS_RING ? 2 : 1;
  DiagScratch<float4> ds{};
  if (DIAG) {
    unsigned char *after = reinterpret_cast<unsigned char *>(scratch + 3 * n) +
                           (p.table_mode < 2 ? (static_cast<size_t>(n) + 1 + 2 * static_cast<size_t>(p.nnz)) * 4 : 0);
    ds = diag_scratch<float4>(after, HAS_RING);
    for (int i = threadIdx.x; i < tile_items; i += kTmaThreads) ds.slots[i] = make_float2(0.f, 0.f);
  }
  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) {
      mbar_init(full_bar + s, 1);
      mbar_init(empty_bar + s, kTmaConsumers / 32);
    }
    s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  const int64_t ld = p.ld;
  const int64_t ncols = p.col_end - p.col_begin;
  const int64_t tile_cols = static_cast<int64_t>(tv) * 4;
  const int64_t ntiles = (ncols + tile_cols - 1) / tile_cols;
  const int64_t my_tiles = ntiles > blockIdx.x ? (ntiles - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile int *abort_flag = &s_abort;
  const uint64_t limit_ns = static_cast<uint64_t>(p.wait_limit_ms) * 1000000ull;

  if (warp == kTmaConsumers / 32) {
    // ---------------- producer warp
    int64_t issued = 0;
    const uint64_t policy = l2_evict_first_policy();
    for (int64_t it = 0; it < my_tiles && !*abort_flag; ++it) {
      const int s = static_cast<int>(it % stages);
      const int64_t round = it / stages;
      if (round > 0 && !mbar_wait_bounded(empty_bar + s, static_cast<uint32_t>((round - 1) & 1), limit_ns)) {
        if (lane == 0) atomicOr(p.status, kStatusEmptyTimeout);
        *abort_flag = 1;
        break;
      }
      if (p.inject_stall && blockIdx.x == 0 && it == 0) continue;   // test hook: this tile is never requested
      const int64_t tile = blockIdx.x + it * gridDim.x;
      const int64_t col0 = p.col_begin + tile * tile_cols;
      const int64_t valid = min(tile_cols, p.col_end - col0);
      const uint32_t seg_bytes = static_cast<uint32_t>(valid * 4);
      unsigned char *stage = smem_raw + s * stage_bytes;
      if (use_tensor_maps) {
        // one box per array: tile columns x n rows; columns past d are zero-filled by the copy engine
        if (lane == 0) {
          const size_t arr_bytes = static_cast<size_t>(tile_items) * sizeof(float4);
          mbar_arrive_expect_tx(full_bar + s, static_cast<uint32_t>(stage_bytes));
          tma_load_2d(stage, &maps.x, static_cast<int>(col0), 0, full_bar + s);
          tma_load_2d(stage + arr_bytes, &maps.g, static_cast<int>(col0), 0, full_bar + s);
          if (HAS_M) tma_load_2d(stage + kIdxM * arr_bytes, &maps.m, static_cast<int>(col0), 0, full_bar + s);
          if (HAS_V) tma_load_2d(stage + kIdxV * arr_bytes, &maps.v, static_cast<int>(col0), 0, full_bar + s);
          if (HAS_RING) tma_load_2d(stage + kIdxR * arr_bytes, &maps.r, static_cast<int>(col0), 0, full_bar + s);
        }
        issued = it + 1;
        continue;
      }
      if (lane == 0) mbar_arrive_expect_tx(full_bar + s, seg_bytes * static_cast<uint32_t>(n * kArrays));
      __syncwarp();
      for (int c = lane; c < n * kArrays; c += 32) {
        const int arr = c / n, row = c - arr * n;
        const float *src;
        if (arr == 0) src = p.X;
        else if (arr == 1) src = p.G;
        else if (HAS_M && arr == kIdxM) src = p.M;
        else if (HAS_V && arr == kIdxV) src = p.V;
        else src = p.ring_x;
        void *dst = stage + (static_cast<size_t>(arr) * tile_items + static_cast<size_t>(row) * tv) * sizeof(float4);
        if (p.l2_hint == 1 || (p.l2_hint == 3 && arr == 1) || (p.l2_hint == 4 && arr != 1))
          bulk_copy_g2s_hint(dst, src + static_cast<int64_t>(row) * ld + col0, seg_bytes, full_bar + s, policy);
        else bulk_copy_g2s(dst, src + static_cast<int64_t>(row) * ld + col0, seg_bytes, full_bar + s);
      }
      issued = it + 1;
    }
    // On an aborted run copies may still be in flight to this CTA's shared memory: wait for them (bounded).
    if (*abort_flag) {
      for (int64_t it = (issued > stages ? issued - stages : 0); it < issued; ++it) {
        if (p.inject_stall && blockIdx.x == 0 && it == 0) continue;   // was never requested
        const int s = static_cast<int>(it % stages);
        if (!mbar_wait_bounded(full_bar + s, static_cast<uint32_t>((it / stages) & 1), limit_ns) && lane == 0)
          atomicOr(p.status, kStatusDrainTimeout);
      }
    }
  } else {
    // ---------------- consumer warps
    const int ctid = threadIdx.x;
    for (int64_t it = 0; it < my_tiles; ++it) {
      const int s = static_cast<int>(it % stages);
      const int64_t round = it / stages;
      // bounded wait, then a vote: either every consumer goes on or every consumer leaves
      const bool arrived = !*abort_flag && mbar_wait_bounded(full_bar + s, static_cast<uint32_t>(round & 1), limit_ns);
      if (!consumer_all(arrived)) {
        if (ctid == 0) atomicOr(p.status, kStatusFullTimeout);
        *abort_flag = 1;
        break;
      }
      const int64_t tile = blockIdx.x + it * gridDim.x;
      const int64_t col0 = p.col_begin + tile * tile_cols;
      float4 *Xs = reinterpret_cast<float4 *>(smem_raw + s * stage_bytes);
      const float4 *Gs = Xs + tile_items;
      const float4 *Ms = Xs + static_cast<size_t>(kIdxM) * tile_items;
      const float4 *Vs = Xs + static_cast<size_t>(kIdxV) * tile_items;
      const float4 *Rs = Xs + static_cast<size_t>(kIdxR) * tile_items;
      // phase 1: local update; x^(k+1/2) replaces x in the stage
      float4 csum = make_float4(0.f, 0.f, 0.f, 0.f), rsum = csum;   // diagnostics: this thread's share of its column's sums
#pragma unroll 4
      for (int item = ctid; item < tile_items; item += kTmaConsumers) {
        const int row = item >> p.log2_tile_vecs;
        const int c = item & (tv - 1);
        const int64_t col = col0 + static_cast<int64_t>(c) * 4;
        if (col < p.col_end) {
          float4 u = HAS_M ? Ms[item] : make_float4(0.f, 0.f, 0.f, 0.f);
          float4 v2 = HAS_V ? Vs[item] : make_float4(0.f, 0.f, 0.f, 0.f);
          const float4 h = local_update<UPD, float4>(Xs[item], Gs[item], u, v2, p);
          if (HAS_M) st_stream(reinterpret_cast<float4 *>(p.M + static_cast<int64_t>(row) * ld + col), u);
          if (HAS_V) st_stream(reinterpret_cast<float4 *>(p.V + static_cast<int64_t>(row) * ld + col), v2);
          Xs[item] = h;
          if (DIAG) {
            csum = vadd(csum, h);
            // everything in transit in this column: this step's slot is in the stage, the others come from HBM
            if (HAS_RING) rsum = vadd(rsum, vadd(Rs[item], diag_ring_sum<float4>(p, static_cast<int64_t>(row) * ld + col, p.ring_x)));
          }
        }
      }
      const int dbuf = static_cast<int>(it & 1);
      if (DIAG) {
        ds.part[(dbuf * kDiagArrays + 0) * 256 + ctid] = csum;
        if (HAS_RING) ds.part[(dbuf * kDiagArrays + 1) * 256 + ctid] = rsum;
      }
      consumer_barrier();
      float4 mean_h = make_float4(0.f, 0.f, 0.f, 0.f), mean_x = mean_h;
      if (DIAG)
        diag_means<HAS_RING, float4>(p, ds.part + (dbuf * kDiagArrays + 0) * 256, ds.part + (dbuf * kDiagArrays + 1) * 256, ctid,
                                     &mean_h, &mean_x);
      if (!HAS_RING && p.uniform_parts > 0) {
        // all receivers alike (complete graph): one weighted column sum, shared by every row
        const int parts = p.uniform_parts;
        const int e0 = tab.rowptr[0], e1 = tab.rowptr[1];
        for (int idx = ctid; idx < tv * parts; idx += kTmaConsumers) {
          const int c = idx & (tv - 1), part = idx >> p.log2_tile_vecs;
          float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
          for (int e = e0 + part; e < e1; e += parts) acc = vfma(tab.val[e], Xs[(tab.col[e] << p.log2_tile_vecs) + c], acc);
          partial[idx] = acc;
        }
        consumer_barrier();
        for (int item = ctid; item < tile_items; item += kTmaConsumers) {
          const int row = item >> p.log2_tile_vecs;
          const int c = item & (tv - 1);
          const int64_t col = col0 + static_cast<int64_t>(c) * 4;
          if (col < p.col_end) {
            const int64_t o = static_cast<int64_t>(row) * ld + col;
            float4 acc = partial[c];
            for (int part = 1; part < parts; ++part) acc = vadd(acc, partial[part * tv + c]);
            const float4 z = vmul(tab.inv_w[row], acc);
            st_stream(reinterpret_cast<float4 *>(p.X + o), acc);
            if (HAS_Z) st_stream(reinterpret_cast<float4 *>(p.Z + o), z);
            if (DIAG) {
              float2 sq = ds.slots[item];
              sq.x += vsq(vsub(Xs[item], mean_h));
              sq.y += vsq(vsub(z, mean_x));
              ds.slots[item] = sq;
            }
          }
        }
        consumer_barrier();          // the partial sums are rewritten by the next tile
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(empty_bar + s);
        continue;
      }
      // phase 2: gather-mix, ring exchange, de-bias.  A thread works on kGather of its items at once: their
      // in-neighbour lists are walked together, so that kGather independent shared-memory loads and FMA chains are
      // in flight instead of one (the eight consumer warps are all the latency hiding this kernel has).
      constexpr int kGather = 4;
      for (int it0 = ctid; it0 < tile_items; it0 += kGather * kTmaConsumers) {
        int e0[kGather], len[kGather], cc[kGather];
        bool act[kGather];
        float4 acc[kGather], offd[kGather];
        int maxlen = 0;
#pragma unroll
        for (int q = 0; q < kGather; ++q) {
          const int item = it0 + q * kTmaConsumers;
          const int row = item >> p.log2_tile_vecs;
          cc[q] = item & (tv - 1);
          act[q] = item < tile_items && col0 + static_cast<int64_t>(cc[q]) * 4 < p.col_end;
          e0[q] = act[q] ? tab.rowptr[row] : 0;
          len[q] = act[q] ? tab.rowptr[row + 1] - e0[q] : 0;
          maxlen = max(maxlen, len[q]);
          acc[q] = make_float4(0.f, 0.f, 0.f, 0.f);
          offd[q] = acc[q];
        }
        for (int e = 0; e < maxlen; ++e) {
#pragma unroll
          for (int q = 0; q < kGather; ++q) {
            if (e < len[q]) {
              const int j = tab.col[e0[q] + e];
              if (SGP_BOUNDS_OK(p, j >= 0 && j < n)) {
                const float pv = tab.val[e0[q] + e];
                const float4 hj = Xs[(j << p.log2_tile_vecs) + cc[q]];
                if (HAS_RING && j != ((it0 + q * kTmaConsumers) >> p.log2_tile_vecs)) offd[q] = vfma(pv, hj, offd[q]);
                else acc[q] = vfma(pv, hj, acc[q]);
              }
            }
          }
        }
#pragma unroll
        for (int q = 0; q < kGather; ++q) {
          if (act[q]) {
            const int item = it0 + q * kTmaConsumers;
            const int row = item >> p.log2_tile_vecs;
            const int64_t o = static_cast<int64_t>(row) * ld + col0 + static_cast<int64_t>(cc[q]) * 4;
            float4 a = acc[q];
            if (HAS_RING) {
              a = vadd(a, Rs[item]);
              st_stream(reinterpret_cast<float4 *>(p.ring_x + o), offd[q]);
            }
            const float4 z = vmul(tab.inv_w[row], a);
            st_stream(reinterpret_cast<float4 *>(p.X + o), a);
            if (HAS_Z) st_stream(reinterpret_cast<float4 *>(p.Z + o), z);
            if (DIAG) {
              float2 sq = ds.slots[item];
              sq.x += vsq(vsub(Xs[item], mean_h));
              sq.y += vsq(vsub(z, mean_x));
              ds.slots[item] = sq;
            }
          }
        }
      }
      // the stage may be refilled by the async proxy once every consumer warp has released it
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive(empty_bar + s);
    }
    if (DIAG) {
      consumer_barrier();            // every consumer is here: all leave the loop together, also on an aborted run
      diag_flush(p, ds.slots, ctid, kTmaConsumers);
    }
  }
}

using TmaKernel = void (*)(const StepParams, const ConstTable, const TmaMaps, const int, const int);
// The instantiation for (optimiser, Z written, delay ring, fused diagnostics); one translation unit per DIAG value.
template <bool DIAG> TmaKernel tma_kernel_of(int upd, bool has_z, bool has_ring);

}  // namespace sgp
