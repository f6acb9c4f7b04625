// Register-staged fused SGP step kernel: every thread keeps kItemsPerThread (row, vector-column) items in
// flight, writes x^(k+1/2) into a shared tile, one barrier, then gathers its receivers' rows from the tile
// (Alg. 1 lines 4-8, Alg. 3 lines 4-5, Alg. 2 with the delayed-message ring).  The tile is double-buffered so
// one barrier per tile suffices; large n uses one tile and two barriers so that row segments stay long.
#pragma once
#include "step_common.cuh"

namespace sgp {

template <int VEC, int UPD, bool HAS_Z, bool HAS_RING, bool DIAG, bool GATHER_FIRST>
__global__ void __launch_bounds__(kThreads, 2)
sgp_step_regs_kernel(const __grid_constant__ StepParams p, const __grid_constant__ ConstTable ct) {
  using V = typename VecT<VEC>::type;
  constexpr bool HAS_M = UpdTraits<UPD>::kHasM;
  constexpr bool HAS_V = UpdTraits<UPD>::kHasV;
  // Adam with a delay ring keeps three items per thread: with four (20 loads in flight) it drops from 0.95 to 0.78
  // of the copy bandwidth, and with diagnostics on top it spills
  constexpr int kItemsPerThread = (UPD == kUpdAdam && HAS_RING) ? 3 : UpdTraits<UPD>::kItems;
  constexpr int kDiagArrays = HAS_RING ? 2 : 1;
  // GATHER_FIRST (momentum updates without a ring only; the launcher picks it for tiles made of full four-item batches
  // with row segments of 512 bytes or more): every gather of a batch before its stores, every update before its
  // momentum stores.  Plain SGD (8 items per thread) loses with this ordering: 0.85 against 0.95.
  constexpr bool kGatherFirst = GATHER_FIRST;
  static_assert(!GATHER_FIRST || (!HAS_RING && (UPD == kUpdHeavyBall || UPD == kUpdNesterov)), "not instantiated");
  extern __shared__ __align__(128) unsigned char smem_raw[];
  const int n = p.n;
  const int tv = 1 << p.log2_tile_vecs;
  const int tile_items = n * tv;
  V *H0 = reinterpret_cast<V *>(smem_raw);
  V *H1 = p.single_buffer ? H0 : H0 + tile_items;
  V *partial = H0 + (p.single_buffer ? 1 : 2) * tile_items;          // uniform_parts x tv vectors (uniform rows only)
  float *scratch = reinterpret_cast<float *>(partial + p.uniform_parts * tv);
  const CtaTables tab = cta_prologue<HAS_RING>(p, ct, scratch, kThreads);
  // Fused diagnostics (a separate instantiation, so the plain step pays nothing): scratch after the weights
  // and, when it was copied, the table.
  DiagScratch<V> ds{};
  int dbuf = 0;
  if (DIAG) {
    unsigned char *after = reinterpret_cast<unsigned char *>(scratch + 3 * n) +
                           (p.table_mode < 2 ? (static_cast<size_t>(n) + 1 + 2 * static_cast<size_t>(p.nnz)) * 4 : 0);
    ds = diag_scratch<V>(after, HAS_RING);
    for (int i = threadIdx.x; i < tile_items; i += kThreads) ds.slots[i] = make_float2(0.f, 0.f);
    __syncthreads();
  }

  const int64_t ld = p.ld;
  const int64_t ncols = p.col_end - p.col_begin;
  const int64_t tile_cols = static_cast<int64_t>(tv) * VEC;
  const int64_t ntiles = (ncols + tile_cols - 1) / tile_cols;
  int buf = 0;
  // The tile is worked off in batches of at most kItemsPerThread items per thread; the batches are made
  // equal (e.g. 1280 items: 3 + 2 per thread, not 4 + 1) so that no batch runs with few loads in flight.
  const int batches = (tile_items + kThreads * kItemsPerThread - 1) / (kThreads * kItemsPerThread);
  const int q_max = ((tile_items + batches - 1) / batches + kThreads - 1) / kThreads;   // items per thread per batch
  const int batch_items = q_max * kThreads;

  // Lockstep clusters: the CTAs of a cluster take neighbouring tiles and start each tile together, so that the parts
  // of a 1 KB block of a row that straddles their common tile edge are requested at about the same time.  Nothing
  // is shared between them; the barrier only aligns them in time.  (Written so that nothing but `tile` lives across
  // the loop: the instantiations at the register cap lose 1 % to one more live value.)
  for (int64_t tile = blockIdx.x;; tile += gridDim.x) {
    if (p.lockstep) {
      unsigned rank_in_cluster;
      asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(rank_in_cluster));
      if (tile - rank_in_cluster >= ntiles) break;      // the whole cluster is past the last tile
      asm volatile("barrier.cluster.arrive.relaxed.aligned;\n\tbarrier.cluster.wait.aligned;" ::: "memory");
    }
    if (tile >= ntiles) break;                           // a CTA past the last tile has kept the barrier count
    const int64_t col0 = p.col_begin + tile * tile_cols;
    V *H = buf ? H1 : H0;
    V csum = vzero<V>(), rsum = vzero<V>();      // diagnostics: this thread's share of its column's sums
    // ---- phase 1: local update, all batches of this tile
    for (int base = 0; base < tile_items; base += batch_items) {
      V x[kItemsPerThread], g[kItemsPerThread], u[kItemsPerThread], vv[kItemsPerThread];
      V rr[DIAG && HAS_RING ? kItemsPerThread : 1];   // diagnostics: everything in transit at this item
      bool ok[kItemsPerThread];
      int64_t off[kItemsPerThread];
#pragma unroll
      for (int q = 0; q < kItemsPerThread; ++q) {
        const int item = base + q * kThreads + threadIdx.x;
        const int row = item >> p.log2_tile_vecs;
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
          // issued with the batch's other loads (the mix re-reads this step's slot a moment later, from L2)
          if (DIAG && HAS_RING) rr[q] = diag_ring_sum<V>(p, off[q], nullptr);
        }
      }
      if constexpr (kGatherFirst) {
        // the same ordering in this phase: every update of the batch, then every momentum store (another +0.3 to
        // +0.5 %); x[q] becomes the half step
#pragma unroll
        for (int q = 0; q < kItemsPerThread; ++q)
          if (ok[q]) x[q] = local_update<UPD, V>(x[q], g[q], u[q], vv[q], p);
#pragma unroll
        for (int q = 0; q < kItemsPerThread; ++q)
          if (ok[q]) st_stream(reinterpret_cast<V *>(p.M + off[q]), u[q]);
      }
#pragma unroll
      for (int q = 0; q < kItemsPerThread; ++q) {
        const int item = base + q * kThreads + threadIdx.x;
        if (ok[q]) {
          V h = x[q];
          if constexpr (!kGatherFirst) {
            h = local_update<UPD, V>(x[q], g[q], u[q], vv[q], p);
            if (HAS_M) st_stream(reinterpret_cast<V *>(p.M + off[q]), u[q]);
            if (HAS_V) st_stream(reinterpret_cast<V *>(p.V + off[q]), vv[q]);
          }
          H[item] = h;
          if (DIAG) {
            csum = vadd(csum, h);
            if (HAS_RING) rsum = vadd(rsum, rr[q]);
          }
        } else if (q < q_max && item < tile_items) {
          H[item] = vzero<V>();
        }
      }
    }
    if (DIAG) {
      ds.part[(dbuf * kDiagArrays + 0) * 256 + threadIdx.x] = csum;
      if (HAS_RING) ds.part[(dbuf * kDiagArrays + 1) * 256 + threadIdx.x] = rsum;
    }
    __syncthreads();
    V mean_h = vzero<V>(), mean_x = vzero<V>();
    if (DIAG) {
      diag_means<HAS_RING, V>(p, ds.part + (dbuf * kDiagArrays + 0) * 256, ds.part + (dbuf * kDiagArrays + 1) * 256,
                              threadIdx.x, &mean_h, &mean_x);
      dbuf ^= 1;
    }
    // ---- phase 2, all receivers alike (complete graph): one weighted column sum, shared by every row
    if (!HAS_RING && p.uniform_parts > 0) {
      const int parts = p.uniform_parts;
      const int e0 = tab.rowptr[0], e1 = tab.rowptr[1];
      for (int idx = threadIdx.x; idx < tv * parts; idx += kThreads) {
        const int c = idx & (tv - 1), part = idx >> p.log2_tile_vecs;
        V acc = vzero<V>();
        for (int e = e0 + part; e < e1; e += parts) {
          const int j = tab.col[e];
          if (SGP_BOUNDS_OK(p, j >= 0 && j < n)) acc = vfma(tab.val[e], H[(j << p.log2_tile_vecs) + c], acc);
        }
        partial[idx] = acc;
      }
      __syncthreads();
      for (int item = threadIdx.x; item < tile_items; item += kThreads) {
        const int row = item >> p.log2_tile_vecs;
        const int c = item & (tv - 1);
        const int64_t col = col0 + static_cast<int64_t>(c) * VEC;
        if (col < p.col_end) {
          const int64_t o = static_cast<int64_t>(row) * ld + col;
          V acc = partial[c];
          for (int part = 1; part < parts; ++part) acc = vadd(acc, partial[part * tv + c]);
          const V z = vmul(tab.inv_w[row], acc);
          st_stream(reinterpret_cast<V *>(p.X + o), acc);
          if (HAS_Z) st_stream(reinterpret_cast<V *>(p.Z + o), z);
          if (DIAG) {
            float2 s = ds.slots[item];
            s.x += vsq(vsub(H[item], mean_h));
            s.y += vsq(vsub(z, mean_x));
            ds.slots[item] = s;
          }
        }
      }
      buf ^= 1;
      if (p.single_buffer) __syncthreads();
      continue;
    }
    // ---- phase 2: gather-mix over the step's in-neighbour lists, ring exchange, de-bias
    auto gather = [&](int row, int c, V &acc, V &offd) {
      const int e1 = tab.rowptr[row + 1];
      for (int e = tab.rowptr[row]; e < e1; ++e) {
        const int j = tab.col[e];
        if (!SGP_BOUNDS_OK(p, j >= 0 && j < n)) continue;
        const float pv = tab.val[e];
        const V hj = H[(j << p.log2_tile_vecs) + c];
        if (HAS_RING && j != row) offd = vfma(pv, hj, offd);
        else acc = vfma(pv, hj, acc);
      }
    };
    auto finish = [&](int item, int row, int64_t col, V acc, V offd, V ring) {
      const int64_t o = static_cast<int64_t>(row) * ld + col;
      if (HAS_RING) {
        acc = vadd(acc, ring);
        st_stream(reinterpret_cast<V *>(p.ring_x + o), offd);
      }
      const V z = vmul(tab.inv_w[row], acc);
      st_stream(reinterpret_cast<V *>(p.X + o), acc);
      if (HAS_Z) st_stream(reinterpret_cast<V *>(p.Z + o), z);
      if (DIAG) {
        float2 sq = ds.slots[item];
        sq.x += vsq(vsub(H[item], mean_h));
        sq.y += vsq(vsub(z, mean_x));
        ds.slots[item] = sq;
      }
    };
    for (int base = 0; base < tile_items; base += batch_items) {
      V ring_in[kItemsPerThread];
      if (HAS_RING) {
#pragma unroll
        for (int q = 0; q < kItemsPerThread; ++q) {
          const int item = base + q * kThreads + threadIdx.x;
          const int row = item >> p.log2_tile_vecs;
          const int c = item & (tv - 1);
          const int64_t col = col0 + static_cast<int64_t>(c) * VEC;
          if (q < q_max && item < tile_items && col < p.col_end)
            ring_in[q] = ld_inplace(reinterpret_cast<const V *>(p.ring_x + static_cast<int64_t>(row) * ld + col));
        }
      }
      if constexpr (kGatherFirst) {
        // every gather of the batch, then every store: the global stores leave in one run instead of being
        // threaded between the shared-memory reads (momentum updates, n = 16..64: +1 to +1.5 % of the copy
        // bandwidth; with Adam or a ring the extra live registers cost more than that, so those keep one loop)
        V accs[kItemsPerThread], offs[kItemsPerThread];
#pragma unroll
        for (int q = 0; q < kItemsPerThread; ++q) {
          const int item = base + q * kThreads + threadIdx.x;
          const int c = item & (tv - 1);
          accs[q] = vzero<V>();
          offs[q] = vzero<V>();
          if (q < q_max && item < tile_items && col0 + static_cast<int64_t>(c) * VEC < p.col_end)
            gather(item >> p.log2_tile_vecs, c, accs[q], offs[q]);
        }
#pragma unroll
        for (int q = 0; q < kItemsPerThread; ++q) {
          const int item = base + q * kThreads + threadIdx.x;
          const int64_t col = col0 + static_cast<int64_t>(item & (tv - 1)) * VEC;
          if (q < q_max && item < tile_items && col < p.col_end)
            finish(item, item >> p.log2_tile_vecs, col, accs[q], offs[q], HAS_RING ? ring_in[q] : vzero<V>());
        }
      } else {
#pragma unroll
        for (int q = 0; q < kItemsPerThread; ++q) {
          const int item = base + q * kThreads + threadIdx.x;
          const int row = item >> p.log2_tile_vecs;
          const int c = item & (tv - 1);
          const int64_t col = col0 + static_cast<int64_t>(c) * VEC;
          if (q < q_max && item < tile_items && col < p.col_end) {
            V acc = vzero<V>(), offd = vzero<V>();
            gather(row, c, acc, offd);
            finish(item, row, col, acc, offd, HAS_RING ? ring_in[q] : vzero<V>());
          }
        }
      }
    }
    buf ^= 1;
    if (p.single_buffer) __syncthreads();   // the only tile is about to be overwritten
  }
  if (DIAG) {
    __syncthreads();
    diag_flush(p, ds.slots, threadIdx.x, kThreads);
  }
}

using RegsKernel = void (*)(const StepParams, const ConstTable);
// The instantiation for (vector width 4 or 1, optimiser, Z written, delay ring, fused diagnostics); the kernels are
// spread over several translation units so that they compile in parallel.
// gather_first is honoured for momentum updates without a ring and ignored elsewhere.
RegsKernel regs_kernel(int vec, int upd, bool has_z, bool has_ring, bool diag, bool gather_first);
template <int VEC, bool DIAG> RegsKernel regs_kernel_of(int upd, bool has_z, bool has_ring, bool gather_first);

}  // namespace sgp
