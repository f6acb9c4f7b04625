// Fused SGP step kernels for sm_100a.
//
// One persistent CTA owns, tile after tile, ALL n rows of a block of columns: the mix of Alg. 1
// line 6 couples rows (nodes) but never columns, so a CTA that holds x^(k+1/2) of every node for
// its columns can finish the whole iteration -- local update (Alg. 3 lines 4-5), gather-mix,
// delayed-message ring (Alg. 2), de-bias (Alg. 1 line 8) -- with one read and one write of each
// array and no inter-CTA dependency (no grid sync, no device-side wait on another CTA).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace sgp {

constexpr int kThreads = 256;       // threads per CTA of the register-staged kernel

// Mixing table of one step small enough to travel as a kernel argument (constant bank).
constexpr int kConstRows = 64;
constexpr int kConstNnz = 320;
struct ConstTable {
  int32_t rowptr[kConstRows + 1];
  int32_t col[kConstNnz];
  float val[kConstNnz];
};

struct StepParams {
  float *X;
  float *W;
  float *M;        // momentum buffer / Adam first moment; null for plain SGD
  float *V;        // Adam second moment; null otherwise
  const float *G;
  float *Z;        // may be null
  float *ring_x;   // this step's ring slot (n x ld) or null when tau == 0
  float *ring_w;   // this step's weight-ring slot (n) or null
  int64_t ld;
  int64_t col_begin;  // first column this launch processes
  int64_t col_end;    // one past the last column
  int n;
  int nnz;
  int log2_tile_vecs;  // tile width in vectors (power of two)
  int update_w;        // 1: this launch also commits W (and the weight ring) for the step
  int table_mode;      // 0: copy table from the kernel argument, 1: copy from global, 2: read global in place
  int uniform_parts;   // > 0: every row of P is the same (complete graph) and tau == 0: the mix is ONE weighted
                       // column sum shared by all receivers, formed by this many interleaved partial sums
  int single_buffer;   // register kernel: 1 = one exchange tile and two barriers per tile (large n)
  int l2_hint;         // TMA kernel, L2 evict-first policy on the bulk copies: 0 none, 1 every array, 3 only G
                       // (dead after its read; X, M, V, ring are rewritten in place and keep the normal
                       // policy: measured 0.985 of the copy bandwidth against 0.967 without), 4 all but G
  int wait_limit_ms;   // TMA kernel: bound of every mbarrier wait in milliseconds
  int inject_stall;    // TMA kernel, fault-injection for tests: CTA 0 never requests its first tile, so its
                       // consumers' bounded wait runs out and the status word is set (nothing hangs)
  float lr, momentum, wd;
  // Adam only: decay rates, epsilon, lr / (1 - beta1^t) and 1 / sqrt(1 - beta2^t)
  float beta1, beta2, eps, adam_step, adam_rsqrt_bc2;
  const int32_t *rowptr;  // global copy of the step's CSR (always valid)
  const int32_t *col;
  const float *val;
  unsigned *ticket;  // arrival counter for the last-CTA-commits-W protocol (self-resetting)
  unsigned *status;  // device status word
};

template <int VEC> struct VecT;
template <> struct VecT<4> { using type = float4; };
template <> struct VecT<1> { using type = float; };

// Every array is read once and written once per step.  G is dead after its read: streaming load
// (evict first).  X, M, V and the ring are rewritten in place a moment later: their lines should stay
// in L2 until the store hits them, so they are loaded with the normal policy, bypassing L1 only.
__device__ __forceinline__ float4 ld_stream(const float4 *p) { return __ldcs(p); }
__device__ __forceinline__ float ld_stream(const float *p) { return __ldcs(p); }
__device__ __forceinline__ float4 ld_inplace(const float4 *p) { return __ldcg(p); }
__device__ __forceinline__ float ld_inplace(const float *p) { return __ldcg(p); }
__device__ __forceinline__ void st_stream(float4 *p, float4 v) { __stcs(p, v); }
__device__ __forceinline__ void st_stream(float *p, float v) { __stcs(p, v); }

__device__ __forceinline__ float4 vfma(float a, float4 b, float4 c) {
  return make_float4(fmaf(a, b.x, c.x), fmaf(a, b.y, c.y), fmaf(a, b.z, c.z), fmaf(a, b.w, c.w));
}
__device__ __forceinline__ float vfma(float a, float b, float c) { return fmaf(a, b, c); }
__device__ __forceinline__ float4 vmul(float a, float4 b) { return make_float4(a * b.x, a * b.y, a * b.z, a * b.w); }
__device__ __forceinline__ float vmul(float a, float b) { return a * b; }
__device__ __forceinline__ float4 vadd(float4 a, float4 b) { return make_float4(a.x + b.x, a.y + b.y, a.z + b.z, a.w + b.w); }
__device__ __forceinline__ float vadd(float a, float b) { return a + b; }
template <typename V> __device__ __forceinline__ V vzero();
template <> __device__ __forceinline__ float4 vzero<float4>() { return make_float4(0.f, 0.f, 0.f, 0.f); }
template <> __device__ __forceinline__ float vzero<float>() { return 0.f; }

__device__ __forceinline__ float4 vmulv(float4 a, float4 b) { return make_float4(a.x * b.x, a.y * b.y, a.z * b.z, a.w * b.w); }
__device__ __forceinline__ float vmulv(float a, float b) { return a * b; }
// a / (sqrt(v) * r + eps), IEEE square root and division
__device__ __forceinline__ float adam_ratio(float a, float v, float r, float eps) { return a / fmaf(sqrtf(v), r, eps); }
__device__ __forceinline__ float4 adam_ratio(float4 a, float4 v, float r, float eps) {
  return make_float4(adam_ratio(a.x, v.x, r, eps), adam_ratio(a.y, v.y, r, eps), adam_ratio(a.z, v.z, r, eps),
                     adam_ratio(a.w, v.w, r, eps));
}

// Which local optimiser runs on the biased numerators before the mix.
enum : int { kUpdSgd = 0, kUpdHeavyBall = 1, kUpdNesterov = 2, kUpdAdam = 3 };
template <int UPD> struct UpdTraits {
  static constexpr bool kHasM = UPD != kUpdSgd;
  static constexpr bool kHasV = UPD == kUpdAdam;
  // items a thread of the register kernel keeps in flight: 12 to 16 vector loads with every optimiser
  static constexpr int kItems = UPD == kUpdAdam ? 3 : (UPD == kUpdSgd ? 8 : 4);
};

// Local update of one element group: returns h = x^(k+1/2) and updates the optimiser state in place.
// SGD: Alg. 1 line 4.  Momentum / Nesterov: Alg. 3 lines 4-5.  Adam (Sec. 6.2, App. C.1: Adam-preconditioned
// SGP): bias-corrected Adam step on the numerator, moments stay local.
// Weight decay adds wd * x to the gradient in every case.
template <int UPD, typename V>
__device__ __forceinline__ V local_update(V x, V g, V &u, V &v, const StepParams &p) {
  const V gt = vfma(p.wd, x, g);
  if (UPD == kUpdAdam) {
    u = vfma(p.beta1, u, vmul(1.0f - p.beta1, gt));
    v = vfma(p.beta2, v, vmul(1.0f - p.beta2, vmulv(gt, gt)));
    return vfma(-p.adam_step, adam_ratio(u, v, p.adam_rsqrt_bc2, p.eps), x);
  }
  V s;
  if (UPD == kUpdSgd) {
    s = gt;
  } else {
    u = vfma(p.momentum, u, gt);
    s = UPD == kUpdNesterov ? vfma(p.momentum, u, gt) : u;
  }
  return vfma(-p.lr, s, x);
}

// Per-CTA scratch after the tiles/stages in dynamic shared memory: [w_old n][rw_in n][inv_w n], then the
// CSR copy [rowptr n+1][col nnz][val nnz] when table_mode < 2.
struct CtaTables {
  const int32_t *rowptr;
  const int32_t *col;
  const float *val;
  float *inv_w;
};

// Per-CTA prologue shared by the step kernels: stage the step's CSR, mix the push-sum weights
// (Alg. 1 line 7 / Alg. 2 lines 8, 22) and, when this launch owns the commit, let the LAST CTA to
// arrive write W and the weight ring back.  Every CTA takes its ticket only after its own reads of
// the old W have completed, so the committing CTA knows no reader is left; nobody waits for anybody.
template <bool HAS_RING>
__device__ __forceinline__ CtaTables cta_prologue(const StepParams &p, const ConstTable &ct, float *scratch, int nthreads) {
  const int n = p.n;
  float *w_old = scratch;
  float *rw_in = scratch + n;
  float *inv_w = scratch + 2 * n;
  int32_t *s_rowptr = reinterpret_cast<int32_t *>(scratch + 3 * n);
  int32_t *s_col = s_rowptr + (n + 1);
  float *s_val = reinterpret_cast<float *>(s_col + p.nnz);
  __shared__ int s_is_last;

  CtaTables t;
  t.inv_w = inv_w;
  if (p.table_mode == 2) {
    t.rowptr = p.rowptr;
    t.col = p.col;
    t.val = p.val;
  } else {
    const int32_t *src_rowptr = p.table_mode == 0 ? ct.rowptr : p.rowptr;
    const int32_t *src_col = p.table_mode == 0 ? ct.col : p.col;
    const float *src_val = p.table_mode == 0 ? ct.val : p.val;
    for (int i = threadIdx.x; i <= n; i += nthreads) s_rowptr[i] = src_rowptr[i];
    for (int e = threadIdx.x; e < p.nnz; e += nthreads) {
      s_col[e] = src_col[e];
      s_val[e] = src_val[e];
    }
    t.rowptr = s_rowptr;
    t.col = s_col;
    t.val = s_val;
  }
  for (int i = threadIdx.x; i < n; i += nthreads) {
    w_old[i] = p.W[i];
    if (HAS_RING) rw_in[i] = p.ring_w[i];
  }
  __syncthreads();
  if (p.update_w && threadIdx.x == 0) {
    __threadfence();
    const unsigned ticket = atomicAdd(p.ticket, 1u);
    s_is_last = (ticket == gridDim.x - 1) ? 1 : 0;
  }
  __syncthreads();
  const bool commit = p.update_w && s_is_last;
  for (int i = threadIdx.x; i < n; i += nthreads) {
    float acc = 0.f, off = 0.f;
    for (int e = t.rowptr[i]; e < t.rowptr[i + 1]; ++e) {
      const int j = t.col[e];
      const float pv = t.val[e];
      if (HAS_RING && j != i) off = fmaf(pv, w_old[j], off);
      else acc = fmaf(pv, w_old[j], acc);
    }
    if (HAS_RING) acc += rw_in[i];
    inv_w[i] = 1.0f / acc;
    if (commit) {
      p.W[i] = acc;
      if (HAS_RING) p.ring_w[i] = off;
    }
  }
  if (commit && threadIdx.x == 0) *p.ticket = 0u;  // ready for the next launch
  __syncthreads();
  return t;
}

// ------------------------------------------------------------------------------------------------
// Register-staged kernel: every thread keeps kItemsPerThread (row, vector-column) items in flight,
// writes x^(k+1/2) into a shared tile, one barrier, then gathers its receivers' rows from the tile.
// The tile is double-buffered so one barrier per batch suffices.
// ------------------------------------------------------------------------------------------------
template <int VEC, int UPD, bool HAS_Z, bool HAS_RING>
__global__ void __launch_bounds__(kThreads, 2)
sgp_step_regs_kernel(const __grid_constant__ StepParams p, const __grid_constant__ ConstTable ct) {
  using V = typename VecT<VEC>::type;
  constexpr bool HAS_M = UpdTraits<UPD>::kHasM;
  constexpr bool HAS_V = UpdTraits<UPD>::kHasV;
  constexpr int kItemsPerThread = UpdTraits<UPD>::kItems;
  extern __shared__ __align__(128) unsigned char smem_raw[];
  const int n = p.n;
  const int tv = 1 << p.log2_tile_vecs;
  const int tile_items = n * tv;
  V *H0 = reinterpret_cast<V *>(smem_raw);
  V *H1 = p.single_buffer ? H0 : H0 + tile_items;
  V *partial = H0 + (p.single_buffer ? 1 : 2) * tile_items;          // uniform_parts x tv vectors (uniform rows only)
  float *scratch = reinterpret_cast<float *>(partial + p.uniform_parts * tv);
  const CtaTables tab = cta_prologue<HAS_RING>(p, ct, scratch, kThreads);

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

  for (int64_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
    const int64_t col0 = p.col_begin + tile * tile_cols;
    V *H = buf ? H1 : H0;
    // ---- phase 1: local update, all batches of this tile
    for (int base = 0; base < tile_items; base += batch_items) {
      V x[kItemsPerThread], g[kItemsPerThread], u[kItemsPerThread], vv[kItemsPerThread];
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
    __syncthreads();
    // ---- phase 2, all receivers alike (complete graph): one weighted column sum, shared by every row
    if (!HAS_RING && p.uniform_parts > 0) {
      const int parts = p.uniform_parts;
      const int e0 = tab.rowptr[0], e1 = tab.rowptr[1];
      for (int idx = threadIdx.x; idx < tv * parts; idx += kThreads) {
        const int c = idx & (tv - 1), part = idx >> p.log2_tile_vecs;
        V acc = vzero<V>();
        for (int e = e0 + part; e < e1; e += parts) acc = vfma(tab.val[e], H[(tab.col[e] << p.log2_tile_vecs) + c], acc);
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
          st_stream(reinterpret_cast<V *>(p.X + o), acc);
          if (HAS_Z) st_stream(reinterpret_cast<V *>(p.Z + o), vmul(tab.inv_w[row], acc));
        }
      }
      buf ^= 1;
      if (p.single_buffer) __syncthreads();
      continue;
    }
    // ---- phase 2: gather-mix over the step's in-neighbour lists, ring exchange, de-bias
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
#pragma unroll
      for (int q = 0; q < kItemsPerThread; ++q) {
        const int item = base + q * kThreads + threadIdx.x;
        const int row = item >> p.log2_tile_vecs;
        const int c = item & (tv - 1);
        const int64_t col = col0 + static_cast<int64_t>(c) * VEC;
        if (q < q_max && item < tile_items && col < p.col_end) {
          const int64_t o = static_cast<int64_t>(row) * ld + col;
          V acc = vzero<V>(), offd = vzero<V>();
          const int e1 = tab.rowptr[row + 1];
          for (int e = tab.rowptr[row]; e < e1; ++e) {
            const int j = tab.col[e];
            const float pv = tab.val[e];
            const V hj = H[(j << p.log2_tile_vecs) + c];
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
    buf ^= 1;
    if (p.single_buffer) __syncthreads();   // the only tile is about to be overwritten
  }
}

}  // namespace sgp

namespace sgp {

// ------------------------------------------------------------------------------------------------
// Bulk-copy (TMA) pipelined kernel.  A producer warp streams whole column tiles -- every node's row
// segment of X, G (and M, ring) -- into a ring of shared-memory stages with cp.async.bulk, completion
// counted on an mbarrier per stage; eight consumer warps update, exchange through the stage itself
// (x^(k+1/2) overwrites the X tile in place), gather-mix and store with 128-bit streaming stores.
// Loads therefore stay in flight while the consumers compute and store.  No multicast, no cluster.
// Every wait is bounded: on expiry the CTA records a status bit and leaves.
// ------------------------------------------------------------------------------------------------
constexpr int kTmaConsumers = 256;
constexpr int kTmaThreads = kTmaConsumers + 32;
constexpr unsigned kStatusFullTimeout = 1u;
constexpr unsigned kStatusEmptyTimeout = 2u;
constexpr unsigned kStatusDrainTimeout = 4u;

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

template <int UPD, bool HAS_Z, bool HAS_RING>
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
        }
      }
      consumer_barrier();
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
            st_stream(reinterpret_cast<float4 *>(p.X + o), acc);
            if (HAS_Z) st_stream(reinterpret_cast<float4 *>(p.Z + o), vmul(tab.inv_w[row], acc));
          }
        }
        consumer_barrier();          // the partial sums are rewritten by the next tile
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(empty_bar + s);
        continue;
      }
      // phase 2: gather-mix, ring exchange, de-bias
      for (int item = ctid; item < tile_items; item += kTmaConsumers) {
        const int row = item >> p.log2_tile_vecs;
        const int c = item & (tv - 1);
        const int64_t col = col0 + static_cast<int64_t>(c) * 4;
        if (col < p.col_end) {
          const int64_t o = static_cast<int64_t>(row) * ld + col;
          float4 acc = make_float4(0.f, 0.f, 0.f, 0.f), offd = acc;
          const int e1 = tab.rowptr[row + 1];
          for (int e = tab.rowptr[row]; e < e1; ++e) {
            const int j = tab.col[e];
            const float pv = tab.val[e];
            const float4 hj = Xs[(j << p.log2_tile_vecs) + c];
            if (HAS_RING && j != row) offd = vfma(pv, hj, offd);
            else acc = vfma(pv, hj, acc);
          }
          if (HAS_RING) {
            acc = vadd(acc, Rs[item]);
            st_stream(reinterpret_cast<float4 *>(p.ring_x + o), offd);
          }
          st_stream(reinterpret_cast<float4 *>(p.X + o), acc);
          if (HAS_Z) st_stream(reinterpret_cast<float4 *>(p.Z + o), vmul(tab.inv_w[row], acc));
        }
      }
      // the stage may be refilled by the async proxy once every consumer warp has released it
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive(empty_bar + s);
    }
  }
}

}  // namespace sgp
