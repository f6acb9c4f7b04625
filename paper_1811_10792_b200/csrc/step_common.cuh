// Pieces shared by the fused SGP step kernels for sm_100a: kernel arguments, vector helpers, the local
// optimiser update and the per-CTA prologue (schedule table, push-sum weight mix).
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

// Bits of the device status word.
constexpr unsigned kStatusFullTimeout = 1u;    // pipelined kernel: consumers gave up waiting for a tile
constexpr unsigned kStatusEmptyTimeout = 2u;   // pipelined kernel: the producer gave up waiting for a free stage
constexpr unsigned kStatusDrainTimeout = 4u;   // pipelined kernel: copies still pending at exit
constexpr unsigned kStatusZeroWeight = 8u;     // a push-sum weight was <= 0 or not a number (z set to 0, never inf)
constexpr unsigned kStatusNonFinite = 16u;     // invariant check: non-finite entries in X or the ring
constexpr unsigned kStatusWeightSum = 32u;     // invariant check: sum of weights (incl. in transit) is not n
constexpr unsigned kStatusColumnSum = 64u;     // invariant check: a column sum drifted (mix not column-stochastic)
constexpr unsigned kStatusBounds = 128u;       // bounds-checked build: an index was out of range (access skipped)

// Bounds-checked build (-DSGP_CHECKED): every table index and every global offset is tested before use; a
// violation sets kStatusBounds and the access is skipped.  Nothing traps.
#ifdef SGP_CHECKED
#define SGP_BOUNDS_OK(p, cond) ((cond) ? true : (atomicOr((p).status, ::sgp::kStatusBounds), false))
#else
#define SGP_BOUNDS_OK(p, cond) (true)
#endif

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
  int biased;          // 1: z = x, the push-sum weight is left out of the de-bias (Table 4, biased OSGP)
  int peel_phase0;     // peeled kernel: floats between the last 16-byte boundary and element (row 0, col_begin)
  int peel_phase_step; // peeled kernel: ld mod 4, what a row adds to that distance
  int lockstep;        // register kernel: > 0 = launched as clusters of this many CTAs that take neighbouring tiles and
                       // meet at a cluster barrier before each tile (no data is shared between them)
  float lr, momentum, wd;
  // Adam only: decay rates, epsilon, lr / (1 - beta1^t) and 1 / sqrt(1 - beta2^t)
  float beta1, beta2, eps, adam_step, adam_rsqrt_bc2;
  const int32_t *rowptr;  // global copy of the step's CSR (always valid)
  const int32_t *col;
  const float *val;
  unsigned *ticket;  // arrival counter for the last-CTA-commits-W protocol (self-resetting)
  unsigned *status;  // device status word
  // Diagnostics fused into the pass (null = off): diag[i] += sum_c (h_ic - hbar_c)^2, the parameter deviation
  // of Sec. 6.1 taken after the gradient step and before the mix; diag[n + i] += sum_c (z_ic - xbar_c)^2 with
  // xbar the node-wise average that counts the messages in transit (consensus lemma of the supplement).
  double *diag;
  const float *ring_base;  // slot 0 of the ring (diagnostics read every slot), null when tau == 0
  int tau;
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
__device__ __forceinline__ float4 vsub(float4 a, float4 b) { return make_float4(a.x - b.x, a.y - b.y, a.z - b.z, a.w - b.w); }
__device__ __forceinline__ float vsub(float a, float b) { return a - b; }
// sum of squares of the components
__device__ __forceinline__ float vsq(float4 a) { return fmaf(a.x, a.x, fmaf(a.y, a.y, fmaf(a.z, a.z, a.w * a.w))); }
__device__ __forceinline__ float vsq(float a) { return a * a; }
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
  // items a thread of the register kernel keeps in flight: 12 to 16 vector loads with every optimiser (Adam: four
  // items = 16 loads reach 0.977 of the copy bandwidth at n = 16 where three reach 0.955)
  static constexpr int kItems = UPD == kUpdAdam ? 4 : (UPD == kUpdSgd ? 8 : 4);
};

// The optimiser's scalars, separate from the launch geometry so that every kernel of the library (fused step,
// expected-column-sum pre-pass of the debug check, one-node-per-GPU update) runs the very same arithmetic.
struct UpdateScalars {
  float lr, momentum, wd, beta1, beta2, eps, adam_step, adam_rsqrt_bc2;
};

// Local update of one element group: returns h = x^(k+1/2) and updates the optimiser state in place.
// SGD: Alg. 1 line 4.  Momentum / Nesterov: Alg. 3 lines 4-5.  Adam (Sec. 6.2, App. C.1: Adam-preconditioned
// SGP): bias-corrected Adam step on the numerator, moments stay local.
// Weight decay adds wd * x to the gradient in every case.
// `p` is anything with the fields lr, momentum, wd, beta1, beta2, eps, adam_step, adam_rsqrt_bc2 (StepParams itself,
// so that the scalars stay constant-bank operands, or UpdateScalars).
template <int UPD, typename V, typename P>
__device__ __forceinline__ V local_update(V x, V g, V &u, V &v, const P &p) {
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

// 1 / w for the de-bias; a weight that is not positive (or not a number) yields 0 and a status bit, never inf.
__device__ __forceinline__ float safe_inverse_weight(float w, unsigned *status) {
  if (!(w > 0.0f)) {
    atomicOr(status, kStatusZeroWeight);
    return 0.0f;
  }
  return 1.0f / w;
}

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
    const int e0 = t.rowptr[i], e1 = t.rowptr[i + 1];
    if (SGP_BOUNDS_OK(p, e0 >= 0 && e0 <= e1 && e1 <= p.nnz)) {
      for (int e = e0; e < e1; ++e) {
        const int j = t.col[e];
        if (!SGP_BOUNDS_OK(p, j >= 0 && j < n)) continue;
        const float pv = t.val[e];
        if (HAS_RING && j != i) off = fmaf(pv, w_old[j], off);
        else acc = fmaf(pv, w_old[j], acc);
      }
    }
    if (HAS_RING) acc += rw_in[i];
    // the weight is checked by the CTA that commits it (one report per step); every CTA guards its own 1/w
    inv_w[i] = p.biased ? 1.0f : (acc > 0.0f ? 1.0f / acc : 0.0f);
    if (commit) {
      if (!(acc > 0.0f)) atomicOr(p.status, kStatusZeroWeight);
      p.W[i] = acc;
      if (HAS_RING) p.ring_w[i] = off;
    }
  }
  if (commit && threadIdx.x == 0) *p.ticket = 0u;  // ready for the next launch
  __syncthreads();
  return t;
}

// ---- fused diagnostics (the DIAG instantiations of the step kernels) -----------------------------
// A thread of either kernel owns the same column c = tid mod tv of every tile (tv <= 256 vectors per row segment
// is enforced by the launchers when diagnostics are on), and the same set of rows.  So:
//   * the column sums of the half step (and of the ring) are formed from per-thread partial sums taken while the
//     half step is computed -- 256 / tv threads share a column; their partials meet in `part` behind the barrier
//     the kernel has anyway (two buffers by tile parity: no extra barrier);
//   * the squared deviations of item (row, c) go to a private fp32 slot per item, summed over the tiles without
//     atomics or shuffles; the slots are reduced per row once, at the end of the kernel.
// Shared-memory scratch, placed by the kernels after their own buffers:
//   [part: 2 parities x (1 + HAS_RING) arrays x 256 vectors][slots: n * tv float2 (deviation^2, consensus^2)]
template <typename V>
struct DiagScratch {
  float2 *slots;
  V *part;
};
template <typename V>
__host__ __device__ inline size_t diag_scratch_bytes(int n, int tv, bool has_ring) {
  return static_cast<size_t>(n) * tv * sizeof(float2) + static_cast<size_t>(2) * (has_ring ? 2 : 1) * 256 * sizeof(V) + 16;
}
template <typename V>
__device__ __forceinline__ DiagScratch<V> diag_scratch(unsigned char *base, bool has_ring) {
  DiagScratch<V> s;
  s.part = reinterpret_cast<V *>((reinterpret_cast<uintptr_t>(base) + 15) & ~uintptr_t{15});
  s.slots = reinterpret_cast<float2 *>(s.part + 2 * (has_ring ? 2 : 1) * 256);
  return s;
}

// Sum over every ring slot of element (row, col) read from global memory, skipping `skip_slot` (the slot a kernel
// already holds on chip); slot stride n * ld.
template <typename V>
__device__ __forceinline__ V diag_ring_sum(const StepParams &p, int64_t offset, const float *skip_slot) {
  V acc = vzero<V>();
  const int64_t slot_stride = static_cast<int64_t>(p.n) * p.ld;
  for (int s = 0; s < p.tau; ++s) {
    const float *slot = p.ring_base + s * slot_stride;
    if (slot != skip_slot) acc = vadd(acc, ld_inplace(reinterpret_cast<const V *>(slot + offset)));
  }
  return acc;
}

// Column means for this thread's column from the partial sums of the 256 / tv threads that share it:
// mean_h = (1/n) sum_i h_i, mean_x = mean_h + (1/n) (ring column sum) -- by column-stochasticity the node-wise
// average AFTER the mix, messages in transit included.
template <bool HAS_RING, typename V>
__device__ __forceinline__ void diag_means(const StepParams &p, const V *part_h, const V *part_r, int tid, V *mean_h, V *mean_x) {
  const int tv = 1 << p.log2_tile_vecs;
  const int c = tid & (tv - 1);
  V acc = vzero<V>(), racc = vzero<V>();
  for (int g = c; g < 256; g += tv) {
    acc = vadd(acc, part_h[g]);
    if (HAS_RING) racc = vadd(racc, part_r[g]);
  }
  const float inv_n = 1.0f / static_cast<float>(p.n);
  *mean_h = vmul(inv_n, acc);
  *mean_x = vmul(inv_n, vadd(acc, racc));
}

// End of the kernel: every warp reduces whole rows of the slots and adds them to the global accumulators
// (fp64 atomics, 2n per CTA).  `nthreads` threads with index `tid` take part.
__device__ __forceinline__ void diag_flush(const StepParams &p, const float2 *slots, int tid, int nthreads) {
  const int tv = 1 << p.log2_tile_vecs;
  const int warp = tid >> 5, lane = tid & 31, nwarps = nthreads >> 5;
  for (int row = warp; row < p.n; row += nwarps) {
    float dq = 0.f, cq = 0.f;
    for (int c = lane; c < tv; c += 32) {
      const float2 v = slots[row * tv + c];
      dq += v.x;
      cq += v.y;
    }
    for (int o = 16; o > 0; o >>= 1) {
      dq += __shfl_xor_sync(0xffffffffu, dq, o);
      cq += __shfl_xor_sync(0xffffffffu, cq, o);
    }
    if (lane == 0) {
      atomicAdd(p.diag + row, static_cast<double>(dq));
      atomicAdd(p.diag + p.n + row, static_cast<double>(cq));
    }
  }
}

}  // namespace sgp
