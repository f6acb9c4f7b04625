// C ABI of the fused SGP step (see include/sgp.h): handle management, argument validation, launch
// plan and dispatch.  All arithmetic of the method lives in the kernels.
#include <cuda_runtime.h>
#include <nvtx3/nvToolsExt.h>

#include <algorithm>
#include <cmath>
#include <cstring>
#include <new>
#include <utility>
#include <vector>

#include "aux_kernels.cuh"
#include "launch.h"
#include "schedule.h"
#include "sgp.h"

using sgp::ConstTable;
using sgp::StepParams;

namespace {
constexpr int kDevStatsCheck = 0;                          // kStatCount doubles of sgp_check
constexpr int kDevStatsDeviation = 8;                      // SGP_MAX_NODES doubles of sgp_param_deviation
constexpr int kDevStatsDiag = 8 + SGP_MAX_NODES;           // 2 * SGP_MAX_NODES doubles of the fused diagnostics
constexpr int kDevStatsCount = 8 + 3 * SGP_MAX_NODES;
constexpr unsigned kWaitBits = sgp::kStatusFullTimeout | sgp::kStatusEmptyTimeout | sgp::kStatusDrainTimeout;
constexpr double kColumnDriftTol = 1e-5;
}  // namespace

struct sgp_handle {
  int n = 0;
  int64_t d = 0, ld = 0;
  int tau = 0;
  unsigned flags = 0;
  sgp::DeviceInfo dev;
  sgp_schedule *sched = nullptr;
  SgpStepCsr identity;           // P = I, the mixing matrix of a step without transmissions (send_period > 1)
  // device copy of every slot's CSR (the schedule's slots, then the identity), concatenated; offsets in elements
  int32_t *d_rowptr = nullptr;
  int32_t *d_col = nullptr;
  float *d_val = nullptr;
  std::vector<int64_t> off_rowptr, off_nnz;
  std::vector<ConstTable> const_tables;  // valid where const_ok[slot]
  std::vector<char> const_ok;
  float *ring_x = nullptr;   // tau * n * ld
  float *ring_w = nullptr;   // tau * n
  unsigned *d_words = nullptr;  // [0] ticket, [1] status
  double *d_stats = nullptr;    // kDevStatsCount doubles
  double *d_expect = nullptr;   // d doubles, allocated when "check_steps" is switched on
  int64_t opt_variant = 0, opt_tile_cols = 0, opt_ctas_per_sm = 0, opt_stages = 0, opt_l2_hint = 0, opt_single_buffer = 0, opt_wait_limit_ms = 0,
          opt_inject_stall = 0, opt_send_period = 1, opt_diagnostics = 0, opt_check_steps = 0, opt_cluster = 0, opt_lockstep = 0;
  sgp::LaunchRecord last;       // of the most recent step launch
  int64_t launches = 0;         // step kernels launched so far
  bool diag_valid = false;      // a step with diagnostics has been enqueued since the last reset
  unsigned seen_status = 0;     // status bits a synchronising call has read back
  cudaStream_t s_h2d = nullptr, s_compute = nullptr, s_d2h = nullptr;
  cudaEvent_t ev_entry = nullptr;
  std::vector<cudaEvent_t> ev_in, ev_done;
  int last_cuda_error = 0;
  // tensor maps already encoded for (base pointer, box columns)
  struct MapEntry {
    const void *ptr;
    int box_cols;
    CUtensorMap map;
  };
  std::vector<MapEntry> map_cache;
  void *encode_fn = nullptr;   // cuTensorMapEncodeTiled, resolved lazily through the runtime
  bool encode_tried = false;
};

namespace {

#define SGP_CUDA_TRY(h, expr)                                   \
  do {                                                          \
    cudaError_t e_ = (expr);                                    \
    if (e_ != cudaSuccess) {                                    \
      if (h) (h)->last_cuda_error = static_cast<int>(e_);       \
      (void)cudaGetLastError();                                 \
      return SGP_ERR_CUDA;                                      \
    }                                                           \
  } while (0)

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// NVTX range around an entry point's host work (header-only NVTX: a no-op unless a tool is attached).
struct NvtxRange {
  explicit NvtxRange(const char *name) { nvtxRangePushA(name); }
  ~NvtxRange() { nvtxRangePop(); }
  NvtxRange(const NvtxRange &) = delete;
  NvtxRange &operator=(const NvtxRange &) = delete;
};

void free_handle(sgp_handle *h) {
  if (h == nullptr) return;
  cudaFree(h->d_rowptr);
  cudaFree(h->d_col);
  cudaFree(h->d_val);
  cudaFree(h->ring_x);
  cudaFree(h->ring_w);
  cudaFree(h->d_words);
  cudaFree(h->d_stats);
  cudaFree(h->d_expect);
  for (cudaEvent_t e : h->ev_in) cudaEventDestroy(e);
  for (cudaEvent_t e : h->ev_done) cudaEventDestroy(e);
  if (h->ev_entry) cudaEventDestroy(h->ev_entry);
  if (h->s_h2d) cudaStreamDestroy(h->s_h2d);
  if (h->s_compute) cudaStreamDestroy(h->s_compute);
  if (h->s_d2h) cudaStreamDestroy(h->s_d2h);
  delete h->sched;
  delete h;
}

struct StepArgs {
  float *X, *W, *M;
  const float *G;
  float *Z;
  int64_t k;
  float lr, momentum, wd;
  int upd;                 // sgp::kUpd*
  float *V = nullptr;      // Adam second moment
  float beta1 = 0.f, beta2 = 0.f, eps = 0.f, adam_step = 0.f, adam_rsqrt_bc2 = 0.f;
};

inline int update_kind(float momentum, int nesterov) {
  if (momentum == 0.0f) return sgp::kUpdSgd;
  return nesterov != 0 ? sgp::kUpdNesterov : sgp::kUpdHeavyBall;
}

// Table slot of step k: the c-th transmission (c = k / send_period) uses slot c mod period; a step on which
// nobody transmits mixes with the identity, stored after the schedule's slots (Alg. 2 lines 5-12).
inline size_t slot_of(const sgp_handle *h, int64_t k) {
  const int64_t s = h->opt_send_period;
  if (k % s != 0) return static_cast<size_t>(h->sched->period());
  return static_cast<size_t>((k / s) % h->sched->period());
}
inline const SgpStepCsr &csr_of(const sgp_handle *h, size_t slot) {
  return slot == static_cast<size_t>(h->sched->period()) ? h->identity : h->sched->steps[slot];
}

// Fills the launch-independent part of the kernel arguments for step a.k.
void fill_params(const sgp_handle *h, const StepArgs &a, int64_t c0, int64_t c1, bool update_w, StepParams *out) {
  const size_t slot = slot_of(h, a.k);
  const SgpStepCsr &csr = csr_of(h, slot);
  StepParams p{};
  p.X = a.X;
  p.W = a.W;
  p.M = a.M;
  p.V = a.V;
  p.G = a.G;
  p.Z = a.Z;
  p.beta1 = a.beta1;
  p.beta2 = a.beta2;
  p.eps = a.eps;
  p.adam_step = a.adam_step;
  p.adam_rsqrt_bc2 = a.adam_rsqrt_bc2;
  if (h->tau > 0) {
    const int64_t rs = a.k % h->tau;
    p.ring_x = h->ring_x + rs * h->n * h->ld;
    p.ring_w = h->ring_w + rs * h->n;
    p.ring_base = h->ring_x;
  }
  p.tau = h->tau;
  p.ld = h->ld;
  p.col_begin = c0;
  p.col_end = c1;
  p.n = h->n;
  p.nnz = static_cast<int>(csr.col.size());
  p.update_w = update_w ? 1 : 0;
  p.uniform_parts = 0;
  p.biased = (h->flags & SGP_FLAG_BIASED) ? 1 : 0;
  p.lr = a.lr;
  p.momentum = a.momentum;
  p.wd = a.wd;
  p.rowptr = h->d_rowptr + h->off_rowptr[slot];
  p.col = h->d_col + h->off_nnz[slot];
  p.val = h->d_val + h->off_nnz[slot];
  p.ticket = h->d_words;
  p.status = h->d_words + 1;
  p.diag = h->opt_diagnostics ? h->d_stats + kDevStatsDiag : nullptr;
  *out = p;
}

// Launch plan of one step: which kernel, how wide a tile, how deep a pipeline, how many CTAs per SM.
struct Plan {
  int variant;        // 1 register-staged, 2 TMA with tensor maps, 3 TMA with per-row bulk copies, 4 thread-block cluster
  int64_t tile_cols;  // 0 = kernel default
  int stages;
  int cps;
};

// Heuristics from measurements on B200.  The step is HBM-bound; what decides the achieved bandwidth
// is the length of the contiguous row segments (>= 1 KB), the bytes in flight per SM and a grid that
// is exactly one wave.  Measured (fraction of the copy bandwidth, rows on 1 KB boundaries):
//   momentum, n <= 24 : register-staged 0.97, TMA 0.90      momentum, n = 32 : TMA 0.985, register-staged 0.95
//   no momentum, n=16 : TMA 0.98, register-staged 0.97      tau = 1, n = 32  : register-staged 0.97
// cps = 0 means "as many CTAs per SM as are resident" (worked out at launch).
// Explicit options override each field.
Plan make_plan(const sgp_handle *h, int arrays, bool has_m, int nnz, bool vec) {
  Plan pl{1, 0, 2, 0};
  if (vec) {
    const size_t table = sgp::table_smem_bytes(h->n, nnz);
    const size_t fixed = 16 * sizeof(uint64_t) + 3 * static_cast<size_t>(h->n) * 4 + 1024 + (table <= 40 * 1024 ? table : 0);
    const size_t per_kb = static_cast<size_t>(arrays) * h->n * 1024;   // one stage at 1 KB per row segment
    const size_t full_sm = 224 * 1024;
    // The pipelined kernel has ONE consumer group, so its gather is on the critical path: it is only used
    // for sparse steps (at most three in-neighbours per node on average; with five it drops to 0.94, with
    // nine to 0.88, while the register-staged kernel holds 0.98 and 0.95).
    const bool sparse = static_cast<int64_t>(nnz) <= 3 * static_cast<int64_t>(h->n);
    if (!sparse) {
      pl.tile_cols = sgp::regs_tile_cols(h->n, fixed);
    } else if (!has_m && per_kb >= 24 * 1024 && per_kb <= 40 * 1024) {
      // plain SGD with about 32 KB per stage (n = 16): two CTAs per SM, two stages: 0.98 against 0.97 for the
      // register-staged kernel, which wins at every other n (n = 4: 0.97 against 0.93, n = 32: 0.98 against 0.88)
      pl = Plan{3, 256, 2, 2};
    } else if (has_m && per_kb == 96 * 1024 && 2 * per_kb + fixed <= full_sm) {
      // momentum with exactly 96 KB per stage (n = 32 with three arrays): one CTA per SM, two stages: 0.985 on
      // the one-peer graph against 0.97 for the register-staged kernel; at n = 26..30, 34, 36 the
      // register-staged kernel wins (0.96-0.99 against 0.91-0.95)
      pl = Plan{3, 256, 2, 1};
    } else {
      pl.tile_cols = sgp::regs_tile_cols(h->n, fixed);
    }
  }
  // Diagnostics with a momentum update: the register-staged instantiation carries them for free (n = 32: 0.971 of the
  // copy bandwidth with them, 0.955 without; the pipelined kernel 0.964 with them).
  if (vec && h->opt_diagnostics && has_m && pl.variant >= 2) pl = Plan{1, sgp::regs_tile_cols(h->n, 4 * 1024), 2, 0};
  if (h->opt_variant > 0 && (h->opt_variant == 1) != (pl.variant == 1)) {
    // the caller forces the other kernel family: take that family's defaults
    if (h->opt_variant == 1 || h->opt_variant >= 4) {
      pl = Plan{1, vec ? sgp::regs_tile_cols(h->n, 4 * 1024) : 0, 2, 0};
    } else {
      pl = Plan{static_cast<int>(h->opt_variant), 256, 2, 2};
    }
  }
  if (h->opt_variant > 0 && h->opt_variant < 4) pl.variant = static_cast<int>(h->opt_variant);
  if (h->opt_tile_cols > 0) pl.tile_cols = h->opt_tile_cols;
  if (h->opt_stages > 0) pl.stages = static_cast<int>(h->opt_stages);
  if (h->opt_ctas_per_sm > 0) pl.cps = static_cast<int>(h->opt_ctas_per_sm);
  return pl;
}

void record_launch(sgp_handle *h, const sgp::LaunchRecord &rec, int rc) {
  if (rc == SGP_OK) {
    h->last = rec;
    ++h->launches;
  } else if (rc == SGP_ERR_CUDA) {
    h->last_cuda_error = rec.cuda_error;
  }
}

// One launch of the register-staged kernel over columns [c0, c1) with vector width vec.
int launch_regs(sgp_handle *h, const StepArgs &a, const Plan &pl, int64_t c0, int64_t c1, int vec, bool update_w,
                cudaStream_t stream) {
  const size_t slot = slot_of(h, a.k);
  StepParams p{};
  fill_params(h, a, c0, c1, update_w, &p);
  sgp::RegsOptions opt;
  opt.tile_cols = pl.tile_cols;
  opt.tile_cols_forced = h->opt_tile_cols > 0;
  opt.cps = pl.cps;
  opt.single_buffer = static_cast<int>(h->opt_single_buffer);
  opt.lockstep = static_cast<int>(h->opt_lockstep);
  sgp::LaunchRecord rec;
  const int rc = sgp::launch_regs(h->dev, p, h->const_ok[slot] ? &h->const_tables[slot] : nullptr, a.upd, vec,
                                  csr_of(h, slot).uniform_rows, opt, stream, &rec);
  record_launch(h, rec, rc);
  return rc;
}

using EncodeTiledFn = CUresult (*)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                   const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// Tensor map of an n x d fp32 array with row pitch ld whose box is (box_cols x n); cached per pointer.
// Returns false when the driver entry point is unavailable or the encoding is rejected.
bool get_tensor_map(void *ctx, const float *base, int box_cols, CUtensorMap *out) {
  sgp_handle *h = static_cast<sgp_handle *>(ctx);
  for (const auto &e : h->map_cache)
    if (e.ptr == base && e.box_cols == box_cols) {
      *out = e.map;
      return true;
    }
  if (!h->encode_tried) {
    h->encode_tried = true;
    cudaDriverEntryPointQueryResult qres;
    void *fn = nullptr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      h->encode_fn = fn;
    else
      (void)cudaGetLastError();
  }
  if (h->encode_fn == nullptr || h->d >= (int64_t{1} << 31)) return false;
  const cuuint64_t gdim[2] = {static_cast<cuuint64_t>(h->d), static_cast<cuuint64_t>(h->n)};
  const cuuint64_t gstride[1] = {static_cast<cuuint64_t>(h->ld) * sizeof(float)};
  const cuuint32_t box[2] = {static_cast<cuuint32_t>(box_cols), static_cast<cuuint32_t>(h->n)};
  const cuuint32_t estride[2] = {1, 1};
  CUtensorMap m;
  const CUresult r = reinterpret_cast<EncodeTiledFn>(h->encode_fn)(
      &m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float *>(base), gdim, gstride, box, estride,
      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return false;
  if (h->map_cache.size() >= 256) h->map_cache.clear();
  h->map_cache.push_back({base, box_cols, m});
  *out = m;
  return true;
}

// One launch of the bulk-copy pipelined kernel over columns [c0, c1) (needs the 128-bit preconditions).
// Returns SGP_ERR_STATE when the shape does not fit its shared-memory stages; the caller then uses
// the register-staged kernel.
int launch_tma(sgp_handle *h, const StepArgs &a, const Plan &pl, int64_t c0, int64_t c1, bool update_w,
               cudaStream_t stream) {
  const size_t slot = slot_of(h, a.k);
  StepParams p{};
  fill_params(h, a, c0, c1, update_w, &p);
  sgp::TmaOptions opt;
  opt.variant = pl.variant;
  opt.tile_cols = pl.tile_cols > 0 ? pl.tile_cols : 256;
  opt.tile_cols_forced = h->opt_tile_cols > 0;
  opt.stages = pl.stages;
  opt.stages_forced = h->opt_stages > 0;
  opt.cps = pl.cps > 0 ? pl.cps : 2;
  opt.wait_limit_ms = h->opt_wait_limit_ms > 0 ? static_cast<int>(h->opt_wait_limit_ms) : 2000;
  opt.inject_stall = h->opt_inject_stall ? 1 : 0;
  opt.l2_hint = h->opt_l2_hint == 2 ? 0 : (h->opt_l2_hint == 0 ? 3 : static_cast<int>(h->opt_l2_hint));
  sgp::LaunchRecord rec;
  const int rc = sgp::launch_tma(h->dev, p, h->const_ok[slot] ? &h->const_tables[slot] : nullptr, a.upd,
                                 csr_of(h, slot).uniform_rows, opt, get_tensor_map, h, stream, &rec);
  record_launch(h, rec, rc);
  return rc;
}

// The whole step over columns [c0, c1): 128-bit kernel on the aligned bulk, scalar kernel on what is left.
int launch_step_range(sgp_handle *h, const StepArgs &a, int64_t c0, int64_t c1, bool update_w, cudaStream_t stream) {
  const bool vec_ok = aligned16(a.X) && aligned16(a.G) && (a.M == nullptr || aligned16(a.M)) &&
                      (a.V == nullptr || aligned16(a.V)) && (a.Z == nullptr || aligned16(a.Z)) && (h->ld % 4 == 0) &&
                      (c0 % 4 == 0);
  const int64_t vec_end = vec_ok ? c0 + ((c1 - c0) & ~int64_t{3}) : c0;
  const int arrays = 2 + (a.M != nullptr ? 1 : 0) + (a.V != nullptr ? 1 : 0) + (h->tau > 0 ? 1 : 0);
  const int nnz = static_cast<int>(csr_of(h, slot_of(h, a.k)).col.size());
  // Rows that do not start on 16-byte boundaries (ld not a multiple of 4, or every array offset alike): the peeled
  // kernel cuts each row at its own boundaries and keeps 128-bit accesses (about twice the scalar instantiation's
  // speed).  Steps whose rows of P are all alike keep the shared-column-sum path of the scalar instantiation.
  {
    const size_t slot = slot_of(h, a.k);
    const bool shortcut = h->tau == 0 && csr_of(h, slot).uniform_rows;
    const bool want_peel = h->opt_variant == 5 || (h->opt_variant == 0 && !vec_ok && !shortcut);
    if (want_peel && !h->opt_diagnostics && c1 - c0 >= 16) {
      StepParams p{};
      fill_params(h, a, c0, c1, update_w, &p);
      sgp::PeelOptions po;
      po.tile_cols = h->opt_tile_cols;
      po.cps = static_cast<int>(h->opt_ctas_per_sm);
      po.single_buffer = static_cast<int>(h->opt_single_buffer);
      sgp::LaunchRecord rec;
      const int rc = sgp::launch_peel(h->dev, p, h->const_ok[slot] ? &h->const_tables[slot] : nullptr, a.upd, po, stream, &rec);
      if (rc != SGP_ERR_STATE) {
        record_launch(h, rec, rc);
        return rc;
      }
    }
  }
  if (vec_end > c0) {
    Plan pl = make_plan(h, arrays, a.M != nullptr, nnz, true);
    // short rows (fewer 1 KB tiles than SMs): the register kernel with narrow tiles spreads them better
    if (h->opt_variant == 0 && pl.variant >= 2 && (vec_end - c0) < int64_t{256} * h->dev.sm_count) pl = Plan{1, 256, 2, 0};
    // rows that do not start on 128-byte boundaries (a dense pitch): the register-staged kernel in lockstep pairs
    // reaches 0.91 of the copy bandwidth at n = 32 where the pipelined kernel reaches 0.89
    const uintptr_t row_bits = reinterpret_cast<uintptr_t>(a.X) | reinterpret_cast<uintptr_t>(a.G) | reinterpret_cast<uintptr_t>(a.M) |
                               reinterpret_cast<uintptr_t>(a.Z) | static_cast<uintptr_t>(h->ld * 4);
    if (h->opt_variant == 0 && h->opt_lockstep != 1 && pl.variant >= 2 && a.M != nullptr && (row_bits & 127) != 0)
      pl = Plan{1, sgp::regs_tile_cols(h->n, 4 * 1024), 2, 0};
    int rc = SGP_ERR_STATE;
    // Opt-in (variant 4): a cluster of CTAs shares the tile through distributed shared memory, so that row segments
    // stay 1 KB long at n = 256 (256 bytes with one CTA).  Measured slower than the one-CTA kernel at every shape
    // tried (n = 256, d = 1e7: 0.77 of the copy bandwidth with 4 CTAs, 0.86 with 2, against 0.93; n = 64..128:
    // 0.73-0.87 against 0.92-0.96): two cluster barriers per tile and remote-shared-memory latency in the
    // gather's dependent chain cost more than the longer segments return.  Never chosen automatically.
    const size_t slot = slot_of(h, a.k);
    const bool cluster_ok = !h->opt_diagnostics && !(h->tau == 0 && csr_of(h, slot).uniform_rows) && h->n >= 2;
    const bool want_cluster = h->opt_variant == 4 && h->opt_cluster != 1;
    if (cluster_ok && want_cluster) {
      StepParams p{};
      fill_params(h, a, c0, vec_end, update_w && vec_end == c1, &p);
      sgp::ClusterOptions copt;
      copt.cluster_size = h->opt_cluster >= 2 ? static_cast<int>(h->opt_cluster) : 2;
      if (h->opt_tile_cols > 0) {
        copt.tile_cols = h->opt_tile_cols;
        copt.tile_cols_forced = true;
      }
      sgp::LaunchRecord rec;
      rc = sgp::launch_cluster(h->dev, p, h->const_ok[slot] ? &h->const_tables[slot] : nullptr, a.upd, copt, stream, &rec);
      record_launch(h, rec, rc);
    }
    if (rc == SGP_ERR_STATE && pl.variant >= 2) rc = launch_tma(h, a, pl, c0, vec_end, update_w && vec_end == c1, stream);
    if (rc == SGP_ERR_STATE) {
      Plan fallback = pl;
      if (pl.variant >= 2 && h->opt_ctas_per_sm == 0) fallback.cps = 0;
      rc = launch_regs(h, a, fallback, c0, vec_end, 4, update_w && vec_end == c1, stream);
    }
    if (rc != SGP_OK) return rc;
  }
  if (vec_end < c1) return launch_regs(h, a, make_plan(h, arrays, a.M != nullptr, nnz, false), vec_end, c1, 1, update_w, stream);
  return SGP_OK;
}

unsigned column_grid(const sgp_handle *h) {
  return static_cast<unsigned>(std::max<int64_t>(1, std::min<int64_t>((h->d + 255) / 256, static_cast<int64_t>(h->dev.sm_count) * 8)));
}

// Debug pre-pass of a checked step: what every column of X plus ring must sum to after the step.
int launch_expected(sgp_handle *h, const StepArgs &a, cudaStream_t st) {
  const sgp::UpdateScalars us{a.lr, a.momentum, a.wd, a.beta1, a.beta2, a.eps, a.adam_step, a.adam_rsqrt_bc2};
  const unsigned grid = column_grid(h);
  const int ring_rows = h->tau * h->n;
  switch (a.upd) {
    case sgp::kUpdSgd:
      sgp::sgp_expected_colsum_kernel<sgp::kUpdSgd><<<grid, 256, 0, st>>>(a.X, a.G, a.M, a.V, h->n, h->d, h->ld, us, h->ring_x, ring_rows, h->d_expect);
      break;
    case sgp::kUpdHeavyBall:
      sgp::sgp_expected_colsum_kernel<sgp::kUpdHeavyBall><<<grid, 256, 0, st>>>(a.X, a.G, a.M, a.V, h->n, h->d, h->ld, us, h->ring_x, ring_rows, h->d_expect);
      break;
    case sgp::kUpdNesterov:
      sgp::sgp_expected_colsum_kernel<sgp::kUpdNesterov><<<grid, 256, 0, st>>>(a.X, a.G, a.M, a.V, h->n, h->d, h->ld, us, h->ring_x, ring_rows, h->d_expect);
      break;
    default:
      sgp::sgp_expected_colsum_kernel<sgp::kUpdAdam><<<grid, 256, 0, st>>>(a.X, a.G, a.M, a.V, h->n, h->d, h->ld, us, h->ring_x, ring_rows, h->d_expect);
  }
  // the weight sum before the step (weights in transit included) lands in d_stats[6] (and the minimum in [7]): the
  // scan writes at kStatSumW = 2 and kStatMinW = 3 from the pointer it is given
  sgp::sgp_weight_scan_kernel<<<1, 256, 0, st>>>(a.W, h->n, h->ring_w, h->tau * h->n, h->d_stats + kDevStatsCheck + 4);
  SGP_CUDA_TRY(h, cudaGetLastError());
  return SGP_OK;
}

// Enqueues the invariant scan of (X, W, ring) against an optional column-sum reference; statistics stay on the
// device (d_stats) and violations are ORed into the status word.  No synchronisation.
int enqueue_check(sgp_handle *h, const float *X, const float *W, const double *ref, cudaStream_t st,
                  const double *sum_before = nullptr) {
  double *stats = h->d_stats + kDevStatsCheck;
  SGP_CUDA_TRY(h, cudaMemsetAsync(stats, 0, sgp::kStatCount * sizeof(double), st));
  sgp::sgp_colsum_kernel<<<column_grid(h), 256, 0, st>>>(X, h->n, h->d, h->ld, h->ring_x, h->tau * h->n, nullptr, ref, stats);
  sgp::sgp_weight_scan_kernel<<<1, 256, 0, st>>>(W, h->n, h->ring_w, h->tau * h->n, stats);
  sgp::sgp_check_finalize_kernel<<<1, 1, 0, st>>>(stats, h->n, 1, ref != nullptr ? 1 : 0, kColumnDriftTol, h->d_words + 1, sum_before);
  SGP_CUDA_TRY(h, cudaGetLastError());
  return SGP_OK;
}

// A whole step on the device arrays: optional debug bracket, optional diagnostics, the fused launch(es).
int run_step(sgp_handle *h, const StepArgs &a, cudaStream_t st) {
  const NvtxRange range(a.upd == sgp::kUpdAdam ? "sgp_step_adam" : "sgp_step");
  if (h->seen_status & kWaitBits) return SGP_ERR_DEVICE;
  if (h->seen_status & sgp::kStatusZeroWeight) return SGP_ERR_ZERO_WEIGHT;
  if (h->opt_check_steps) {
    const int rc = launch_expected(h, a, st);
    if (rc != SGP_OK) return rc;
  }
  if (h->opt_diagnostics) {
    SGP_CUDA_TRY(h, cudaMemsetAsync(h->d_stats + kDevStatsDiag, 0, 2 * static_cast<size_t>(h->n) * sizeof(double), st));
    h->diag_valid = true;
  }
  const int rc = launch_step_range(h, a, 0, h->d, true, st);
  if (rc != SGP_OK) return rc;
  // the bracket compares the weight sum with the one taken before the step (d_stats[6]), not with n
  if (h->opt_check_steps) return enqueue_check(h, a.X, a.W, h->d_expect, st, h->d_stats + kDevStatsCheck + 6);
  return SGP_OK;
}

// The handle's tables and ring live on the device that was current at sgp_create.
int check_device(const sgp_handle *h) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) {
    (void)cudaGetLastError();
    return SGP_ERR_CUDA;
  }
  return dev == h->dev.device ? SGP_OK : SGP_ERR_STATE;
}

int validate_step(const sgp_handle *h, const float *X, const float *W, const float *M, const float *G, int64_t k,
                  float momentum) {
  if (h == nullptr || X == nullptr || W == nullptr || G == nullptr || k < 0) return SGP_ERR_ARG;
  if (momentum != 0.0f && M == nullptr) return SGP_ERR_ARG;
  return check_device(h);
}

// Builds the device tables of a compiled schedule (plus the identity step) and installs them (and the schedule)
// in the handle, releasing whatever the handle held before.  The caller guarantees that no kernel still reads
// the old tables.
int upload_schedule(sgp_handle *h, sgp_schedule *sched) {
  std::vector<int32_t> rowptr, col;
  std::vector<float> val;
  std::vector<int64_t> off_rowptr, off_nnz;
  std::vector<ConstTable> const_tables;
  std::vector<char> const_ok;
  const SgpStepCsr identity = sgp_identity_step(h->n);
  for (int64_t s = 0; s <= sched->period(); ++s) {
    const SgpStepCsr &c = s < sched->period() ? sched->steps[static_cast<size_t>(s)] : identity;
    off_rowptr.push_back(static_cast<int64_t>(rowptr.size()));
    off_nnz.push_back(static_cast<int64_t>(col.size()));
    rowptr.insert(rowptr.end(), c.rowptr.begin(), c.rowptr.end());
    col.insert(col.end(), c.col.begin(), c.col.end());
    val.insert(val.end(), c.val.begin(), c.val.end());
    ConstTable ct{};
    const bool fits = h->n <= sgp::kConstRows && static_cast<int>(c.col.size()) <= sgp::kConstNnz;
    if (fits) {
      std::copy(c.rowptr.begin(), c.rowptr.end(), ct.rowptr);
      std::copy(c.col.begin(), c.col.end(), ct.col);
      std::copy(c.val.begin(), c.val.end(), ct.val);
    }
    const_tables.push_back(ct);
    const_ok.push_back(fits ? 1 : 0);
  }
  int32_t *d_rowptr = nullptr, *d_col = nullptr;
  float *d_val = nullptr;
  auto release = [&]() {
    cudaFree(d_rowptr);
    cudaFree(d_col);
    cudaFree(d_val);
    (void)cudaGetLastError();
  };
  if (cudaMalloc(&d_rowptr, rowptr.size() * sizeof(int32_t)) != cudaSuccess ||
      cudaMalloc(&d_col, col.size() * sizeof(int32_t)) != cudaSuccess ||
      cudaMalloc(&d_val, val.size() * sizeof(float)) != cudaSuccess) {
    release();
    return SGP_ERR_ALLOC;
  }
  if (cudaMemcpy(d_rowptr, rowptr.data(), rowptr.size() * sizeof(int32_t), cudaMemcpyHostToDevice) != cudaSuccess ||
      cudaMemcpy(d_col, col.data(), col.size() * sizeof(int32_t), cudaMemcpyHostToDevice) != cudaSuccess ||
      cudaMemcpy(d_val, val.data(), val.size() * sizeof(float), cudaMemcpyHostToDevice) != cudaSuccess) {
    release();
    return SGP_ERR_CUDA;
  }
  cudaFree(h->d_rowptr);
  cudaFree(h->d_col);
  cudaFree(h->d_val);
  h->d_rowptr = d_rowptr;
  h->d_col = d_col;
  h->d_val = d_val;
  h->off_rowptr.swap(off_rowptr);
  h->off_nnz.swap(off_nnz);
  h->const_tables.swap(const_tables);
  h->const_ok.swap(const_ok);
  h->identity = identity;
  if (h->sched != sched) delete h->sched;
  h->sched = sched;
  return SGP_OK;
}

// Reads the device status word back (the stream must already be synchronised) and remembers what it saw.
int refresh_status(sgp_handle *h, unsigned *out) {
  unsigned v = 0;
  SGP_CUDA_TRY(h, cudaMemcpy(&v, h->d_words + 1, sizeof(unsigned), cudaMemcpyDeviceToHost));
  h->seen_status |= v;
  if (out) *out = v;
  return SGP_OK;
}

// The host-buffer step: column chunks pipelined over three streams (H2D of chunk c+1, fused step on chunk c, D2H of
// chunk c-1); `a` carries the device arrays and the optimiser, a.G / a.Z are the device staging arrays.
int run_host_step(sgp_handle *h, const StepArgs &a, const float *h_G, float *h_Z, int64_t chunk_cols, void *stream) {
  const NvtxRange range("sgp_step_host");
  float *d_G = const_cast<float *>(a.G);
  float *d_Z = a.Z;
  int rc = SGP_OK;
  if (h->seen_status & kWaitBits) return SGP_ERR_DEVICE;
  if (h->seen_status & sgp::kStatusZeroWeight) return SGP_ERR_ZERO_WEIGHT;
  if (h->s_h2d == nullptr) {
    SGP_CUDA_TRY(h, cudaStreamCreateWithFlags(&h->s_h2d, cudaStreamNonBlocking));
    SGP_CUDA_TRY(h, cudaStreamCreateWithFlags(&h->s_compute, cudaStreamNonBlocking));
    SGP_CUDA_TRY(h, cudaStreamCreateWithFlags(&h->s_d2h, cudaStreamNonBlocking));
    SGP_CUDA_TRY(h, cudaEventCreateWithFlags(&h->ev_entry, cudaEventDisableTiming));
  }
  // default chunk: about 64 MB of gradient per chunk, a multiple of 1024 columns; the first and last chunks are
  // smaller (8, 16, 32 MB ...) so that the pipeline fills and drains in a fraction of a chunk time
  const bool ramp = chunk_cols <= 0;
  if (chunk_cols <= 0) chunk_cols = std::max<int64_t>(1024, (int64_t{64} << 20) / (4 * h->n) / 1024 * 1024);
  chunk_cols = (chunk_cols + 3) / 4 * 4;
  std::vector<int64_t> bounds{0};
  if (ramp && h->d >= 4 * chunk_cols) {
    std::vector<int64_t> head;
    for (int64_t w = std::max<int64_t>(1024, chunk_cols / 8 / 1024 * 1024); w < chunk_cols; w *= 2) head.push_back(w);
    int64_t head_cols = 0;
    for (int64_t w : head) head_cols += w;
    for (int64_t w : head) bounds.push_back(bounds.back() + w);
    while (h->d - head_cols - bounds.back() > chunk_cols) bounds.push_back(bounds.back() + chunk_cols);
    // what is left (at most a chunk plus the tail ramp) goes out in halves down to the smallest head chunk
    int64_t left = h->d - bounds.back();
    for (size_t i = head.size(); i-- > 0 && left > head[i];) {
      const int64_t w = std::max<int64_t>(head[i], (left / 2 + 1023) / 1024 * 1024);
      if (w >= left) break;
      bounds.push_back(bounds.back() + w);
      left -= w;
    }
    bounds.push_back(h->d);
  } else {
    while (bounds.back() + chunk_cols < h->d) bounds.push_back(bounds.back() + chunk_cols);
    bounds.push_back(h->d);
  }
  const int64_t nchunks = static_cast<int64_t>(bounds.size()) - 1;
  while (static_cast<int64_t>(h->ev_in.size()) < nchunks) {
    cudaEvent_t ev_a = nullptr, ev_b = nullptr;
    SGP_CUDA_TRY(h, cudaEventCreateWithFlags(&ev_a, cudaEventDisableTiming));
    h->ev_in.push_back(ev_a);
    SGP_CUDA_TRY(h, cudaEventCreateWithFlags(&ev_b, cudaEventDisableTiming));
    h->ev_done.push_back(ev_b);
  }
  // what the caller already enqueued on its stream (it may produce X, W, M or read d_G, d_Z) comes first:
  // an event wait on the device, not a host synchronisation
  SGP_CUDA_TRY(h, cudaEventRecord(h->ev_entry, static_cast<cudaStream_t>(stream)));
  SGP_CUDA_TRY(h, cudaStreamWaitEvent(h->s_h2d, h->ev_entry, 0));
  SGP_CUDA_TRY(h, cudaStreamWaitEvent(h->s_compute, h->ev_entry, 0));
  SGP_CUDA_TRY(h, cudaStreamWaitEvent(h->s_d2h, h->ev_entry, 0));
  if (h->opt_diagnostics) {
    SGP_CUDA_TRY(h, cudaMemsetAsync(h->d_stats + kDevStatsDiag, 0, 2 * static_cast<size_t>(h->n) * sizeof(double), h->s_compute));
    h->diag_valid = true;
  }
  const size_t pitch = static_cast<size_t>(h->ld) * sizeof(float);
  for (int64_t c = 0; c < nchunks; ++c) {
    const int64_t c0 = bounds[static_cast<size_t>(c)], c1 = bounds[static_cast<size_t>(c) + 1];
    const size_t width = static_cast<size_t>(c1 - c0) * sizeof(float);
    SGP_CUDA_TRY(h, cudaMemcpy2DAsync(d_G + c0, pitch, h_G + c0, pitch, width, static_cast<size_t>(h->n),
                                      cudaMemcpyHostToDevice, h->s_h2d));
    SGP_CUDA_TRY(h, cudaEventRecord(h->ev_in[static_cast<size_t>(c)], h->s_h2d));
    SGP_CUDA_TRY(h, cudaStreamWaitEvent(h->s_compute, h->ev_in[static_cast<size_t>(c)], 0));
    rc = launch_step_range(h, a, c0, c1, c == nchunks - 1, h->s_compute);
    if (rc != SGP_OK) return rc;
    if (h_Z != nullptr) {
      SGP_CUDA_TRY(h, cudaEventRecord(h->ev_done[static_cast<size_t>(c)], h->s_compute));
      SGP_CUDA_TRY(h, cudaStreamWaitEvent(h->s_d2h, h->ev_done[static_cast<size_t>(c)], 0));
      SGP_CUDA_TRY(h, cudaMemcpy2DAsync(h_Z + c0, pitch, d_Z + c0, pitch, width, static_cast<size_t>(h->n),
                                        cudaMemcpyDeviceToHost, h->s_d2h));
    }
  }
  SGP_CUDA_TRY(h, cudaStreamSynchronize(h->s_h2d));
  SGP_CUDA_TRY(h, cudaStreamSynchronize(h->s_compute));
  SGP_CUDA_TRY(h, cudaStreamSynchronize(h->s_d2h));
  return refresh_status(h, nullptr);
}

}  // namespace

extern "C" {

int sgp_version(void) { return 200; }

const char *sgp_strerror(int code) {
  switch (code) {
    case SGP_OK: return "ok";
    case SGP_ERR_ARG: return "invalid argument";
    case SGP_ERR_GRAPH: return "schedule is not a column-stochastic digraph with self-loops";
    case SGP_ERR_CUDA: return "CUDA runtime error";
    case SGP_ERR_ALLOC: return "allocation failed";
    case SGP_ERR_STATE: return "call not valid for this handle";
    case SGP_ERR_DEVICE: return "a kernel gave up a bounded wait";
    case SGP_ERR_ZERO_WEIGHT: return "a push-sum weight is not positive";
    case SGP_ERR_INVARIANT: return "an invariant of column-stochastic mixing does not hold";
    default: return "unknown error";
  }
}

int sgp_create(sgp_handle **out, int n, int64_t d, int64_t ld, const sgp_graph_desc *g, int tau, unsigned flags) {
  if (out == nullptr) return SGP_ERR_ARG;
  *out = nullptr;
  if (n < 1 || n > SGP_MAX_NODES || d < 1 || ld < d || tau < 0 || tau > 64 || g == nullptr || (flags & ~SGP_FLAG_BIASED) != 0)
    return SGP_ERR_ARG;
  sgp_schedule *sched = nullptr;
  int rc = sgp_schedule_build(&sched, n, g);
  if (rc != SGP_OK) return rc;
  sgp_handle *h = new (std::nothrow) sgp_handle;
  if (h == nullptr) {
    delete sched;
    return SGP_ERR_ALLOC;
  }
  h->n = n;
  h->d = d;
  h->ld = ld;
  h->tau = tau;
  h->flags = flags;
  h->sched = sched;

  auto fail = [&](int code) {
    free_handle(h);
    (void)cudaGetLastError();
    return code;
  };
  if (cudaGetDevice(&h->dev.device) != cudaSuccess) return fail(SGP_ERR_CUDA);
  if (cudaDeviceGetAttribute(&h->dev.sm_count, cudaDevAttrMultiProcessorCount, h->dev.device) != cudaSuccess) return fail(SGP_ERR_CUDA);
  if (cudaDeviceGetAttribute(&h->dev.smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, h->dev.device) != cudaSuccess)
    return fail(SGP_ERR_CUDA);
  {
    const int rc_up = upload_schedule(h, sched);
    if (rc_up != SGP_OK) return fail(rc_up);
  }
  if (cudaMalloc(&h->d_words, 2 * sizeof(unsigned)) != cudaSuccess) return fail(SGP_ERR_ALLOC);
  if (cudaMalloc(&h->d_stats, kDevStatsCount * sizeof(double)) != cudaSuccess) return fail(SGP_ERR_ALLOC);
  if (tau > 0) {
    if (cudaMalloc(&h->ring_x, static_cast<size_t>(tau) * n * ld * sizeof(float)) != cudaSuccess) return fail(SGP_ERR_ALLOC);
    if (cudaMalloc(&h->ring_w, static_cast<size_t>(tau) * n * sizeof(float)) != cudaSuccess) return fail(SGP_ERR_ALLOC);
    if (cudaMemset(h->ring_x, 0, static_cast<size_t>(tau) * n * ld * sizeof(float)) != cudaSuccess) return fail(SGP_ERR_CUDA);
    if (cudaMemset(h->ring_w, 0, static_cast<size_t>(tau) * n * sizeof(float)) != cudaSuccess) return fail(SGP_ERR_CUDA);
  }
  if (cudaMemset(h->d_words, 0, 2 * sizeof(unsigned)) != cudaSuccess) return fail(SGP_ERR_CUDA);
  if (cudaMemset(h->d_stats, 0, kDevStatsCount * sizeof(double)) != cudaSuccess) return fail(SGP_ERR_CUDA);
  if (cudaDeviceSynchronize() != cudaSuccess) return fail(SGP_ERR_CUDA);
  *out = h;
  return SGP_OK;
}

int sgp_destroy(sgp_handle *h) {
  if (h == nullptr) return SGP_OK;
  (void)cudaDeviceSynchronize();
  free_handle(h);
  return SGP_OK;
}

int sgp_set_graph(sgp_handle *h, const sgp_graph_desc *g) {
  if (h == nullptr || g == nullptr) return SGP_ERR_ARG;
  int rc = check_device(h);
  if (rc != SGP_OK) return rc;
  sgp_schedule *sched = nullptr;
  rc = sgp_schedule_build(&sched, h->n, g);
  if (rc != SGP_OK) return rc;                       // the handle keeps its current schedule
  SGP_CUDA_TRY(h, cudaDeviceSynchronize());          // no kernel may still read the old tables
  rc = upload_schedule(h, sched);
  if (rc != SGP_OK) delete sched;
  return rc;
}

int sgp_get_schedule(const sgp_handle *h, const sgp_schedule **s) {
  if (h == nullptr || s == nullptr) return SGP_ERR_ARG;
  *s = h->sched;
  return SGP_OK;
}

int sgp_step(sgp_handle *h, float *d_X, float *d_W, float *d_M, const float *d_G, float *d_Z, int64_t k, float lr,
             float momentum, float weight_decay, int nesterov, void *stream) {
  const int rc = validate_step(h, d_X, d_W, d_M, d_G, k, momentum);
  if (rc != SGP_OK) return rc;
  const StepArgs a{d_X, d_W, momentum != 0.0f ? d_M : nullptr, d_G, d_Z, k, lr, momentum, weight_decay,
                   update_kind(momentum, nesterov)};
  return run_step(h, a, static_cast<cudaStream_t>(stream));
}

int sgp_step_adam(sgp_handle *h, float *d_X, float *d_W, float *d_M1, float *d_M2, const float *d_G, float *d_Z,
                  int64_t k, int64_t t, float lr, float beta1, float beta2, float eps, float weight_decay, void *stream) {
  if (h == nullptr || d_X == nullptr || d_W == nullptr || d_M1 == nullptr || d_M2 == nullptr || d_G == nullptr ||
      k < 0 || t < 1 || !(beta1 >= 0.0f && beta1 < 1.0f) || !(beta2 >= 0.0f && beta2 < 1.0f) || !(eps >= 0.0f))
    return SGP_ERR_ARG;
  if (check_device(h) != SGP_OK) return check_device(h);
  StepArgs a{d_X, d_W, d_M1, d_G, d_Z, k, lr, 0.0f, weight_decay, sgp::kUpdAdam};
  a.V = d_M2;
  a.beta1 = beta1;
  a.beta2 = beta2;
  a.eps = eps;
  // bias corrections in double, rounded once (t >= 1)
  const double bc1 = 1.0 - std::pow(static_cast<double>(beta1), static_cast<double>(t));
  const double bc2 = 1.0 - std::pow(static_cast<double>(beta2), static_cast<double>(t));
  a.adam_step = static_cast<float>(static_cast<double>(lr) / bc1);
  a.adam_rsqrt_bc2 = static_cast<float>(1.0 / std::sqrt(bc2));
  return run_step(h, a, static_cast<cudaStream_t>(stream));
}

int sgp_debias(sgp_handle *h, const float *d_X, const float *d_W, float *d_Z, void *stream) {
  if (h == nullptr || d_X == nullptr || d_W == nullptr || d_Z == nullptr) return SGP_ERR_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const bool vec_ok = aligned16(d_X) && aligned16(d_Z) && (h->ld % 4 == 0);
  const int64_t work = vec_ok ? (h->d + 3) / 4 : h->d;
  const int64_t per_row = std::max<int64_t>(1, (static_cast<int64_t>(h->dev.sm_count) * 8 + h->n - 1) / h->n);
  const unsigned gx = static_cast<unsigned>(std::max<int64_t>(1, std::min<int64_t>((work + 255) / 256, per_row)));
  const dim3 grid(gx, static_cast<unsigned>(h->n));
  const int biased = (h->flags & SGP_FLAG_BIASED) ? 1 : 0;
  if (vec_ok) sgp::sgp_debias_kernel<4><<<grid, 256, 0, st>>>(d_X, d_W, d_Z, h->d, h->ld, biased, h->d_words + 1);
  else sgp::sgp_debias_kernel<1><<<grid, 256, 0, st>>>(d_X, d_W, d_Z, h->d, h->ld, biased, h->d_words + 1);
  SGP_CUDA_TRY(h, cudaGetLastError());
  return SGP_OK;
}

int sgp_step_host(sgp_handle *h, float *d_X, float *d_W, float *d_M, const float *h_G, float *h_Z, float *d_G,
                  float *d_Z, int64_t k, float lr, float momentum, float weight_decay, int nesterov,
                  int64_t chunk_cols, void *stream) {
  const int rc = validate_step(h, d_X, d_W, d_M, d_G, k, momentum);
  if (rc != SGP_OK) return rc;
  if (h_G == nullptr || (h_Z != nullptr && d_Z == nullptr)) return SGP_ERR_ARG;
  const StepArgs a{d_X, d_W, momentum != 0.0f ? d_M : nullptr, d_G, h_Z != nullptr ? d_Z : nullptr,
                   k, lr, momentum, weight_decay, update_kind(momentum, nesterov)};
  return run_host_step(h, a, h_G, h_Z, chunk_cols, stream);
}

int sgp_step_adam_host(sgp_handle *h, float *d_X, float *d_W, float *d_M1, float *d_M2, const float *h_G, float *h_Z,
                       float *d_G, float *d_Z, int64_t k, int64_t t, float lr, float beta1, float beta2, float eps,
                       float weight_decay, int64_t chunk_cols, void *stream) {
  if (h == nullptr || d_X == nullptr || d_W == nullptr || d_M1 == nullptr || d_M2 == nullptr || d_G == nullptr ||
      h_G == nullptr || (h_Z != nullptr && d_Z == nullptr) || k < 0 || t < 1 || !(beta1 >= 0.0f && beta1 < 1.0f) ||
      !(beta2 >= 0.0f && beta2 < 1.0f) || !(eps >= 0.0f))
    return SGP_ERR_ARG;
  if (check_device(h) != SGP_OK) return check_device(h);
  StepArgs a{d_X, d_W, d_M1, d_G, h_Z != nullptr ? d_Z : nullptr, k, lr, 0.0f, weight_decay, sgp::kUpdAdam};
  a.V = d_M2;
  a.beta1 = beta1;
  a.beta2 = beta2;
  a.eps = eps;
  const double bc1 = 1.0 - std::pow(static_cast<double>(beta1), static_cast<double>(t));
  const double bc2 = 1.0 - std::pow(static_cast<double>(beta2), static_cast<double>(t));
  a.adam_step = static_cast<float>(static_cast<double>(lr) / bc1);
  a.adam_rsqrt_bc2 = static_cast<float>(1.0 / std::sqrt(bc2));
  return run_host_step(h, a, h_G, h_Z, chunk_cols, stream);
}

int sgp_reset(sgp_handle *h, void *stream) {
  if (h == nullptr) return SGP_ERR_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (h->tau > 0) {
    SGP_CUDA_TRY(h, cudaMemsetAsync(h->ring_x, 0, static_cast<size_t>(h->tau) * h->n * h->ld * sizeof(float), st));
    SGP_CUDA_TRY(h, cudaMemsetAsync(h->ring_w, 0, static_cast<size_t>(h->tau) * h->n * sizeof(float), st));
  }
  SGP_CUDA_TRY(h, cudaMemsetAsync(h->d_words, 0, 2 * sizeof(unsigned), st));
  h->seen_status = 0;
  h->diag_valid = false;
  return SGP_OK;
}

int sgp_ring_export(sgp_handle *h, float *d_ring_x, float *d_ring_w, void *stream) {
  if (h == nullptr || d_ring_x == nullptr || d_ring_w == nullptr) return SGP_ERR_ARG;
  if (h->tau == 0) return SGP_ERR_STATE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  SGP_CUDA_TRY(h, cudaMemcpyAsync(d_ring_x, h->ring_x, static_cast<size_t>(h->tau) * h->n * h->ld * sizeof(float),
                                  cudaMemcpyDeviceToDevice, st));
  SGP_CUDA_TRY(h, cudaMemcpyAsync(d_ring_w, h->ring_w, static_cast<size_t>(h->tau) * h->n * sizeof(float),
                                  cudaMemcpyDeviceToDevice, st));
  return SGP_OK;
}

int sgp_ring_import(sgp_handle *h, const float *d_ring_x, const float *d_ring_w, void *stream) {
  if (h == nullptr || d_ring_x == nullptr || d_ring_w == nullptr) return SGP_ERR_ARG;
  if (h->tau == 0) return SGP_ERR_STATE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  SGP_CUDA_TRY(h, cudaMemcpyAsync(h->ring_x, d_ring_x, static_cast<size_t>(h->tau) * h->n * h->ld * sizeof(float),
                                  cudaMemcpyDeviceToDevice, st));
  SGP_CUDA_TRY(h, cudaMemcpyAsync(h->ring_w, d_ring_w, static_cast<size_t>(h->tau) * h->n * sizeof(float),
                                  cudaMemcpyDeviceToDevice, st));
  return SGP_OK;
}

int sgp_colsum(sgp_handle *h, const float *d_A, int include_ring, double *d_out, void *stream) {
  if (h == nullptr || d_A == nullptr || d_out == nullptr) return SGP_ERR_ARG;
  const int rc = check_device(h);
  if (rc != SGP_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // the statistics of this pass are not wanted: they go to the slots sgp_check clears before it runs
  sgp::sgp_colsum_kernel<<<column_grid(h), 256, 0, st>>>(d_A, h->n, h->d, h->ld, include_ring ? h->ring_x : nullptr,
                                                         include_ring ? h->tau * h->n : 0, d_out, nullptr,
                                                         h->d_stats + kDevStatsCheck);
  SGP_CUDA_TRY(h, cudaGetLastError());
  return SGP_OK;
}

int sgp_check(sgp_handle *h, const float *d_X, const float *d_W, const double *d_colsum_ref, double *h_stats,
              void *stream) {
  if (h == nullptr || d_X == nullptr || d_W == nullptr || h_stats == nullptr) return SGP_ERR_ARG;
  const NvtxRange range("sgp_check");
  int rc = check_device(h);
  if (rc != SGP_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  rc = enqueue_check(h, d_X, d_W, d_colsum_ref, st);
  if (rc != SGP_OK) return rc;
  double tmp[sgp::kStatCount];
  SGP_CUDA_TRY(h, cudaMemcpyAsync(tmp, h->d_stats + kDevStatsCheck, sizeof(tmp), cudaMemcpyDeviceToHost, st));
  SGP_CUDA_TRY(h, cudaStreamSynchronize(st));
  unsigned status = 0;
  rc = refresh_status(h, &status);
  if (rc != SGP_OK) return rc;
  h_stats[0] = tmp[sgp::kStatSumW];
  h_stats[1] = tmp[sgp::kStatMinW];
  h_stats[2] = tmp[sgp::kStatNonFinite];
  h_stats[3] = tmp[sgp::kStatTotal];
  h_stats[4] = tmp[sgp::kStatMaxDrift];
  h_stats[5] = tmp[sgp::kStatMaxRelDrift];
  h_stats[6] = std::fabs(tmp[sgp::kStatSumW] - static_cast<double>(h->n));
  h_stats[7] = static_cast<double>(status);
  if (!(tmp[sgp::kStatMinW] > 0.0)) return SGP_ERR_ZERO_WEIGHT;
  if (status & kWaitBits) return SGP_ERR_DEVICE;
  const bool bad = tmp[sgp::kStatNonFinite] > 0.0 || !(h_stats[6] <= 1e-4 * h->n) ||
                   (d_colsum_ref != nullptr && !(tmp[sgp::kStatMaxRelDrift] <= kColumnDriftTol));
  return bad ? SGP_ERR_INVARIANT : SGP_OK;
}

int sgp_get_diagnostics(sgp_handle *h, double *h_param_dev, double *h_consensus, double *h_summary, void *stream) {
  if (h == nullptr) return SGP_ERR_ARG;
  if (!h->diag_valid) return SGP_ERR_STATE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  double tmp[2 * SGP_MAX_NODES];
  const int n = h->n;
  SGP_CUDA_TRY(h, cudaMemcpyAsync(tmp, h->d_stats + kDevStatsDiag, 2 * static_cast<size_t>(n) * sizeof(double), cudaMemcpyDeviceToHost, st));
  SGP_CUDA_TRY(h, cudaStreamSynchronize(st));
  if (h->s_compute != nullptr) SGP_CUDA_TRY(h, cudaStreamSynchronize(h->s_compute));
  for (int i = 0; i < 2 * n; ++i) tmp[i] = std::sqrt(tmp[i]);
  for (int part = 0; part < 2; ++part) {
    double *dst = part == 0 ? h_param_dev : h_consensus;
    double mean = 0.0, mn = tmp[part * n], mx = tmp[part * n];
    for (int i = 0; i < n; ++i) {
      const double v = tmp[part * n + i];
      if (dst) dst[i] = v;
      mean += v;
      mn = std::min(mn, v);
      mx = std::max(mx, v);
    }
    if (h_summary) {
      h_summary[3 * part + 0] = mean / n;
      h_summary[3 * part + 1] = mn;
      h_summary[3 * part + 2] = mx;
    }
  }
  return SGP_OK;
}

int sgp_param_deviation(sgp_handle *h, const float *d_A, double *h_dev, void *stream) {
  if (h == nullptr || d_A == nullptr || h_dev == nullptr) return SGP_ERR_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  double *acc = h->d_stats + kDevStatsDeviation;
  SGP_CUDA_TRY(h, cudaMemsetAsync(acc, 0, static_cast<size_t>(h->n) * sizeof(double), st));
  // tile of n rows x tile_cols columns in shared memory, at most ~64 KB
  int tile_cols = 256;
  while (tile_cols > 32 && static_cast<size_t>(h->n) * tile_cols * 4 > 64 * 1024) tile_cols >>= 1;
  const size_t smem = (static_cast<size_t>(h->n) * tile_cols + tile_cols + h->n) * sizeof(float);
  {
    sgp::KernelInfo ki;
    const int rc = sgp::kernel_info(h->dev.device, reinterpret_cast<const void *>(sgp::sgp_deviation_kernel), smem, &ki,
                                    &h->last_cuda_error);
    if (rc != SGP_OK) return rc;
  }
  const int64_t ntiles = (h->d + tile_cols - 1) / tile_cols;
  const unsigned grid = static_cast<unsigned>(std::min<int64_t>(ntiles, static_cast<int64_t>(h->dev.sm_count) * 2));
  sgp::sgp_deviation_kernel<<<grid, 256, smem, st>>>(d_A, h->n, h->d, h->ld, tile_cols, acc);
  SGP_CUDA_TRY(h, cudaGetLastError());
  SGP_CUDA_TRY(h, cudaMemcpyAsync(h_dev, acc, static_cast<size_t>(h->n) * sizeof(double), cudaMemcpyDeviceToHost, st));
  SGP_CUDA_TRY(h, cudaStreamSynchronize(st));
  for (int i = 0; i < h->n; ++i) h_dev[i] = std::sqrt(h_dev[i]);
  return SGP_OK;
}

int sgp_set_option(sgp_handle *h, const char *key, int64_t value) {
  if (h == nullptr || key == nullptr || value < 0) return SGP_ERR_ARG;
  if (std::strcmp(key, "variant") == 0) {
    if (value > 5) return SGP_ERR_ARG;
    h->opt_variant = value;
  } else if (std::strcmp(key, "cluster") == 0) {
    if (value != 0 && value != 1 && value != 2 && value != 4) return SGP_ERR_ARG;
    h->opt_cluster = value;
  } else if (std::strcmp(key, "tile_cols") == 0) {
    if (value % 4 != 0 || value > 4096) return SGP_ERR_ARG;
    h->opt_tile_cols = value;
  } else if (std::strcmp(key, "ctas_per_sm") == 0) {
    if (value > 16) return SGP_ERR_ARG;
    h->opt_ctas_per_sm = value;
  } else if (std::strcmp(key, "stages") == 0) {
    if (value > 8) return SGP_ERR_ARG;
    h->opt_stages = value;
  } else if (std::strcmp(key, "wait_limit_ms") == 0) {
    if (value > 10000) return SGP_ERR_ARG;
    h->opt_wait_limit_ms = value;
  } else if (std::strcmp(key, "inject_stall") == 0) {
    if (value > 1) return SGP_ERR_ARG;
    h->opt_inject_stall = value;
  } else if (std::strcmp(key, "single_buffer") == 0) {
    if (value > 2) return SGP_ERR_ARG;
    h->opt_single_buffer = value;
  } else if (std::strcmp(key, "lockstep") == 0) {
    if (value != 0 && value != 1 && value != 2 && value != 4) return SGP_ERR_ARG;
    h->opt_lockstep = value;
  } else if (std::strcmp(key, "l2_hint") == 0) {
    if (value > 4) return SGP_ERR_ARG;
    h->opt_l2_hint = value;
  } else if (std::strcmp(key, "send_period") == 0) {
    if (value < 1 || value > (1 << 20)) return SGP_ERR_ARG;
    h->opt_send_period = value;
#ifdef SGP_CHECKED
  } else if (std::strcmp(key, "poke_table") == 0) {
    // Bounds-checked build only, test hook: overwrites the first sender index of slot 0's table with `value`, so that
    // a test can watch an out-of-range index being caught (status bit, access skipped) instead of dereferenced.
    const int32_t bad = static_cast<int32_t>(value);
    if (cudaMemcpy(h->d_col + h->off_nnz[0], &bad, sizeof(bad), cudaMemcpyHostToDevice) != cudaSuccess) {
      (void)cudaGetLastError();
      return SGP_ERR_CUDA;
    }
    if (h->const_ok[0]) h->const_tables[0].col[0] = bad;
#endif
  } else if (std::strcmp(key, "diagnostics") == 0) {
    if (value > 1) return SGP_ERR_ARG;
    h->opt_diagnostics = value;
  } else if (std::strcmp(key, "check_steps") == 0) {
    if (value > 1) return SGP_ERR_ARG;
    if (value == 1 && h->d_expect == nullptr) {
      if (check_device(h) != SGP_OK) return SGP_ERR_STATE;
      if (cudaMalloc(&h->d_expect, static_cast<size_t>(h->d) * sizeof(double)) != cudaSuccess) {
        (void)cudaGetLastError();
        h->d_expect = nullptr;
        return SGP_ERR_ALLOC;
      }
    }
    h->opt_check_steps = value;
  } else {
    return SGP_ERR_ARG;
  }
  return SGP_OK;
}

int sgp_get_option(const sgp_handle *h, const char *key, int64_t *value) {
  if (h == nullptr || key == nullptr || value == nullptr) return SGP_ERR_ARG;
  if (std::strcmp(key, "variant") == 0) *value = h->opt_variant;
  else if (std::strcmp(key, "tile_cols") == 0) *value = h->opt_tile_cols;
  else if (std::strcmp(key, "ctas_per_sm") == 0) *value = h->opt_ctas_per_sm;
  else if (std::strcmp(key, "stages") == 0) *value = h->opt_stages;
  else if (std::strcmp(key, "l2_hint") == 0) *value = h->opt_l2_hint;
  else if (std::strcmp(key, "single_buffer") == 0) *value = h->opt_single_buffer;
  else if (std::strcmp(key, "lockstep") == 0) *value = h->opt_lockstep;
  else if (std::strcmp(key, "wait_limit_ms") == 0) *value = h->opt_wait_limit_ms;
  else if (std::strcmp(key, "inject_stall") == 0) *value = h->opt_inject_stall;
  else if (std::strcmp(key, "send_period") == 0) *value = h->opt_send_period;
  else if (std::strcmp(key, "cluster") == 0) *value = h->opt_cluster;
  else if (std::strcmp(key, "diagnostics") == 0) *value = h->opt_diagnostics;
  else if (std::strcmp(key, "check_steps") == 0) *value = h->opt_check_steps;
  else if (std::strcmp(key, "last_variant") == 0) *value = h->last.variant;
  else if (std::strcmp(key, "last_grid") == 0) *value = h->last.grid;
  else if (std::strcmp(key, "launches") == 0) *value = h->launches;
  else if (std::strcmp(key, "last_smem") == 0) *value = h->last.smem;
  else if (std::strcmp(key, "last_tile_cols") == 0) *value = h->last.tile_cols;
  else if (std::strcmp(key, "last_lockstep") == 0) *value = h->last.lockstep;
  else return SGP_ERR_ARG;
  return SGP_OK;
}

int sgp_device_status(sgp_handle *h, unsigned *status) {
  if (h == nullptr || status == nullptr) return SGP_ERR_ARG;
  SGP_CUDA_TRY(h, cudaDeviceSynchronize());
  return refresh_status(h, status);
}

int sgp_last_cuda_error(const sgp_handle *h) { return h == nullptr ? 0 : h->last_cuda_error; }

}  // extern "C"
