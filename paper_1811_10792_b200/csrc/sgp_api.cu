// C ABI of the fused SGP step (see include/sgp.h): handle management, argument validation, launch
// configuration and dispatch.  All arithmetic of the method lives in the kernels.
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstring>
#include <map>
#include <mutex>
#include <new>
#include <utility>
#include <vector>

#include "aux_kernels.cuh"
#include "schedule.h"
#include "sgp.h"
#include "step_kernels.cuh"

using sgp::ConstTable;
using sgp::StepParams;

struct sgp_handle {
  int n = 0;
  int64_t d = 0, ld = 0;
  int tau = 0;
  unsigned flags = 0;
  int device = 0;
  int sm_count = 0;
  int smem_optin = 0;
  sgp_schedule *sched = nullptr;
  // device copy of every slot's CSR, concatenated; offsets in elements
  int32_t *d_rowptr = nullptr;
  int32_t *d_col = nullptr;
  float *d_val = nullptr;
  std::vector<int64_t> off_rowptr, off_nnz;
  std::vector<ConstTable> const_tables;  // valid where const_ok[slot]
  std::vector<char> const_ok;
  float *ring_x = nullptr;   // tau * n * ld
  float *ring_w = nullptr;   // tau * n
  unsigned *d_words = nullptr;  // [0] ticket, [1] status
  double *d_stats = nullptr;    // 4 doubles for sgp_check, then SGP_MAX_NODES doubles for sgp_param_deviation
  int64_t opt_variant = 0, opt_tile_cols = 0, opt_ctas_per_sm = 0, opt_stages = 0, opt_l2_hint = 0, opt_single_buffer = 0, opt_wait_limit_ms = 0,
          opt_inject_stall = 0;
  int64_t last_variant = 0, last_grid = 0, last_smem = 0, last_tile_cols = 0;   // of the most recent step launch
  int64_t launches = 0;                                                          // step kernels launched so far
  cudaStream_t s_h2d = nullptr, s_compute = nullptr, s_d2h = nullptr;
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

inline int floor_log2(int64_t v) {
  int l = 0;
  while ((int64_t{1} << (l + 1)) <= v) ++l;
  return l;
}

void free_handle(sgp_handle *h) {
  if (h == nullptr) return;
  cudaFree(h->d_rowptr);
  cudaFree(h->d_col);
  cudaFree(h->d_val);
  cudaFree(h->ring_x);
  cudaFree(h->ring_w);
  cudaFree(h->d_words);
  cudaFree(h->d_stats);
  for (cudaEvent_t e : h->ev_in) cudaEventDestroy(e);
  for (cudaEvent_t e : h->ev_done) cudaEventDestroy(e);
  if (h->s_h2d) cudaStreamDestroy(h->s_h2d);
  if (h->s_compute) cudaStreamDestroy(h->s_compute);
  if (h->s_d2h) cudaStreamDestroy(h->s_d2h);
  delete h->sched;
  delete h;
}

using StepKernel = void (*)(const StepParams, const ConstTable);

// Per-kernel facts that do not change during the process: registers, static shared memory, and the
// largest dynamic shared-memory size already enabled (so the attribute calls leave the launch path).
struct KernelInfo {
  int num_regs = 0;
  size_t static_smem = 0;
  size_t enabled_smem = 48 * 1024;
};
std::mutex g_kernel_info_mutex;
std::map<std::pair<int, const void *>, KernelInfo> g_kernel_info;   // function attributes are per device

int kernel_info(sgp_handle *h, const void *kern, size_t smem, KernelInfo *out) {
  std::lock_guard<std::mutex> lock(g_kernel_info_mutex);
  const std::pair<int, const void *> key(h->device, kern);
  auto it = g_kernel_info.find(key);
  if (it == g_kernel_info.end()) {
    cudaFuncAttributes fa;
    SGP_CUDA_TRY(h, cudaFuncGetAttributes(&fa, kern));
    KernelInfo ki;
    ki.num_regs = fa.numRegs;
    ki.static_smem = fa.sharedSizeBytes;
    it = g_kernel_info.emplace(key, ki).first;
  }
  if (smem > it->second.enabled_smem) {
    SGP_CUDA_TRY(h, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
    it->second.enabled_smem = smem;
  }
  *out = it->second;
  return SGP_OK;
}

template <int VEC, int UPD>
StepKernel pick_regs_flags(bool has_z, bool has_ring) {
  if (has_z) return has_ring ? sgp::sgp_step_regs_kernel<VEC, UPD, true, true> : sgp::sgp_step_regs_kernel<VEC, UPD, true, false>;
  return has_ring ? sgp::sgp_step_regs_kernel<VEC, UPD, false, true> : sgp::sgp_step_regs_kernel<VEC, UPD, false, false>;
}
template <int VEC>
StepKernel pick_regs(int upd, bool has_z, bool has_ring) {
  switch (upd) {
    case sgp::kUpdSgd: return pick_regs_flags<VEC, sgp::kUpdSgd>(has_z, has_ring);
    case sgp::kUpdHeavyBall: return pick_regs_flags<VEC, sgp::kUpdHeavyBall>(has_z, has_ring);
    case sgp::kUpdNesterov: return pick_regs_flags<VEC, sgp::kUpdNesterov>(has_z, has_ring);
    default: return pick_regs_flags<VEC, sgp::kUpdAdam>(has_z, has_ring);
  }
}

using TmaKernel = void (*)(const StepParams, const ConstTable, const sgp::TmaMaps, const int, const int);

template <int UPD>
TmaKernel pick_tma_flags(bool has_z, bool has_ring) {
  if (has_z) return has_ring ? sgp::sgp_step_tma_kernel<UPD, true, true> : sgp::sgp_step_tma_kernel<UPD, true, false>;
  return has_ring ? sgp::sgp_step_tma_kernel<UPD, false, true> : sgp::sgp_step_tma_kernel<UPD, false, false>;
}
TmaKernel pick_tma(int upd, bool has_z, bool has_ring) {
  switch (upd) {
    case sgp::kUpdSgd: return pick_tma_flags<sgp::kUpdSgd>(has_z, has_ring);
    case sgp::kUpdHeavyBall: return pick_tma_flags<sgp::kUpdHeavyBall>(has_z, has_ring);
    case sgp::kUpdNesterov: return pick_tma_flags<sgp::kUpdNesterov>(has_z, has_ring);
    default: return pick_tma_flags<sgp::kUpdAdam>(has_z, has_ring);
  }
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

// Fills the launch-independent part of the kernel arguments for step a.k.
void fill_params(const sgp_handle *h, const StepArgs &a, int64_t c0, int64_t c1, bool update_w, StepParams *out) {
  const int64_t slot = a.k % h->sched->period();
  const SgpStepCsr &csr = h->sched->slot(a.k);
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
  }
  p.ld = h->ld;
  p.col_begin = c0;
  p.col_end = c1;
  p.n = h->n;
  p.nnz = static_cast<int>(csr.col.size());
  p.update_w = update_w ? 1 : 0;
  p.uniform_parts = 0;
  p.lr = a.lr;
  p.momentum = a.momentum;
  p.wd = a.wd;
  p.rowptr = h->d_rowptr + h->off_rowptr[static_cast<size_t>(slot)];
  p.col = h->d_col + h->off_nnz[static_cast<size_t>(slot)];
  p.val = h->d_val + h->off_nnz[static_cast<size_t>(slot)];
  p.ticket = h->d_words;
  p.status = h->d_words + 1;
  *out = p;
}

// Launch plan of one step: which kernel, how wide a tile, how deep a pipeline, how many CTAs per SM.
struct Plan {
  int variant;        // 1 register-staged, 2 TMA with tensor maps, 3 TMA with per-row bulk copies
  int64_t tile_cols;  // 0 = kernel default
  int stages;
  int cps;
};

// Register-staged kernel: one exchange tile (two barriers per tile) where that keeps the row segments long
// (n = 64: 1 KB segments 0.95 against 0.92; n = 80: 0.97 against 0.82; n = 96: 512 B 0.92 against 0.89;
// n > 128: 256 B 0.91 against 0.70); two tiles and one barrier elsewhere (n = 112, 128: 0.94 against 0.92).
bool auto_single_buffer(int n) { return (n > 32 && n <= 104) || n > 128; }

size_t table_smem_bytes(const sgp_handle *h, int nnz) { return (static_cast<size_t>(h->n) + 1 + 2 * static_cast<size_t>(nnz)) * 4; }

// Tile width of the register-staged kernel (128-bit path): row segments of at least 1 KB and about 2048
// vector items per tile, shrunk until the exchange tile(s) plus `fixed` bytes stay near 80 KB per CTA --
// two resident CTAs then leave about half of the SM's 256 KB to the L1 that tracks the loads in flight
// (measured: n = 48 at 2 x 100 KB reaches 0.74 of the copy bandwidth, at 2 x 50 KB 0.93).
int64_t regs_tile_cols(const sgp_handle *h, size_t fixed) {
  int64_t cols = std::max<int64_t>(256, int64_t{4} << floor_log2(std::max<int64_t>(1, 2048 / h->n)));
  const size_t copies = auto_single_buffer(h->n) ? 1 : 2;
  const size_t cap = (copies == 1 ? 88 : 80) * 1024;     // n = 80 at 85 KB: 0.97; n = 96 at 102 KB: 0.79
  while (cols > 32 && copies * static_cast<size_t>(h->n) * cols * 4 + fixed > cap) cols >>= 1;
  return cols;
}

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
    const size_t fixed = 16 * sizeof(uint64_t) + 3 * static_cast<size_t>(h->n) * 4 + 1024 +
                         (table_smem_bytes(h, nnz) <= 40 * 1024 ? table_smem_bytes(h, nnz) : 0);
    const size_t per_kb = static_cast<size_t>(arrays) * h->n * 1024;   // one stage at 1 KB per row segment
    const size_t full_sm = 224 * 1024;
    // The pipelined kernel has ONE consumer group, so its gather is on the critical path: it is only used
    // for sparse steps (at most three in-neighbours per node on average; with five it drops to 0.94, with
    // nine to 0.88, while the register-staged kernel holds 0.98 and 0.95).
    const bool sparse = static_cast<int64_t>(nnz) <= 3 * static_cast<int64_t>(h->n);
    if (!sparse) {
      pl.tile_cols = regs_tile_cols(h, fixed);
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
      pl.tile_cols = regs_tile_cols(h, fixed);
    }
  }
  if (h->opt_variant > 0 && (h->opt_variant == 1) != (pl.variant == 1)) {
    // the caller forces the other kernel family: take that family's defaults
    if (h->opt_variant == 1) {
      pl = Plan{1, vec ? regs_tile_cols(h, 4 * 1024) : 0, 2, 0};
    } else {
      pl = Plan{static_cast<int>(h->opt_variant), 256, 2, 2};
    }
  }
  if (h->opt_variant > 0) pl.variant = static_cast<int>(h->opt_variant);
  if (h->opt_tile_cols > 0) pl.tile_cols = h->opt_tile_cols;
  if (h->opt_stages > 0) pl.stages = static_cast<int>(h->opt_stages);
  if (h->opt_ctas_per_sm > 0) pl.cps = static_cast<int>(h->opt_ctas_per_sm);
  return pl;
}

// One launch of the register-staged kernel over columns [c0, c1) with vector width vec.
int launch_regs(sgp_handle *h, const StepArgs &a, const Plan &pl, int64_t c0, int64_t c1, int vec, bool update_w,
                cudaStream_t stream) {
  const int64_t slot = a.k % h->sched->period();
  StepParams p{};
  fill_params(h, a, c0, c1, update_w, &p);

  // tile width: the plan's, else about four items per thread; at least 128 bytes per row segment
  const int64_t ncols = c1 - c0;
  const int min_tv = vec == 4 ? 8 : 32;
  int64_t tv = int64_t{1} << floor_log2(std::max<int64_t>(1, sgp::kThreads * 4 / h->n));
  if (pl.tile_cols > 0) tv = int64_t{1} << floor_log2(std::max<int64_t>(1, pl.tile_cols / vec));
  tv = std::max<int64_t>(tv, min_tv);
  // short rows: narrower tiles until there is about a tile per SM (launch-latency regime)
  if (h->opt_tile_cols == 0)
    while (tv > min_tv && tv * vec > 128 && (ncols + tv * vec - 1) / (tv * vec) < h->sm_count) tv >>= 1;
  const size_t table_bytes = table_smem_bytes(h, p.nnz);
  if (h->const_ok[static_cast<size_t>(slot)]) p.table_mode = 0;
  else p.table_mode = table_bytes <= 40 * 1024 ? 1 : 2;
  const bool uniform = h->tau == 0 && h->sched->slot(a.k).uniform_rows;
  // large n: one exchange tile (two barriers per tile) so that the row segments can stay twice as long
  p.single_buffer = h->opt_single_buffer == 1 ? 1 : (h->opt_single_buffer == 2 ? 0 : (auto_single_buffer(h->n) ? 1 : 0));
  size_t smem = 0;
  for (;;) {
    p.uniform_parts = uniform ? static_cast<int>(std::max<int64_t>(1, std::min<int64_t>(8, sgp::kThreads / tv))) : 0;
    smem = (p.single_buffer ? 1 : 2) * static_cast<size_t>(h->n) * tv * vec * 4 + 3 * static_cast<size_t>(h->n) * 4 +
           static_cast<size_t>(p.uniform_parts) * tv * vec * 4 + (p.table_mode < 2 ? table_bytes : 0);
    if (smem <= 110 * 1024 || tv <= min_tv) break;
    tv >>= 1;
  }
  if (smem > static_cast<size_t>(h->smem_optin)) return SGP_ERR_ARG;
  p.log2_tile_vecs = floor_log2(tv);
  const int64_t tile_cols = tv * vec;
  const int64_t ntiles = (ncols + tile_cols - 1) / tile_cols;
  StepKernel kern = vec == 4 ? pick_regs<4>(a.upd, a.Z != nullptr, h->tau > 0)
                             : pick_regs<1>(a.upd, a.Z != nullptr, h->tau > 0);
  KernelInfo ki;
  {
    const int rc = kernel_info(h, reinterpret_cast<const void *>(kern), smem, &ki);
    if (rc != SGP_OK) return rc;
  }
  int cps = pl.cps;
  if (cps <= 0) {
    // Persistent grid of exactly one wave: CTAs resident per SM by registers, shared memory and threads.
    // (Computed here rather than asked of the occupancy calculator, whose answer depends on the
    // shared-memory carve-out it assumes; the hardware picks the carve-out that fits the launch.)
    const int regs_per_cta = ((ki.num_regs + 7) / 8 * 8) * sgp::kThreads;
    const int by_regs = regs_per_cta > 0 ? 65536 / regs_per_cta : 8;
    const int by_smem = static_cast<int>((227 * 1024) / (smem + ki.static_smem + 1024));
    cps = std::max(1, std::min({by_regs, by_smem, 2048 / sgp::kThreads}));
  }
  const int64_t grid = std::min<int64_t>(ntiles, static_cast<int64_t>(h->sm_count) * cps);
  static const ConstTable kEmptyTable{};
  const ConstTable &ct = p.table_mode == 0 ? h->const_tables[static_cast<size_t>(slot)] : kEmptyTable;
  kern<<<static_cast<unsigned>(grid), sgp::kThreads, smem, stream>>>(p, ct);
  SGP_CUDA_TRY(h, cudaGetLastError());
  h->last_variant = 1;
  ++h->launches;
  h->last_grid = grid;
  h->last_smem = static_cast<int64_t>(smem);
  h->last_tile_cols = tile_cols;
  return SGP_OK;
}

using EncodeTiledFn = CUresult (*)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                   const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// Tensor map of an n x d fp32 array with row pitch ld whose box is (box_cols x n); cached per pointer.
// Returns false when the driver entry point is unavailable or the encoding is rejected.
bool get_tensor_map(sgp_handle *h, const float *base, int box_cols, CUtensorMap *out) {
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
  const int64_t slot = a.k % h->sched->period();
  StepParams p{};
  fill_params(h, a, c0, c1, update_w, &p);
  const bool has_m = a.M != nullptr, has_v = a.V != nullptr, has_ring = h->tau > 0;
  const int arrays = 2 + (has_m ? 1 : 0) + (has_v ? 1 : 0) + (has_ring ? 1 : 0);
  int64_t tv = int64_t{1} << floor_log2(std::max<int64_t>(1, (pl.tile_cols > 0 ? pl.tile_cols : 256) / 4));
  tv = std::max<int64_t>(tv, 8);
  int stages = std::max(1, pl.stages);
  const int cps = pl.cps > 0 ? pl.cps : 2;
  const size_t table_bytes = table_smem_bytes(h, p.nnz);
  if (h->const_ok[static_cast<size_t>(slot)]) p.table_mode = 0;
  else p.table_mode = table_bytes <= 40 * 1024 ? 1 : 2;
  const bool uniform = h->tau == 0 && h->sched->slot(a.k).uniform_rows;
  size_t fixed = 16 * sizeof(uint64_t) + 3 * static_cast<size_t>(h->n) * 4 + (p.table_mode < 2 ? table_bytes : 0);
  const size_t budget = std::min<size_t>(static_cast<size_t>(h->smem_optin), (228 * 1024) / static_cast<size_t>(cps) - 2048);
  size_t smem = 0;
  for (;;) {
    p.uniform_parts = uniform ? static_cast<int>(std::max<int64_t>(1, std::min<int64_t>(8, sgp::kTmaConsumers / tv))) : 0;
    smem = static_cast<size_t>(stages) * arrays * h->n * tv * 16 + fixed + static_cast<size_t>(p.uniform_parts) * tv * 16;
    if (smem <= budget) break;
    if (h->opt_stages == 0 && stages > 2) --stages;
    else if (h->opt_tile_cols == 0 && tv > 8) tv >>= 1;
    else return SGP_ERR_STATE;
  }
  p.log2_tile_vecs = floor_log2(tv);
  const int64_t tile_cols = tv * 4;
  const int64_t ntiles = (c1 - c0 + tile_cols - 1) / tile_cols;
  const int64_t grid = std::min<int64_t>(ntiles, static_cast<int64_t>(h->sm_count) * cps);
  p.wait_limit_ms = h->opt_wait_limit_ms > 0 ? static_cast<int>(h->opt_wait_limit_ms) : 2000;
  p.inject_stall = h->opt_inject_stall ? 1 : 0;
  p.l2_hint = h->opt_l2_hint == 2 ? 0 : (h->opt_l2_hint == 0 ? 3 : static_cast<int>(h->opt_l2_hint));
  TmaKernel kern = pick_tma(a.upd, a.Z != nullptr, has_ring);
  {
    KernelInfo ki;
    const int rc = kernel_info(h, reinterpret_cast<const void *>(kern), smem, &ki);
    if (rc != SGP_OK) return rc;
  }
  static const ConstTable kEmptyTable{};
  const ConstTable &ct = p.table_mode == 0 ? h->const_tables[static_cast<size_t>(slot)] : kEmptyTable;
  // 2-D tensor maps (one copy per array per tile) when the box fits; else one bulk copy per row segment
  sgp::TmaMaps maps;
  std::memset(&maps, 0, sizeof(maps));
  bool use_maps = pl.variant == 2 && tile_cols <= 256 && tile_cols * 4 % 128 == 0;
  if (use_maps) use_maps = get_tensor_map(h, a.X, static_cast<int>(tile_cols), &maps.x);
  if (use_maps) use_maps = get_tensor_map(h, a.G, static_cast<int>(tile_cols), &maps.g);
  if (use_maps && has_m) use_maps = get_tensor_map(h, a.M, static_cast<int>(tile_cols), &maps.m);
  if (use_maps && has_v) use_maps = get_tensor_map(h, a.V, static_cast<int>(tile_cols), &maps.v);
  if (use_maps && has_ring) use_maps = get_tensor_map(h, p.ring_x, static_cast<int>(tile_cols), &maps.r);
  kern<<<static_cast<unsigned>(grid), sgp::kTmaThreads, smem, stream>>>(p, ct, maps, stages, use_maps ? 1 : 0);
  SGP_CUDA_TRY(h, cudaGetLastError());
  h->last_variant = use_maps ? 2 : 3;
  ++h->launches;
  h->last_grid = grid;
  h->last_smem = static_cast<int64_t>(smem);
  h->last_tile_cols = tile_cols;
  return SGP_OK;
}

// The whole step over columns [c0, c1): 128-bit kernel on the aligned bulk, scalar kernel on what is left.
int launch_step_range(sgp_handle *h, const StepArgs &a, int64_t c0, int64_t c1, bool update_w, cudaStream_t stream) {
  const bool vec_ok = aligned16(a.X) && aligned16(a.G) && (a.M == nullptr || aligned16(a.M)) &&
                      (a.V == nullptr || aligned16(a.V)) && (a.Z == nullptr || aligned16(a.Z)) && (h->ld % 4 == 0) &&
                      (c0 % 4 == 0);
  const int64_t vec_end = vec_ok ? c0 + ((c1 - c0) & ~int64_t{3}) : c0;
  const int arrays = 2 + (a.M != nullptr ? 1 : 0) + (a.V != nullptr ? 1 : 0) + (h->tau > 0 ? 1 : 0);
  const int nnz = static_cast<int>(h->sched->slot(a.k).col.size());
  if (vec_end > c0) {
    Plan pl = make_plan(h, arrays, a.M != nullptr, nnz, true);
    // short rows (fewer 1 KB tiles than SMs): the register kernel with narrow tiles spreads them better
    if (h->opt_variant == 0 && pl.variant >= 2 && (vec_end - c0) < int64_t{256} * h->sm_count) pl = Plan{1, 256, 2, 0};
    int rc = SGP_ERR_STATE;
    if (pl.variant >= 2) rc = launch_tma(h, a, pl, c0, vec_end, update_w && vec_end == c1, stream);
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

// The handle's tables and ring live on the device that was current at sgp_create.
int check_device(const sgp_handle *h) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) {
    (void)cudaGetLastError();
    return SGP_ERR_CUDA;
  }
  return dev == h->device ? SGP_OK : SGP_ERR_STATE;
}

int validate_step(const sgp_handle *h, const float *X, const float *W, const float *M, const float *G, int64_t k,
                  float momentum) {
  if (h == nullptr || X == nullptr || W == nullptr || G == nullptr || k < 0) return SGP_ERR_ARG;
  if (momentum != 0.0f && M == nullptr) return SGP_ERR_ARG;
  return check_device(h);
}

// Builds the device tables of a compiled schedule and installs them (and the schedule) in the handle,
// releasing whatever the handle held before.  The caller guarantees that no kernel still reads the old tables.
int upload_schedule(sgp_handle *h, sgp_schedule *sched) {
  std::vector<int32_t> rowptr, col;
  std::vector<float> val;
  std::vector<int64_t> off_rowptr, off_nnz;
  std::vector<ConstTable> const_tables;
  std::vector<char> const_ok;
  for (int64_t s = 0; s < sched->period(); ++s) {
    const SgpStepCsr &c = sched->steps[static_cast<size_t>(s)];
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
  if (h->sched != sched) delete h->sched;
  h->sched = sched;
  return SGP_OK;
}

}  // namespace

extern "C" {

int sgp_version(void) { return 100; }

const char *sgp_strerror(int code) {
  switch (code) {
    case SGP_OK: return "ok";
    case SGP_ERR_ARG: return "invalid argument";
    case SGP_ERR_GRAPH: return "schedule is not a column-stochastic digraph with self-loops";
    case SGP_ERR_CUDA: return "CUDA runtime error";
    case SGP_ERR_ALLOC: return "allocation failed";
    case SGP_ERR_STATE: return "call not valid for this handle";
    case SGP_ERR_DEVICE: return "a kernel gave up a bounded wait";
    default: return "unknown error";
  }
}

int sgp_create(sgp_handle **out, int n, int64_t d, int64_t ld, const sgp_graph_desc *g, int tau, unsigned flags) {
  if (out == nullptr) return SGP_ERR_ARG;
  *out = nullptr;
  if (n < 1 || n > SGP_MAX_NODES || d < 1 || ld < d || tau < 0 || tau > 64 || g == nullptr || flags != SGP_FLAG_NONE)
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

  auto fail = [&](int code, cudaError_t e) {
    const int err = static_cast<int>(e);
    free_handle(h);
    (void)cudaGetLastError();
    (void)err;
    return code;
  };
  cudaError_t e = cudaGetDevice(&h->device);
  if (e != cudaSuccess) return fail(SGP_ERR_CUDA, e);
  e = cudaDeviceGetAttribute(&h->sm_count, cudaDevAttrMultiProcessorCount, h->device);
  if (e != cudaSuccess) return fail(SGP_ERR_CUDA, e);
  e = cudaDeviceGetAttribute(&h->smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, h->device);
  if (e != cudaSuccess) return fail(SGP_ERR_CUDA, e);

  {
    const int rc_up = upload_schedule(h, sched);
    if (rc_up != SGP_OK) return fail(rc_up, cudaSuccess);
  }
  e = cudaMalloc(&h->d_words, 2 * sizeof(unsigned));
  if (e != cudaSuccess) return fail(SGP_ERR_ALLOC, e);
  e = cudaMalloc(&h->d_stats, (4 + SGP_MAX_NODES) * sizeof(double));
  if (e != cudaSuccess) return fail(SGP_ERR_ALLOC, e);
  if (tau > 0) {
    e = cudaMalloc(&h->ring_x, static_cast<size_t>(tau) * n * ld * sizeof(float));
    if (e != cudaSuccess) return fail(SGP_ERR_ALLOC, e);
    e = cudaMalloc(&h->ring_w, static_cast<size_t>(tau) * n * sizeof(float));
    if (e != cudaSuccess) return fail(SGP_ERR_ALLOC, e);
    e = cudaMemset(h->ring_x, 0, static_cast<size_t>(tau) * n * ld * sizeof(float));
    if (e != cudaSuccess) return fail(SGP_ERR_CUDA, e);
    e = cudaMemset(h->ring_w, 0, static_cast<size_t>(tau) * n * sizeof(float));
    if (e != cudaSuccess) return fail(SGP_ERR_CUDA, e);
  }
  e = cudaMemset(h->d_words, 0, 2 * sizeof(unsigned));
  if (e != cudaSuccess) return fail(SGP_ERR_CUDA, e);
  e = cudaDeviceSynchronize();
  if (e != cudaSuccess) return fail(SGP_ERR_CUDA, e);
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
  return launch_step_range(h, a, 0, h->d, true, static_cast<cudaStream_t>(stream));
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
  return launch_step_range(h, a, 0, h->d, true, static_cast<cudaStream_t>(stream));
}

int sgp_debias(sgp_handle *h, const float *d_X, const float *d_W, float *d_Z, void *stream) {
  if (h == nullptr || d_X == nullptr || d_W == nullptr || d_Z == nullptr) return SGP_ERR_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const bool vec_ok = aligned16(d_X) && aligned16(d_Z) && (h->ld % 4 == 0);
  const int64_t work = vec_ok ? (h->d + 3) / 4 : h->d;
  const int64_t per_row = std::max<int64_t>(1, (static_cast<int64_t>(h->sm_count) * 8 + h->n - 1) / h->n);
  const unsigned gx = static_cast<unsigned>(std::max<int64_t>(1, std::min<int64_t>((work + 255) / 256, per_row)));
  const dim3 grid(gx, static_cast<unsigned>(h->n));
  if (vec_ok) sgp::sgp_debias_kernel<4><<<grid, 256, 0, st>>>(d_X, d_W, d_Z, h->d, h->ld);
  else sgp::sgp_debias_kernel<1><<<grid, 256, 0, st>>>(d_X, d_W, d_Z, h->d, h->ld);
  SGP_CUDA_TRY(h, cudaGetLastError());
  return SGP_OK;
}

int sgp_step_host(sgp_handle *h, float *d_X, float *d_W, float *d_M, const float *h_G, float *h_Z, float *d_G,
                  float *d_Z, int64_t k, float lr, float momentum, float weight_decay, int nesterov,
                  int64_t chunk_cols) {
  int rc = validate_step(h, d_X, d_W, d_M, d_G, k, momentum);
  if (rc != SGP_OK) return rc;
  if (h_G == nullptr || (h_Z != nullptr && d_Z == nullptr)) return SGP_ERR_ARG;
  if (h->s_h2d == nullptr) {
    SGP_CUDA_TRY(h, cudaStreamCreateWithFlags(&h->s_h2d, cudaStreamNonBlocking));
    SGP_CUDA_TRY(h, cudaStreamCreateWithFlags(&h->s_compute, cudaStreamNonBlocking));
    SGP_CUDA_TRY(h, cudaStreamCreateWithFlags(&h->s_d2h, cudaStreamNonBlocking));
  }
  // default chunk: about 64 MB of gradient per chunk, a multiple of 1024 columns
  if (chunk_cols <= 0) chunk_cols = std::max<int64_t>(1024, (int64_t{64} << 20) / (4 * h->n) / 1024 * 1024);
  chunk_cols = (chunk_cols + 3) / 4 * 4;
  const int64_t nchunks = (h->d + chunk_cols - 1) / chunk_cols;
  while (static_cast<int64_t>(h->ev_in.size()) < nchunks) {
    cudaEvent_t a = nullptr, b = nullptr;
    SGP_CUDA_TRY(h, cudaEventCreateWithFlags(&a, cudaEventDisableTiming));
    h->ev_in.push_back(a);
    SGP_CUDA_TRY(h, cudaEventCreateWithFlags(&b, cudaEventDisableTiming));
    h->ev_done.push_back(b);
  }
  // earlier work of the caller on the legacy/default stream must be visible
  SGP_CUDA_TRY(h, cudaDeviceSynchronize());
  const StepArgs a{d_X, d_W, momentum != 0.0f ? d_M : nullptr, d_G, h_Z != nullptr ? d_Z : nullptr,
                   k, lr, momentum, weight_decay, update_kind(momentum, nesterov)};
  const size_t pitch = static_cast<size_t>(h->ld) * sizeof(float);
  for (int64_t c = 0; c < nchunks; ++c) {
    const int64_t c0 = c * chunk_cols, c1 = std::min(h->d, c0 + chunk_cols);
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
  return SGP_OK;
}

int sgp_reset(sgp_handle *h, void *stream) {
  if (h == nullptr) return SGP_ERR_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (h->tau > 0) {
    SGP_CUDA_TRY(h, cudaMemsetAsync(h->ring_x, 0, static_cast<size_t>(h->tau) * h->n * h->ld * sizeof(float), st));
    SGP_CUDA_TRY(h, cudaMemsetAsync(h->ring_w, 0, static_cast<size_t>(h->tau) * h->n * sizeof(float), st));
  }
  SGP_CUDA_TRY(h, cudaMemsetAsync(h->d_words, 0, 2 * sizeof(unsigned), st));
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

int sgp_check(sgp_handle *h, const float *d_X, const float *d_W, double *h_stats, void *stream) {
  if (h == nullptr || d_X == nullptr || d_W == nullptr || h_stats == nullptr) return SGP_ERR_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  SGP_CUDA_TRY(h, cudaMemsetAsync(h->d_stats, 0, 4 * sizeof(double), st));
  const unsigned grid = static_cast<unsigned>(h->sm_count * 8);
  sgp::sgp_scan_kernel<<<grid, 256, 0, st>>>(d_X, h->n, h->d, h->ld, h->d_stats);
  if (h->tau > 0) sgp::sgp_scan_kernel<<<grid, 256, 0, st>>>(h->ring_x, h->tau * h->n, h->d, h->ld, h->d_stats);
  sgp::sgp_weight_scan_kernel<<<1, 256, 0, st>>>(d_W, h->n, h->ring_w, h->tau * h->n, h->d_stats);
  SGP_CUDA_TRY(h, cudaGetLastError());
  double tmp[4];
  SGP_CUDA_TRY(h, cudaMemcpyAsync(tmp, h->d_stats, sizeof(tmp), cudaMemcpyDeviceToHost, st));
  SGP_CUDA_TRY(h, cudaStreamSynchronize(st));
  h_stats[0] = tmp[2];
  h_stats[1] = tmp[3];
  h_stats[2] = tmp[1];
  h_stats[3] = tmp[0];
  return SGP_OK;
}

int sgp_param_deviation(sgp_handle *h, const float *d_A, double *h_dev, void *stream) {
  if (h == nullptr || d_A == nullptr || h_dev == nullptr) return SGP_ERR_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  double *acc = h->d_stats + 4;
  SGP_CUDA_TRY(h, cudaMemsetAsync(acc, 0, static_cast<size_t>(h->n) * sizeof(double), st));
  // tile of n rows x tile_cols columns in shared memory, at most ~64 KB
  int tile_cols = 256;
  while (tile_cols > 32 && static_cast<size_t>(h->n) * tile_cols * 4 > 64 * 1024) tile_cols >>= 1;
  const size_t smem = (static_cast<size_t>(h->n) * tile_cols + tile_cols + h->n) * sizeof(float);
  if (smem > 48 * 1024)
    SGP_CUDA_TRY(h, cudaFuncSetAttribute(reinterpret_cast<const void *>(sgp::sgp_deviation_kernel),
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
  const int64_t ntiles = (h->d + tile_cols - 1) / tile_cols;
  const unsigned grid = static_cast<unsigned>(std::min<int64_t>(ntiles, static_cast<int64_t>(h->sm_count) * 2));
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
    if (value > 3) return SGP_ERR_ARG;
    h->opt_variant = value;
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
  } else if (std::strcmp(key, "l2_hint") == 0) {
    if (value > 4) return SGP_ERR_ARG;
    h->opt_l2_hint = value;
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
  else if (std::strcmp(key, "wait_limit_ms") == 0) *value = h->opt_wait_limit_ms;
  else if (std::strcmp(key, "inject_stall") == 0) *value = h->opt_inject_stall;
  else if (std::strcmp(key, "last_variant") == 0) *value = h->last_variant;
  else if (std::strcmp(key, "last_grid") == 0) *value = h->last_grid;
  else if (std::strcmp(key, "launches") == 0) *value = h->launches;
  else if (std::strcmp(key, "last_smem") == 0) *value = h->last_smem;
  else if (std::strcmp(key, "last_tile_cols") == 0) *value = h->last_tile_cols;
  else return SGP_ERR_ARG;
  return SGP_OK;
}

int sgp_device_status(sgp_handle *h, unsigned *status) {
  if (h == nullptr || status == nullptr) return SGP_ERR_ARG;
  SGP_CUDA_TRY(h, cudaDeviceSynchronize());
  SGP_CUDA_TRY(h, cudaMemcpy(status, h->d_words + 1, sizeof(unsigned), cudaMemcpyDeviceToHost));
  return SGP_OK;
}

int sgp_last_cuda_error(const sgp_handle *h) { return h == nullptr ? 0 : h->last_cuda_error; }

}  // extern "C"
