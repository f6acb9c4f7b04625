// Launchers of the fused step kernels: tile sizing, shared-memory budget, grid size.  Shared by the handle
// path (sgp_api.cu) and the handle-free static path (sgp_static.cu), so that both size a launch identically and
// share ONE per-(device, kernel) attribute cache.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

#include <cstddef>
#include <cstdint>

#include "step_common.cuh"

namespace sgp {

struct DeviceInfo {
  int device = 0;
  int sm_count = 0;
  int smem_optin = 0;
};

// What a launcher did (reported through sgp_get_option) and, on SGP_ERR_CUDA, the runtime's error code.
struct LaunchRecord {
  int variant = 0;
  int64_t grid = 0;
  int64_t smem = 0;
  int64_t tile_cols = 0;
  int lockstep = 0;      // CTAs per lockstep cluster of the register-staged kernel (0 = independent CTAs)
  int cuda_error = 0;
};

// Per-kernel facts that do not change during the process: registers, static shared memory, and the
// largest dynamic shared-memory size already enabled.  The limit is only ever RAISED, and every launcher of the
// library goes through this one cache: a later launch with a smaller request can therefore never lower the
// limit under an earlier, larger configuration of the same kernel.
struct KernelInfo {
  int num_regs = 0;
  size_t static_smem = 0;
  size_t enabled_smem = 48 * 1024;   // largest DYNAMIC size a launch may ask for (48 KB less the static part at first)
};
int kernel_info(int device, const void *kern, size_t smem, KernelInfo *out, int *cuda_error);
// Clusters of `cluster` CTAs (kThreads threads, `smem` dynamic bytes each) of `kern` that `device` holds at once;
// 0 when the query fails.  Cached per (device, kernel, cluster, smem).
int resident_clusters(int device, const void *kern, int cluster, size_t smem);

// Register-staged kernel: one exchange tile (two barriers per tile) where that keeps the row segments long.
bool auto_single_buffer(int n);
// Tile width (columns) of the register-staged kernel's 128-bit path for n nodes with `fixed` bytes of other
// shared memory per CTA.
int64_t regs_tile_cols(int n, size_t fixed);
size_t table_smem_bytes(int n, int nnz);

struct RegsOptions {
  int64_t tile_cols = 0;          // 0 = automatic
  bool tile_cols_forced = false;  // true: the caller asked for exactly this width (no narrowing for short rows)
  int cps = 0;                    // CTAs per SM, 0 = as many as are resident
  int single_buffer = 0;          // 0 automatic, 1 one tile, 2 two tiles
  int lockstep = 0;               // 0 automatic, 1 independent CTAs, 2 / 4 = clusters of that many CTAs in lockstep
};

// One launch of the register-staged kernel over columns [p.col_begin, p.col_end) with vector width vec (4 or 1).
// `p` carries the arrays, n, nnz, ld, the table pointers, the scalars, update_w, diag; the launcher fills the
// tile geometry, table_mode, uniform_parts, single_buffer.  `ct` may be null (table read from global memory).
int launch_regs(const DeviceInfo &dev, StepParams p, const ConstTable *ct, int upd, int vec, bool uniform_rows,
                const RegsOptions &opt, cudaStream_t stream, LaunchRecord *rec);

struct PeelOptions {
  int64_t tile_cols = 0;          // 0 = automatic
  int cps = 0;                    // CTAs per SM, 0 = as many as are resident
  int single_buffer = 0;          // 0 automatic, 1 one tile, 2 two tiles
};
// True when the peeled kernel can take the launch: every array at the same distance (a multiple of 4 bytes) from a
// 16-byte boundary, no fused diagnostics.
bool peel_applicable(const StepParams &p);
// One launch of the peeled kernel (rows that do not start on 16-byte boundaries) over columns [p.col_begin, p.col_end).
// Returns SGP_ERR_STATE when it is not applicable; the caller then uses the scalar instantiation.
int launch_peel(const DeviceInfo &dev, StepParams p, const ConstTable *ct, int upd, const PeelOptions &opt, cudaStream_t stream,
                LaunchRecord *rec);

struct TmaOptions {
  int variant = 3;                // 2 = 2-D tensor maps, 3 = one bulk copy per row segment
  int64_t tile_cols = 256;
  bool tile_cols_forced = false;
  int stages = 2;
  bool stages_forced = false;
  int cps = 2;
  int wait_limit_ms = 2000;
  int inject_stall = 0;
  int l2_hint = 3;
};
// Supplies the tensor map of an n x d array (box = box_cols x n); returns false when unavailable.
using TensorMapFn = bool (*)(void *ctx, const float *base, int box_cols, CUtensorMap *out);

// One launch of the bulk-copy pipelined kernel (128-bit preconditions required).  Returns SGP_ERR_STATE when
// the shape does not fit its shared-memory stages; the caller then uses the register-staged kernel.
int launch_tma(const DeviceInfo &dev, StepParams p, const ConstTable *ct, int upd, bool uniform_rows,
               const TmaOptions &opt, TensorMapFn map_fn, void *map_ctx, cudaStream_t stream, LaunchRecord *rec);

struct ClusterOptions {
  int cluster_size = 4;           // CTAs per cluster: 2 or 4
  int64_t tile_cols = 256;
  bool tile_cols_forced = false;
  int max_clusters = 0;           // 0 = as many as are resident
};
// One launch of the thread-block-cluster kernel (many nodes; 128-bit preconditions, no shared-column-sum path, no
// diagnostics).  Returns SGP_ERR_STATE when clusters of this shape cannot be resident; the caller then uses the
// register-staged kernel.
int launch_cluster(const DeviceInfo &dev, StepParams p, const ConstTable *ct, int upd, const ClusterOptions &opt,
                   cudaStream_t stream, LaunchRecord *rec);

}  // namespace sgp
