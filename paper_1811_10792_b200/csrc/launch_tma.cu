// Launcher of the bulk-copy (TMA) pipelined fused step kernel.
#include <algorithm>
#include <cstring>

#include "launch.h"
#include "sgp.h"
#include "step_tma_kernel.cuh"

namespace sgp {

namespace {

inline int floor_log2(int64_t v) {
  int l = 0;
  while ((int64_t{1} << (l + 1)) <= v) ++l;
  return l;
}

}  // namespace

template <> TmaKernel tma_kernel_of<false>(int, bool, bool);
template <> TmaKernel tma_kernel_of<true>(int, bool, bool);

int launch_tma(const DeviceInfo &dev, StepParams p, const ConstTable *ct, int upd, bool uniform_rows,
               const TmaOptions &opt, TensorMapFn map_fn, void *map_ctx, cudaStream_t stream, LaunchRecord *rec) {
  const int n = p.n;
  const bool has_m = p.M != nullptr, has_v = p.V != nullptr, has_ring = p.ring_x != nullptr;
  const int arrays = 2 + (has_m ? 1 : 0) + (has_v ? 1 : 0) + (has_ring ? 1 : 0);
  int64_t tv = int64_t{1} << floor_log2(std::max<int64_t>(1, (opt.tile_cols > 0 ? opt.tile_cols : 256) / 4));
  tv = std::max<int64_t>(tv, 8);
  if (p.diag != nullptr) tv = std::min<int64_t>(tv, 256);   // diagnostics: a consumer thread owns one column of every tile
  int stages = std::max(1, opt.stages);
  const int cps = opt.cps > 0 ? opt.cps : 2;
  const size_t table_bytes = table_smem_bytes(n, p.nnz);
  if (ct != nullptr) p.table_mode = 0;
  else p.table_mode = table_bytes <= 40 * 1024 ? 1 : 2;
  const bool uniform = !has_ring && uniform_rows;
  const size_t fixed = 16 * sizeof(uint64_t) + 3 * static_cast<size_t>(n) * 4 + (p.table_mode < 2 ? table_bytes : 0);
  const size_t budget = std::min<size_t>(static_cast<size_t>(dev.smem_optin), (228 * 1024) / static_cast<size_t>(cps) - 2048);
  size_t smem = 0;
  for (;;) {
    const int parts = static_cast<int>(std::max<int64_t>(1, std::min<int64_t>(8, kTmaConsumers / tv)));
    p.uniform_parts = uniform ? parts : 0;
    smem = static_cast<size_t>(stages) * arrays * n * tv * 16 + fixed + static_cast<size_t>(p.uniform_parts) * tv * 16;
    if (p.diag != nullptr) smem += diag_scratch_bytes<float4>(n, static_cast<int>(tv), has_ring);
    if (smem <= budget) break;
    if (!opt.stages_forced && stages > 2) --stages;
    else if (!opt.tile_cols_forced && tv > 8) tv >>= 1;
    else return SGP_ERR_STATE;
  }
  p.log2_tile_vecs = floor_log2(tv);
  const int64_t tile_cols = tv * 4;
  const int64_t ntiles = (p.col_end - p.col_begin + tile_cols - 1) / tile_cols;
  const int64_t grid = std::min<int64_t>(ntiles, static_cast<int64_t>(dev.sm_count) * cps);
  p.wait_limit_ms = opt.wait_limit_ms > 0 ? opt.wait_limit_ms : 2000;
  p.inject_stall = opt.inject_stall ? 1 : 0;
  p.l2_hint = opt.l2_hint;
  TmaKernel kern = p.diag != nullptr ? tma_kernel_of<true>(upd, p.Z != nullptr, has_ring) : tma_kernel_of<false>(upd, p.Z != nullptr, has_ring);
  {
    KernelInfo ki;
    const int rc = kernel_info(dev.device, reinterpret_cast<const void *>(kern), smem, &ki, &rec->cuda_error);
    if (rc != SGP_OK) return rc;
  }
  static const ConstTable kEmptyTable{};
  // 2-D tensor maps (one copy per array per tile) when the box fits; else one bulk copy per row segment
  TmaMaps maps;
  std::memset(&maps, 0, sizeof(maps));
  bool use_maps = opt.variant == 2 && map_fn != nullptr && tile_cols <= 256 && tile_cols * 4 % 128 == 0;
  if (use_maps) use_maps = map_fn(map_ctx, p.X, static_cast<int>(tile_cols), &maps.x);
  if (use_maps) use_maps = map_fn(map_ctx, p.G, static_cast<int>(tile_cols), &maps.g);
  if (use_maps && has_m) use_maps = map_fn(map_ctx, p.M, static_cast<int>(tile_cols), &maps.m);
  if (use_maps && has_v) use_maps = map_fn(map_ctx, p.V, static_cast<int>(tile_cols), &maps.v);
  if (use_maps && has_ring) use_maps = map_fn(map_ctx, p.ring_x, static_cast<int>(tile_cols), &maps.r);
  kern<<<static_cast<unsigned>(grid), kTmaThreads, smem, stream>>>(p, ct != nullptr ? *ct : kEmptyTable, maps, stages,
                                                                  use_maps ? 1 : 0);
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) {
    rec->cuda_error = static_cast<int>(e);
    return SGP_ERR_CUDA;
  }
  rec->variant = use_maps ? 2 : 3;
  rec->grid = grid;
  rec->smem = static_cast<int64_t>(smem);
  rec->tile_cols = tile_cols;
  return SGP_OK;
}

}  // namespace sgp
