// Instantiations and launcher of the peeled step kernel (rows that do not start on 16-byte boundaries).
#include <algorithm>

#include "launch.h"
#include "sgp.h"
#include "step_peel_kernel.cuh"

namespace sgp {

namespace {

template <int UPD>
PeelKernel pick_flags(bool has_z, bool has_ring) {
  if (has_z) return has_ring ? sgp_step_peel_kernel<UPD, true, true> : sgp_step_peel_kernel<UPD, true, false>;
  return has_ring ? sgp_step_peel_kernel<UPD, false, true> : sgp_step_peel_kernel<UPD, false, false>;
}

inline int floor_log2(int64_t v) {
  int l = 0;
  while ((int64_t{1} << (l + 1)) <= v) ++l;
  return l;
}

}  // namespace

PeelKernel peel_kernel(int upd, bool has_z, bool has_ring) {
  switch (upd) {
    case kUpdSgd: return pick_flags<kUpdSgd>(has_z, has_ring);
    case kUpdHeavyBall: return pick_flags<kUpdHeavyBall>(has_z, has_ring);
    case kUpdNesterov: return pick_flags<kUpdNesterov>(has_z, has_ring);
    default: return pick_flags<kUpdAdam>(has_z, has_ring);
  }
}

bool peel_applicable(const StepParams &p) {
  // every array must sit at the same distance from a 16-byte boundary, so that one cut per row serves them all
  const uintptr_t ref = reinterpret_cast<uintptr_t>(p.X) & 15u;
  const void *arrays[] = {p.G, p.M, p.V, p.Z, p.ring_x};
  for (const void *a : arrays)
    if (a != nullptr && (reinterpret_cast<uintptr_t>(a) & 15u) != ref) return false;
  return (ref & 3u) == 0 && p.diag == nullptr;
}

int launch_peel(const DeviceInfo &dev, StepParams p, const ConstTable *ct, int upd, const PeelOptions &opt, cudaStream_t stream,
                LaunchRecord *rec) {
  if (!peel_applicable(p)) return SGP_ERR_STATE;
  const int n = p.n;
  const bool has_ring = p.ring_x != nullptr;
  const int64_t ncols = p.col_end - p.col_begin;
  // tile width as for the register-staged kernel (1 KB row segments where the shared tile allows it)
  int64_t cols = opt.tile_cols > 0 ? opt.tile_cols : regs_tile_cols(n, 4 * 1024);
  cols = std::max<int64_t>(16, int64_t{4} << floor_log2(std::max<int64_t>(1, cols / 4)));
  if (opt.tile_cols <= 0)
    while (cols > 64 && (ncols + cols - 1) / cols < dev.sm_count) cols >>= 1;       // short rows: about a tile per SM
  const size_t table_bytes = table_smem_bytes(n, p.nnz);
  if (ct != nullptr) p.table_mode = 0;
  else p.table_mode = table_bytes <= 40 * 1024 ? 1 : 2;
  p.single_buffer = opt.single_buffer == 1 ? 1 : (opt.single_buffer == 2 ? 0 : (auto_single_buffer(n) || n * (cols / 4) > 8 * kThreads ? 1 : 0));
  p.uniform_parts = 0;
  size_t smem = 0;
  for (;;) {
    const size_t tile_floats = static_cast<size_t>(n) * (cols + kPeelRowPad) + kPeelTilePad;
    smem = (p.single_buffer ? 1 : 2) * tile_floats * 4 + 3 * static_cast<size_t>(n) * 4 + (p.table_mode < 2 ? table_bytes : 0);
    if (smem <= 110 * 1024 || cols <= 16) break;
    cols >>= 1;
  }
  if (smem > static_cast<size_t>(dev.smem_optin)) return SGP_ERR_ARG;
  p.log2_tile_vecs = floor_log2(cols / 4);
  p.peel_phase0 = static_cast<int>(((reinterpret_cast<uintptr_t>(p.X) >> 2) + static_cast<uintptr_t>(p.col_begin)) & 3u);
  p.peel_phase_step = static_cast<int>(p.ld & 3);
  const int64_t ntiles = (ncols + cols - 1) / cols;
  PeelKernel kern = peel_kernel(upd, p.Z != nullptr, has_ring);
  KernelInfo ki;
  {
    const int rc = kernel_info(dev.device, reinterpret_cast<const void *>(kern), smem, &ki, &rec->cuda_error);
    if (rc != SGP_OK) return rc;
  }
  int cps = opt.cps;
  if (cps <= 0) {
    const int regs_per_cta = ((ki.num_regs + 7) / 8 * 8) * kThreads;
    const int by_regs = regs_per_cta > 0 ? 65536 / regs_per_cta : 8;
    const int by_smem = static_cast<int>((227 * 1024) / (smem + ki.static_smem + 1024));
    cps = std::max(1, std::min({by_regs, by_smem, 2048 / kThreads}));
  }
  const int64_t grid = std::min<int64_t>(ntiles, static_cast<int64_t>(dev.sm_count) * cps);
  static const ConstTable kEmptyTable{};
  p.lockstep = 0;      // lockstep clusters were measured on this kernel and change nothing (it is not bound by DRAM)
  kern<<<static_cast<unsigned>(grid), kThreads, smem, stream>>>(p, ct != nullptr ? *ct : kEmptyTable);
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) {
    rec->cuda_error = static_cast<int>(e);
    return SGP_ERR_CUDA;
  }
  rec->variant = 5;
  rec->grid = grid;
  rec->smem = static_cast<int64_t>(smem);
  rec->tile_cols = cols;
  rec->lockstep = 0;
  return SGP_OK;
}

}  // namespace sgp
