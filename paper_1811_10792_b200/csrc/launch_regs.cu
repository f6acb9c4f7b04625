// Launcher of the register-staged fused step kernel and the per-(device, kernel) attribute cache.
#include <algorithm>
#include <map>
#include <mutex>
#include <tuple>
#include <utility>

#include "launch.h"
#include "sgp.h"
#include "step_regs_kernel.cuh"

namespace sgp {

namespace {

std::mutex g_kernel_info_mutex;
std::map<std::pair<int, const void *>, KernelInfo> g_kernel_info;   // function attributes are per device

inline int floor_log2(int64_t v) {
  int l = 0;
  while ((int64_t{1} << (l + 1)) <= v) ++l;
  return l;
}

}  // namespace

template <> RegsKernel regs_kernel_of<4, false>(int, bool, bool, bool);
template <> RegsKernel regs_kernel_of<4, true>(int, bool, bool, bool);
template <> RegsKernel regs_kernel_of<1, false>(int, bool, bool, bool);
template <> RegsKernel regs_kernel_of<1, true>(int, bool, bool, bool);

RegsKernel regs_kernel(int vec, int upd, bool has_z, bool has_ring, bool diag, bool gather_first) {
  if (vec == 4)
    return diag ? regs_kernel_of<4, true>(upd, has_z, has_ring, gather_first) : regs_kernel_of<4, false>(upd, has_z, has_ring, gather_first);
  return diag ? regs_kernel_of<1, true>(upd, has_z, has_ring, gather_first) : regs_kernel_of<1, false>(upd, has_z, has_ring, gather_first);
}

int kernel_info(int device, const void *kern, size_t smem, KernelInfo *out, int *cuda_error) {
  std::lock_guard<std::mutex> lock(g_kernel_info_mutex);
  const std::pair<int, const void *> key(device, kern);
  auto it = g_kernel_info.find(key);
  cudaError_t e = cudaSuccess;
  if (it == g_kernel_info.end()) {
    cudaFuncAttributes fa;
    e = cudaFuncGetAttributes(&fa, kern);
    if (e == cudaSuccess) {
      KernelInfo ki;
      ki.num_regs = fa.numRegs;
      ki.static_smem = fa.sharedSizeBytes;
      // without the attribute a launch may use 48 KB of shared memory, static part included
      ki.enabled_smem = 48 * 1024 - std::min<size_t>(48 * 1024, fa.sharedSizeBytes);
      it = g_kernel_info.emplace(key, ki).first;
    }
  }
  if (e == cudaSuccess && smem > it->second.enabled_smem) {
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e == cudaSuccess) it->second.enabled_smem = smem;
  }
  if (e != cudaSuccess) {
    if (cuda_error) *cuda_error = static_cast<int>(e);
    (void)cudaGetLastError();
    return SGP_ERR_CUDA;
  }
  *out = it->second;
  return SGP_OK;
}

int resident_clusters(int device, const void *kern, int cluster, size_t smem) {
  static std::map<std::tuple<int, const void *, int, size_t>, int> cache;
  std::lock_guard<std::mutex> lock(g_kernel_info_mutex);
  const auto key = std::make_tuple(device, kern, cluster, smem);
  auto it = cache.find(key);
  if (it != cache.end()) return it->second;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(static_cast<unsigned>(cluster));
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = smem;
  cudaLaunchAttribute attr{};
  attr.id = cudaLaunchAttributeClusterDimension;
  attr.val.clusterDim.x = static_cast<unsigned>(cluster);
  attr.val.clusterDim.y = 1;
  attr.val.clusterDim.z = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  int clusters = 0;
  if (cudaOccupancyMaxActiveClusters(&clusters, kern, &cfg) != cudaSuccess) {
    (void)cudaGetLastError();
    clusters = 0;
  }
  cache.emplace(key, clusters);
  return clusters;
}

// One exchange tile (two barriers per tile) where that keeps the row segments long (n = 64: 1 KB segments 0.95
// of the copy bandwidth against 0.92; n = 80: 0.97 against 0.82; n = 96: 512 B 0.92 against 0.89; n > 128: 256 B
// 0.91 against 0.70); two tiles and one barrier elsewhere (n = 112, 128: 0.94 against 0.92).
bool auto_single_buffer(int n) { return (n > 32 && n <= 104) || n > 128; }

size_t table_smem_bytes(int n, int nnz) { return (static_cast<size_t>(n) + 1 + 2 * static_cast<size_t>(nnz)) * 4; }

// Row segments of at least 1 KB and about 2048 vector items per tile, shrunk until the exchange tile(s) plus
// `fixed` bytes stay near 80 KB per CTA -- two resident CTAs then leave about half of the SM's 256 KB to the L1
// that tracks the loads in flight (measured: n = 48 at 2 x 100 KB reaches 0.74 of the copy bandwidth, at
// 2 x 50 KB 0.93).
int64_t regs_tile_cols(int n, size_t fixed) {
  int64_t cols = std::max<int64_t>(256, int64_t{4} << floor_log2(std::max<int64_t>(1, 2048 / n)));
  const size_t copies = auto_single_buffer(n) ? 1 : 2;
  const size_t cap = (copies == 1 ? 88 : 80) * 1024;     // n = 80 at 85 KB: 0.97; n = 96 at 102 KB: 0.79
  while (cols > 32 && copies * static_cast<size_t>(n) * cols * 4 + fixed > cap) cols >>= 1;
  // Between four and six items per thread the tile falls into a batch of three and a batch of one to three (n = 5,
  // 10, 20: 0.92-0.93 of the copy bandwidth where the neighbours reach 0.98): twice the width in ONE exchange tile
  // (the same shared memory) gives three fuller batches instead (0.99).
  const int64_t items = static_cast<int64_t>(n) * cols / 4;
  if (copies == 2 && items > 4 * kThreads && items < 6 * kThreads) cols *= 2;
  return cols;
}

int launch_regs(const DeviceInfo &dev, StepParams p, const ConstTable *ct, int upd, int vec, bool uniform_rows,
                const RegsOptions &opt, cudaStream_t stream, LaunchRecord *rec) {
  const int n = p.n;
  const bool has_ring = p.ring_x != nullptr;
  // tile width: the caller's, else about four items per thread; at least 128 bytes per row segment
  const int64_t ncols = p.col_end - p.col_begin;
  const int min_tv = vec == 4 ? 8 : 32;
  int64_t tv = int64_t{1} << floor_log2(std::max<int64_t>(1, kThreads * 4 / n));
  if (opt.tile_cols > 0) tv = int64_t{1} << floor_log2(std::max<int64_t>(1, opt.tile_cols / vec));
  tv = std::max<int64_t>(tv, min_tv);
  if (p.diag != nullptr) tv = std::min<int64_t>(tv, 256);   // diagnostics: a thread owns one column of every tile
  // short rows: narrower tiles until there is about a tile per SM (launch-latency regime)
  if (!opt.tile_cols_forced)
    while (tv > min_tv && tv * vec > 128 && (ncols + tv * vec - 1) / (tv * vec) < dev.sm_count) tv >>= 1;
  const size_t table_bytes = table_smem_bytes(n, p.nnz);
  if (ct != nullptr) p.table_mode = 0;
  else p.table_mode = table_bytes <= 40 * 1024 ? 1 : 2;
  const bool uniform = !has_ring && uniform_rows;
  // large n: one exchange tile (two barriers per tile) so that the row segments can stay twice as long
  // (also for the doubled tiles of regs_tile_cols: more than eight items per thread at n <= 32)
  p.single_buffer = opt.single_buffer == 1 ? 1 : (opt.single_buffer == 2 ? 0 : ((auto_single_buffer(n) || (n <= 32 && n * tv > 8 * kThreads)) ? 1 : 0));
  // diagnostics add up to 32 KB of scratch: one exchange tile then keeps the CTA's footprint (and with it the
  // share of the SM left to the L1) where it was (tau = 1, n = 32: 96 KB per CTA ran at 0.67, 64 KB does not)
  if (p.diag != nullptr && opt.single_buffer == 0) p.single_buffer = 1;
  size_t smem = 0;
  for (;;) {
    const int parts = static_cast<int>(std::max<int64_t>(1, std::min<int64_t>(8, kThreads / tv)));
    p.uniform_parts = uniform ? parts : 0;
    smem = (p.single_buffer ? 1 : 2) * static_cast<size_t>(n) * tv * vec * 4 + 3 * static_cast<size_t>(n) * 4 +
           static_cast<size_t>(p.uniform_parts) * tv * vec * 4 + (p.table_mode < 2 ? table_bytes : 0);
    if (p.diag != nullptr)
      smem += vec == 4 ? diag_scratch_bytes<float4>(n, static_cast<int>(tv), has_ring) : diag_scratch_bytes<float>(n, static_cast<int>(tv), has_ring);
    if (smem <= 110 * 1024 || tv <= min_tv) break;
    tv >>= 1;
  }
  if (smem > static_cast<size_t>(dev.smem_optin)) return SGP_ERR_ARG;
  p.log2_tile_vecs = floor_log2(tv);
  const int64_t tile_cols = tv * vec;
  const int64_t ntiles = (ncols + tile_cols - 1) / tile_cols;
  // Order of instructions inside a phase (momentum updates without a ring): every gather of a batch before its
  // stores wins where the tile is made of full four-item batches and row segments are at least 512 bytes (n = 4..96:
  // +1 to +1.7 % of the copy bandwidth) and loses elsewhere (n = 24, three-item batches: 0.935 against 0.974; ragged
  // last batch, n = 104, 112: 0.89 against 0.92-0.93; 256-byte segments, n = 128, 256: 0.91 against 0.93).  It also
  // costs a launch about 4 us more than it returns below ~0.4 ms of work (n = 64, d = 1e6: 0.267 ms against 0.259;
  // n = 16, d = 1e7, 0.6 ms: 0.604 against 0.607), so short launches keep the interleaved order.
  const bool gather_first = (static_cast<int64_t>(n) * tv) % (4 * kThreads) == 0 && tile_cols * 4 >= 512 &&
                            static_cast<int64_t>(n) * ncols >= (int64_t{1} << 27);
  RegsKernel kern = regs_kernel(vec, upd, p.Z != nullptr, has_ring, p.diag != nullptr, gather_first);
  KernelInfo ki;
  {
    const int rc = kernel_info(dev.device, reinterpret_cast<const void *>(kern), smem, &ki, &rec->cuda_error);
    if (rc != SGP_OK) return rc;
  }
  int cps = opt.cps;
  if (cps <= 0) {
    // Persistent grid of exactly one wave: CTAs resident per SM by registers, shared memory and threads.
    // (Computed here rather than asked of the occupancy calculator, whose answer depends on the
    // shared-memory carve-out it assumes; the hardware picks the carve-out that fits the launch.)
    const int regs_per_cta = ((ki.num_regs + 7) / 8 * 8) * kThreads;
    const int by_regs = regs_per_cta > 0 ? 65536 / regs_per_cta : 8;
    const int by_smem = static_cast<int>((227 * 1024) / (smem + ki.static_smem + 1024));
    cps = std::max(1, std::min({by_regs, by_smem, 2048 / kThreads}));
  }
  int64_t grid = std::min<int64_t>(ntiles, static_cast<int64_t>(dev.sm_count) * cps);
  // Short launches: with k = ceil(ntiles / grid) tiles for the busiest CTA, ceil(ntiles / k) CTAs finish at the same
  // time; the few CTA slots left empty cost less than a last round in which most of the device idles.
  if (grid > 0 && ntiles > grid && ntiles < 32 * grid) {
    const int64_t rounds = (ntiles + grid - 1) / grid;
    grid = (ntiles + rounds - 1) / rounds;
  }
  static const ConstTable kEmptyTable{};
  // Lockstep clusters (what was measured, of the copy bandwidth): rows that do not start on 128-byte boundaries
  // split every 1 KB block between two tiles, and CTAs that take neighbouring tiles at the same moment get most of
  // the loss back (rows on 32-byte boundaries, n = 32: 0.87 -> 0.91 in pairs; tau = 1: 0.86 -> 0.90; n = 64:
  // 0.83 -> 0.88 in pairs, 0.91 in fours; n = 128: 0.61 -> 0.66 / 0.74); a cluster of four leaves 12 of the 296 CTA
  // slots empty, which costs n = 32 more than it returns (0.89).  With rows on 1 KB boundaries pairs are worth
  // +0.6 % with a delay ring at 1 KB segments and -1 to -3 % with narrow (n >= 96) or wide (n <= 24) tiles: off.
  p.lockstep = 0;
  if (opt.lockstep >= 2) {
    p.lockstep = opt.lockstep;
  } else if (opt.lockstep == 0 && vec == 4 && n >= 32 && ntiles >= 2 * grid) {
    const uintptr_t bits = reinterpret_cast<uintptr_t>(p.X) | reinterpret_cast<uintptr_t>(p.G) | reinterpret_cast<uintptr_t>(p.M) |
                           reinterpret_cast<uintptr_t>(p.V) | reinterpret_cast<uintptr_t>(p.Z) | reinterpret_cast<uintptr_t>(p.ring_x) |
                           static_cast<uintptr_t>(p.ld * 4);
    if ((bits & 127) != 0 && tile_cols <= 256) p.lockstep = n >= 64 ? 4 : 2;
    else if ((bits & 1023) == 0 && has_ring && tile_cols == 256) p.lockstep = 2;
  }
  cudaError_t e = cudaSuccess;
  if (p.lockstep) {
    const int clusters = resident_clusters(dev.device, reinterpret_cast<const void *>(kern), p.lockstep, smem);
    if (clusters < 1) p.lockstep = 0;
    else grid = std::min<int64_t>({(ntiles + p.lockstep - 1) / p.lockstep, static_cast<int64_t>(clusters), static_cast<int64_t>(dev.sm_count) * cps / p.lockstep}) * p.lockstep;
  }
  if (p.lockstep) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(static_cast<unsigned>(grid));
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr{};
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = static_cast<unsigned>(p.lockstep);
    attr.val.clusterDim.y = 1;
    attr.val.clusterDim.z = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    e = cudaLaunchKernelEx(&cfg, kern, p, ct != nullptr ? *ct : kEmptyTable);
    if (e != cudaSuccess) {
      // a cluster launch that the device refuses is only a lost optimisation: launch independent CTAs instead
      (void)cudaGetLastError();
      p.lockstep = 0;
    }
  }
  if (!p.lockstep) {
    kern<<<static_cast<unsigned>(grid), kThreads, smem, stream>>>(p, ct != nullptr ? *ct : kEmptyTable);
    e = cudaGetLastError();
  }
  if (e != cudaSuccess) {
    rec->cuda_error = static_cast<int>(e);
    return SGP_ERR_CUDA;
  }
  rec->variant = 1;
  rec->grid = grid;
  rec->smem = static_cast<int64_t>(smem);
  rec->tile_cols = tile_cols;
  rec->lockstep = p.lockstep;
  return SGP_OK;
}

}  // namespace sgp
