// Launcher and instantiations of the thread-block-cluster step kernel (many nodes).
#include <algorithm>
#include <map>
#include <mutex>
#include <utility>

#include "launch.h"
#include "sgp.h"
#include "step_cluster_kernel.cuh"

namespace sgp {

namespace {

inline int floor_log2(int64_t v) {
  int l = 0;
  while ((int64_t{1} << (l + 1)) <= v) ++l;
  return l;
}

template <int UPD>
ClusterKernel pick_flags(bool has_z, bool has_ring) {
  if (has_z) return has_ring ? sgp_step_cluster_kernel<UPD, true, true> : sgp_step_cluster_kernel<UPD, true, false>;
  return has_ring ? sgp_step_cluster_kernel<UPD, false, true> : sgp_step_cluster_kernel<UPD, false, false>;
}

// Clusters of this kernel that can be resident at once, per (device, kernel, cluster size, shared memory).
std::mutex g_mutex;
std::map<std::pair<std::pair<int, const void *>, std::pair<int, size_t>>, int> g_active_clusters;

}  // namespace

ClusterKernel cluster_kernel(int upd, bool has_z, bool has_ring) {
  switch (upd) {
    case kUpdSgd: return pick_flags<kUpdSgd>(has_z, has_ring);
    case kUpdHeavyBall: return pick_flags<kUpdHeavyBall>(has_z, has_ring);
    case kUpdNesterov: return pick_flags<kUpdNesterov>(has_z, has_ring);
    default: return pick_flags<kUpdAdam>(has_z, has_ring);
  }
}

int launch_cluster(const DeviceInfo &dev, StepParams p, const ConstTable *ct, int upd, const ClusterOptions &opt,
                   cudaStream_t stream, LaunchRecord *rec) {
  const int n = p.n;
  const bool has_ring = p.ring_x != nullptr;
  const int cl = opt.cluster_size;
  if (cl != 2 && cl != 4) return SGP_ERR_STATE;
  ClusterGeometry geo;
  geo.cluster_size = cl;
  geo.log2_rows_per_cta = 0;
  while ((cl << geo.log2_rows_per_cta) < n) ++geo.log2_rows_per_cta;
  const int64_t rows_per_cta = int64_t{1} << geo.log2_rows_per_cta;
  const size_t table_bytes = table_smem_bytes(n, p.nnz);
  if (ct != nullptr) p.table_mode = 0;
  else p.table_mode = table_bytes <= 40 * 1024 ? 1 : 2;
  const size_t fixed = 3 * static_cast<size_t>(n) * 4 + (p.table_mode < 2 ? table_bytes : 0);
  // row segments of 1 KB where the slice of the tile stays near 80 KB per CTA (two CTAs per SM)
  int64_t tv = int64_t{1} << floor_log2(std::max<int64_t>(8, (opt.tile_cols > 0 ? opt.tile_cols : 256) / 4));
  while (tv > 8 && static_cast<size_t>(rows_per_cta) * tv * 16 + fixed > (opt.tile_cols_forced ? 200u : 88u) * 1024) tv >>= 1;
  const size_t smem = static_cast<size_t>(rows_per_cta) * tv * 16 + fixed;
  if (smem > static_cast<size_t>(dev.smem_optin)) return SGP_ERR_STATE;
  p.log2_tile_vecs = floor_log2(tv);
  p.single_buffer = 1;
  p.uniform_parts = 0;
  const int64_t tile_cols = tv * 4;
  const int64_t ntiles = (p.col_end - p.col_begin + tile_cols - 1) / tile_cols;
  ClusterKernel kern = cluster_kernel(upd, p.Z != nullptr, has_ring);
  KernelInfo ki;
  {
    const int rc = kernel_info(dev.device, reinterpret_cast<const void *>(kern), smem, &ki, &rec->cuda_error);
    if (rc != SGP_OK) return rc;
  }
  cudaLaunchConfig_t cfg{};
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = static_cast<unsigned>(cl);
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  int max_clusters = 0;
  {
    std::lock_guard<std::mutex> lock(g_mutex);
    const auto key = std::make_pair(std::make_pair(dev.device, reinterpret_cast<const void *>(kern)), std::make_pair(cl, smem));
    auto it = g_active_clusters.find(key);
    if (it == g_active_clusters.end()) {
      cfg.gridDim = dim3(static_cast<unsigned>(cl) * static_cast<unsigned>(dev.sm_count));
      int v = 0;
      const cudaError_t e = cudaOccupancyMaxActiveClusters(&v, reinterpret_cast<const void *>(kern), &cfg);
      if (e != cudaSuccess || v < 1) {
        (void)cudaGetLastError();
        return SGP_ERR_STATE;                       // the caller falls back to the one-CTA kernel
      }
      it = g_active_clusters.emplace(key, v).first;
    }
    max_clusters = it->second;
  }
  const int64_t clusters = std::min<int64_t>(ntiles, opt.max_clusters > 0 ? std::min<int64_t>(opt.max_clusters, max_clusters) : max_clusters);
  cfg.gridDim = dim3(static_cast<unsigned>(clusters * cl));
  static const ConstTable kEmptyTable{};
  const cudaError_t e = cudaLaunchKernelEx(&cfg, kern, p, ct != nullptr ? *ct : kEmptyTable, geo);
  if (e != cudaSuccess) {
    (void)cudaGetLastError();
    rec->cuda_error = static_cast<int>(e);
    return SGP_ERR_CUDA;
  }
  rec->variant = 4;
  rec->grid = clusters * cl;
  rec->smem = static_cast<int64_t>(smem);
  rec->tile_cols = tile_cols;
  return SGP_OK;
}

}  // namespace sgp
