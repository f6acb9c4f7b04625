// sgp_step_static: the fused SGP step for callers that must not allocate device memory.
//
// Some hosts of this library cannot call cudaMalloc at all: a serving or training process whose
// whole device-memory budget was handed to a framework's pool at start-up, a real-time loop where the
// implicit device synchronisation of an allocation is not acceptable, a plug-in that runs under a
// memory-accounting wrapper.  sgp_create allocates (schedule tables, launch scratch), so those callers
// get this handle-free entry point instead.  Everything the kernel needs beyond the caller's arrays --
// the step's in-neighbour table and the two launch words (ticket, status) -- lives in ONE file-scope
// device array that the library image carries; every GPU that loads the library holds those 40 KB
// until the process exits.
//
// The array's name is only a host-side stand-in for the symbol: its device address is asked of the
// runtime (cudaGetSymbolAddress) once per device, by the first call made with that device current,
// and that address is what the kernel receives.  That first call should therefore come before any
// stream capture.  All calls share the array and it keeps the previous call's contents: the table is
// rewritten and the launch words are cleared by every call, in stream order; two calls whose kernels
// can overlap on the GPU (different streams, no dependency) race on it and must not be issued.
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <mutex>

#include "launch.h"
#include "sgp.h"

namespace {

constexpr int kWordsBytes = 256;                                     // ticket, status, padding
constexpr size_t kRowptrBytes = (SGP_MAX_NODES + 1 + 3) / 4 * 4 * sizeof(int32_t);
constexpr size_t kScratchBytes = kWordsBytes + kRowptrBytes + 2 * SGP_STATIC_MAX_NNZ * sizeof(int32_t);

static __device__ __align__(256) unsigned char g_sgp_static_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
struct DeviceSetup {
  bool ready = false;
  unsigned char *scratch = nullptr;   // DEVICE address of g_sgp_static_scratch on this device
  int sm_count = 0;
  int smem_optin = 0;
};
DeviceSetup g_setup[kMaxDevices];
std::mutex g_setup_mutex;

// Once per device, with that device current: resolve the scratch symbol to its device address.
int ensure_setup(int *device_out, DeviceSetup *out) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
    (void)cudaGetLastError();
    return SGP_ERR_CUDA;
  }
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  DeviceSetup &s = g_setup[dev];
  if (!s.ready) {
    void *ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_sgp_static_scratch) != cudaSuccess || ptr == nullptr ||
        cudaDeviceGetAttribute(&s.sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&s.smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess) {
      (void)cudaGetLastError();
      return SGP_ERR_CUDA;
    }
    s.scratch = static_cast<unsigned char *>(ptr);
    s.ready = true;
  }
  *device_out = dev;
  *out = s;
  return SGP_OK;
}

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Same tile sizing, shared-memory budget, grid and kernel-attribute cache as the handle path.
int launch(const DeviceSetup &s, int dev, sgp::StepParams p, int vec, int64_t c0, int64_t c1, bool update_w, int upd,
           bool uniform_rows, cudaStream_t stream) {
  p.col_begin = c0;
  p.col_end = c1;
  p.update_w = update_w ? 1 : 0;
  sgp::DeviceInfo di;
  di.device = dev;
  di.sm_count = s.sm_count;
  di.smem_optin = s.smem_optin;
  sgp::RegsOptions opt;
  if (vec == 4) opt.tile_cols = sgp::regs_tile_cols(p.n, 4 * 1024);
  sgp::LaunchRecord rec;
  return sgp::launch_regs(di, p, nullptr, upd, vec, uniform_rows, opt, stream, &rec);
}

}  // namespace

extern "C" int sgp_step_static(int n, int64_t d, int64_t ld, const int32_t *h_rowptr, const int32_t *h_col,
                               const float *h_val, int64_t nnz, float *d_X, float *d_W, float *d_M, const float *d_G,
                               float *d_Z, float lr, float momentum, float weight_decay, int nesterov, void *stream) {
  if (n < 1 || n > SGP_MAX_NODES || d < 1 || ld < d || h_rowptr == nullptr || h_col == nullptr || h_val == nullptr ||
      d_X == nullptr || d_W == nullptr || d_G == nullptr || (momentum != 0.0f && d_M == nullptr))
    return SGP_ERR_ARG;
  if (nnz < n || nnz > SGP_STATIC_MAX_NNZ) return SGP_ERR_ARG;      // beyond the static table: use a handle
  if (h_rowptr[0] != 0 || h_rowptr[n] != nnz) return SGP_ERR_GRAPH;
  for (int i = 0; i < n; ++i)
    if (h_rowptr[i + 1] < h_rowptr[i]) return SGP_ERR_GRAPH;
  for (int64_t e = 0; e < nnz; ++e)
    if (h_col[e] < 0 || h_col[e] >= n || !std::isfinite(h_val[e]) || !(h_val[e] > 0.0f)) return SGP_ERR_GRAPH;
  {
    // the same acceptance rule as the schedule compiler: every sender's weights sum to one, self-loops present
    double colsum[SGP_MAX_NODES] = {0.0};
    int outdeg[SGP_MAX_NODES] = {0};
    bool has_self[SGP_MAX_NODES] = {false};
    for (int i = 0; i < n; ++i)
      for (int32_t e = h_rowptr[i]; e < h_rowptr[i + 1]; ++e) {
        const int j = h_col[e];
        if (e > h_rowptr[i] && h_col[e - 1] >= j) return SGP_ERR_GRAPH;      // senders ascending, no duplicates
        colsum[j] += static_cast<double>(h_val[e]);
        ++outdeg[j];
        if (j == i) has_self[j] = true;
      }
    for (int j = 0; j < n; ++j)
      if (!has_self[j] || std::fabs(colsum[j] - 1.0) > 4.0 * outdeg[j] * std::ldexp(1.0, -24)) return SGP_ERR_GRAPH;
  }

  int dev = 0;
  DeviceSetup s;
  const int rc = ensure_setup(&dev, &s);
  if (rc != SGP_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  {
    // The table uploads below read the caller's host arrays when they EXECUTE; inside a stream capture that would
    // be at every replay, long after this call returned.  Captured calls are therefore refused.
    cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(st, &cs) != cudaSuccess) {
      (void)cudaGetLastError();
      return SGP_ERR_CUDA;
    }
    if (cs != cudaStreamCaptureStatusNone) return SGP_ERR_STATE;
  }

  unsigned *words = reinterpret_cast<unsigned *>(s.scratch);
  int32_t *t_rowptr = reinterpret_cast<int32_t *>(s.scratch + kWordsBytes);
  int32_t *t_col = reinterpret_cast<int32_t *>(s.scratch + kWordsBytes + kRowptrBytes);
  float *t_val = reinterpret_cast<float *>(t_col + SGP_STATIC_MAX_NNZ);
  // the launch words must start at zero; the table is this step's (stream order keeps earlier kernels safe)
  if (cudaMemsetAsync(words, 0, kWordsBytes, st) != cudaSuccess ||
      cudaMemcpyAsync(t_rowptr, h_rowptr, (static_cast<size_t>(n) + 1) * sizeof(int32_t), cudaMemcpyHostToDevice, st) != cudaSuccess ||
      cudaMemcpyAsync(t_col, h_col, static_cast<size_t>(nnz) * sizeof(int32_t), cudaMemcpyHostToDevice, st) != cudaSuccess ||
      cudaMemcpyAsync(t_val, h_val, static_cast<size_t>(nnz) * sizeof(float), cudaMemcpyHostToDevice, st) != cudaSuccess) {
    (void)cudaGetLastError();
    return SGP_ERR_CUDA;
  }

  sgp::StepParams p{};
  p.X = d_X;
  p.W = d_W;
  p.M = momentum != 0.0f ? d_M : nullptr;
  p.G = d_G;
  p.Z = d_Z;
  p.ld = ld;
  p.n = n;
  p.nnz = static_cast<int>(nnz);
  p.lr = lr;
  p.momentum = momentum;
  p.wd = weight_decay;
  p.rowptr = t_rowptr;
  p.col = t_col;
  p.val = t_val;
  p.ticket = words;
  p.status = words + 1;

  // every receiver alike (complete graph): the mix is one shared column sum, as in the handle path
  bool uniform_rows = n > 1;
  for (int i = 1; i < n && uniform_rows; ++i) {
    const int32_t len = h_rowptr[1] - h_rowptr[0], b = h_rowptr[i];
    if (h_rowptr[i + 1] - b != len) uniform_rows = false;
    for (int32_t e = 0; e < len && uniform_rows; ++e)
      if (h_col[b + e] != h_col[e] || h_val[b + e] != h_val[e]) uniform_rows = false;
  }
  const int upd = momentum == 0.0f ? sgp::kUpdSgd : (nesterov != 0 ? sgp::kUpdNesterov : sgp::kUpdHeavyBall);
  const bool vec_ok = aligned16(d_X) && aligned16(d_G) && (p.M == nullptr || aligned16(p.M)) &&
                      (d_Z == nullptr || aligned16(d_Z)) && (ld % 4 == 0);
  const int64_t vec_end = vec_ok ? (d & ~int64_t{3}) : 0;
  if (vec_end > 0) {
    const int r = launch(s, dev, p, 4, 0, vec_end, vec_end == d, upd, uniform_rows, st);
    if (r != SGP_OK) return r;
  }
  if (vec_end == 0 && !uniform_rows && d >= 16) {
    // rows off the 16-byte grid: the peeled kernel, as on the handle path
    sgp::StepParams q = p;
    q.col_begin = 0;
    q.col_end = d;
    q.update_w = 1;
    sgp::DeviceInfo di;
    di.device = dev;
    di.sm_count = s.sm_count;
    di.smem_optin = s.smem_optin;
    sgp::LaunchRecord rec;
    const int r = sgp::launch_peel(di, q, nullptr, upd, sgp::PeelOptions{}, st, &rec);
    if (r != SGP_ERR_STATE) return r;
  }
  if (vec_end < d) return launch(s, dev, p, 1, vec_end, d, true, upd, uniform_rows, st);
  return SGP_OK;
}
