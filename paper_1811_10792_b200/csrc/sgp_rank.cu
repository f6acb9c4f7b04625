// C ABI of the one-node-per-GPU SGP step (see include/sgp.h, "One node per GPU"): handle, message slots,
// peer tables and launches.  The arithmetic is in rank_kernels.cuh.
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstring>
#include <new>
#include <vector>

#include "rank_kernels.cuh"
#include "schedule.h"
#include "sgp.h"

struct sgp_rank {
  int rank = 0, world = 0, tau = 0, slots = 0;
  unsigned flags = 0;
  int64_t d = 0, slot_floats = 0, w_offset = 0;
  int device = 0, sm_count = 0;
  sgp_schedule *sched = nullptr;
  float *block = nullptr;                 // slots x slot_floats, this rank's messages
  std::vector<const float *> peer_block;  // where every rank's block is mapped in this process
  unsigned *d_words = nullptr;            // [0] ticket, [1] status
  int last_cuda_error = 0;
  int64_t send_period = 1;                // nodes transmit on steps k with k mod send_period == 0 (Alg. 2 line 5)
};

namespace {

#define SGP_RANK_TRY(r, expr)                                   \
  do {                                                          \
    cudaError_t e_ = (expr);                                    \
    if (e_ != cudaSuccess) {                                    \
      if (r) (r)->last_cuda_error = static_cast<int>(e_);       \
      (void)cudaGetLastError();                                 \
      return SGP_ERR_CUDA;                                      \
    }                                                           \
  } while (0)

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

inline int update_kind(float momentum, int nesterov) {
  if (momentum == 0.0f) return sgp::kUpdSgd;
  return nesterov != 0 ? sgp::kUpdNesterov : sgp::kUpdHeavyBall;
}

// Grid of a streaming rank kernel: exactly the CTAs that are resident at once (one wave, grid-stride inside), so
// that no partial second wave is left at the end of a launch that lasts only ~100 us.
// `cap` bounds the CTAs per SM: the fused overlap kernel (four to five loads and as many stores per vector) is
// fastest with four (0.911 of the copy bandwidth against 0.896 with the five to six the occupancy query allows and
// 0.82 with three); the lighter update and mix kernels want every CTA they can get (0.92 with eight, 0.83 with four).
template <typename Kernel>
unsigned stream_grid(const sgp_rank *r, bool vec, Kernel kern, int cap = 64) {
  const int64_t work = vec ? std::max<int64_t>(1, r->d >> 2) : r->d;
  int per_sm = 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, sgp::kRankThreads, 0) != cudaSuccess || per_sm < 1) {
    (void)cudaGetLastError();
    per_sm = 4;
  }
  per_sm = std::min(per_sm, cap);
  return static_cast<unsigned>(std::max<int64_t>(1, std::min<int64_t>((work + sgp::kRankThreads - 1) / sgp::kRankThreads,
                                                                      static_cast<int64_t>(r->sm_count) * per_sm)));
}

int check_device(const sgp_rank *r) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) {
    (void)cudaGetLastError();
    return SGP_ERR_CUDA;
  }
  return dev == r->device ? SGP_OK : SGP_ERR_STATE;
}

// Turns a plan into device pointers: entry e reads the sender's slot `read_slot` (this rank's own block for itself).
int make_sources(const sgp_rank *r, const sgp_rank_plan_t &plan, sgp::RankSources *out) {
  sgp::RankSources s{};
  s.count = plan.count;
  s.self_pos = plan.self_pos;
  for (int e = 0; e < plan.count; ++e) {
    const int j = plan.sender[e];
    const float *base = j == r->rank ? r->block : r->peer_block[static_cast<size_t>(j)];
    if (base == nullptr) return SGP_ERR_STATE;          // sgp_rank_set_peers has not supplied this peer
    s.src[e] = base + static_cast<int64_t>(plan.read_slot) * r->slot_floats;
    s.weight[e] = plan.weight[e];
  }
  *out = s;
  return SGP_OK;
}

void fill_params(const sgp_rank *r, sgp::RankParams *p) {
  p->d = r->d;
  p->w_offset = r->w_offset;
  p->biased = (r->flags & SGP_FLAG_BIASED) ? 1 : 0;
  p->ticket = r->d_words;
  p->status = r->d_words + 1;
}

}  // namespace

extern "C" {

int sgp_rank_plan_period(const sgp_schedule *s, int rank, int64_t k, int tau, int64_t send_period, sgp_rank_plan_t *out) {
  if (s == nullptr || out == nullptr || rank < 0 || rank >= s->n || k < 0 || tau < 0 || tau > 64 || send_period < 1)
    return SGP_ERR_ARG;
  sgp_rank_plan_t plan;
  std::memset(&plan, 0, sizeof(plan));
  const int slots = tau + 2;
  plan.write_slot = static_cast<int32_t>(k % slots);
  plan.self_pos = -1;
  // Matrix of step kk: the c-th transmission (kk = c * send_period) uses P^(c); a step on which nobody transmits
  // mixes with the identity (Alg. 2 lines 5-12).
  const bool sends_now = k % send_period == 0;
  const int64_t k_arrive = k - tau;                       // the step whose messages arrive now
  const bool arrives = tau == 0 ? sends_now : (k_arrive >= 0 && k_arrive % send_period == 0);
  plan.self_weight = 1.0f;
  if (sends_now) {
    // the self weight is this step's p_ii
    const SgpStepCsr &now = s->slot(k / send_period);
    for (int32_t e = now.rowptr[static_cast<size_t>(rank)]; e < now.rowptr[static_cast<size_t>(rank) + 1]; ++e)
      if (now.col[static_cast<size_t>(e)] == rank) plan.self_weight = now.val[static_cast<size_t>(e)];
  }
  if (tau == 0) {
    plan.read_slot = plan.write_slot;
    if (arrives) {
      const SgpStepCsr &c = s->slot(k / send_period);
      const int32_t b = c.rowptr[static_cast<size_t>(rank)], e1 = c.rowptr[static_cast<size_t>(rank) + 1];
      if (e1 - b > SGP_RANK_MAX_SOURCES) return SGP_ERR_ARG;
      for (int32_t e = b; e < e1; ++e) {
        if (c.col[static_cast<size_t>(e)] == rank) plan.self_pos = plan.count;
        plan.sender[plan.count] = c.col[static_cast<size_t>(e)];
        plan.weight[plan.count] = c.val[static_cast<size_t>(e)];
        ++plan.count;
      }
    } else {
      plan.self_pos = 0;                                   // identity: the node keeps its whole half step
      plan.sender[0] = rank;
      plan.weight[0] = 1.0f;
      plan.count = 1;
    }
  } else {
    plan.read_slot = static_cast<int32_t>(((k - tau) % slots + slots) % slots);
    if (arrives) {
      // the messages that arrive now were sent, and weighted, with the matrix of step k - tau
      const SgpStepCsr &c = s->slot(k_arrive / send_period);
      const int32_t b = c.rowptr[static_cast<size_t>(rank)], e1 = c.rowptr[static_cast<size_t>(rank) + 1];
      if (e1 - b - 1 > SGP_RANK_MAX_SOURCES) return SGP_ERR_ARG;
      for (int32_t e = b; e < e1; ++e) {
        if (c.col[static_cast<size_t>(e)] == rank) continue;
        plan.sender[plan.count] = c.col[static_cast<size_t>(e)];
        plan.weight[plan.count] = c.val[static_cast<size_t>(e)];
        ++plan.count;
      }
    }
  }
  *out = plan;
  return SGP_OK;
}

int sgp_rank_plan(const sgp_schedule *s, int rank, int64_t k, int tau, sgp_rank_plan_t *out) {
  return sgp_rank_plan_period(s, rank, k, tau, 1, out);
}

int sgp_rank_set_send_period(sgp_rank *r, int64_t send_period) {
  if (r == nullptr || send_period < 1 || send_period > (1 << 20)) return SGP_ERR_ARG;
  r->send_period = send_period;
  return SGP_OK;
}

int sgp_rank_create(sgp_rank **out, int rank, int world, int64_t d, const sgp_graph_desc *g, int tau, unsigned flags) {
  if (out == nullptr) return SGP_ERR_ARG;
  *out = nullptr;
  if (world < 1 || world > SGP_MAX_NODES || rank < 0 || rank >= world || d < 1 || g == nullptr || tau < 0 || tau > 64 ||
      (flags & ~SGP_FLAG_BIASED) != 0)
    return SGP_ERR_ARG;
  sgp_schedule *sched = nullptr;
  const int rc = sgp_schedule_build(&sched, world, g);
  if (rc != SGP_OK) return rc;
  sgp_rank *r = new (std::nothrow) sgp_rank;
  if (r == nullptr) {
    delete sched;
    return SGP_ERR_ALLOC;
  }
  r->rank = rank;
  r->world = world;
  r->tau = tau;
  r->slots = tau + 2;
  r->flags = flags;
  r->d = d;
  // every slot starts on a 1 KB boundary (the row-pitch lesson of the stacked kernels); the weight sits in the pad
  r->w_offset = (d + 255) / 256 * 256;
  r->slot_floats = r->w_offset + 256;
  r->sched = sched;
  r->peer_block.assign(static_cast<size_t>(world), nullptr);
  auto fail = [&](int code) {
    cudaFree(r->block);
    cudaFree(r->d_words);
    delete r->sched;
    delete r;
    (void)cudaGetLastError();
    return code;
  };
  if (cudaGetDevice(&r->device) != cudaSuccess) return fail(SGP_ERR_CUDA);
  if (cudaDeviceGetAttribute(&r->sm_count, cudaDevAttrMultiProcessorCount, r->device) != cudaSuccess) return fail(SGP_ERR_CUDA);
  const size_t bytes = static_cast<size_t>(r->slots) * r->slot_floats * sizeof(float);
  if (cudaMalloc(&r->block, bytes) != cudaSuccess) return fail(SGP_ERR_ALLOC);
  if (cudaMalloc(&r->d_words, 2 * sizeof(unsigned)) != cudaSuccess) return fail(SGP_ERR_ALLOC);
  if (cudaMemset(r->block, 0, bytes) != cudaSuccess || cudaMemset(r->d_words, 0, 2 * sizeof(unsigned)) != cudaSuccess ||
      cudaDeviceSynchronize() != cudaSuccess)
    return fail(SGP_ERR_CUDA);
  *out = r;
  return SGP_OK;
}

int sgp_rank_destroy(sgp_rank *r) {
  if (r == nullptr) return SGP_OK;
  (void)cudaDeviceSynchronize();
  cudaFree(r->block);
  cudaFree(r->d_words);
  delete r->sched;
  delete r;
  return SGP_OK;
}

int sgp_rank_message_block(sgp_rank *r, void **d_block, size_t *bytes) {
  if (r == nullptr || d_block == nullptr || bytes == nullptr) return SGP_ERR_ARG;
  *d_block = r->block;
  *bytes = static_cast<size_t>(r->slots) * r->slot_floats * sizeof(float);
  return SGP_OK;
}

int sgp_rank_set_peers(sgp_rank *r, void *const *d_peer_blocks) {
  if (r == nullptr || d_peer_blocks == nullptr) return SGP_ERR_ARG;
  for (int j = 0; j < r->world; ++j) {
    if (j == r->rank) continue;
    if (d_peer_blocks[j] != nullptr && !aligned16(d_peer_blocks[j])) return SGP_ERR_ARG;
    r->peer_block[static_cast<size_t>(j)] = static_cast<const float *>(d_peer_blocks[j]);
  }
  return SGP_OK;
}

int sgp_rank_get_schedule(const sgp_rank *r, const sgp_schedule **s) {
  if (r == nullptr || s == nullptr) return SGP_ERR_ARG;
  *s = r->sched;
  return SGP_OK;
}

}  // extern "C"

namespace {

sgp::UpdateScalars adam_scalars(float lr, float beta1, float beta2, float eps, float weight_decay, int64_t t) {
  // bias corrections in double, rounded once (t >= 1), as in the stacked Adam step
  const double bc1 = 1.0 - std::pow(static_cast<double>(beta1), static_cast<double>(t));
  const double bc2 = 1.0 - std::pow(static_cast<double>(beta2), static_cast<double>(t));
  return sgp::UpdateScalars{lr, 0.0f, weight_decay, beta1, beta2, eps, static_cast<float>(static_cast<double>(lr) / bc1),
                            static_cast<float>(1.0 / std::sqrt(bc2))};
}

bool adam_args_ok(int64_t t, float beta1, float beta2, float eps) {
  return t >= 1 && beta1 >= 0.0f && beta1 < 1.0f && beta2 >= 0.0f && beta2 < 1.0f && eps >= 0.0f;
}

int rank_update(sgp_rank *r, const float *d_x, float *d_w, float *d_m, float *d_v, const float *d_g, int64_t k, int upd,
                const sgp::UpdateScalars &us, void *stream) {
  int rc = check_device(r);
  if (rc != SGP_OK) return rc;
  sgp::RankParams p{};
  fill_params(r, &p);
  p.x = const_cast<float *>(d_x);
  p.w = d_w;
  p.m = d_m;
  p.v = d_v;
  p.g = d_g;
  p.msg = r->block + (k % r->slots) * r->slot_floats;
  p.us = us;
  const bool vec = aligned16(d_x) && aligned16(d_g) && (d_m == nullptr || aligned16(d_m)) && (d_v == nullptr || aligned16(d_v));
  cudaStream_t st = static_cast<cudaStream_t>(stream);
#define SGP_LAUNCH_ONE(KERNEL, ...) KERNEL<<<stream_grid(r, vec, KERNEL), sgp::kRankThreads, 0, st>>>(__VA_ARGS__)
#define SGP_LAUNCH_UPDATE(VEC)                                                                  \
  switch (upd) {                                                                                \
    case sgp::kUpdSgd: SGP_LAUNCH_ONE((sgp::sgp_rank_update_kernel<VEC, sgp::kUpdSgd>), p); break; \
    case sgp::kUpdHeavyBall: SGP_LAUNCH_ONE((sgp::sgp_rank_update_kernel<VEC, sgp::kUpdHeavyBall>), p); break; \
    case sgp::kUpdNesterov: SGP_LAUNCH_ONE((sgp::sgp_rank_update_kernel<VEC, sgp::kUpdNesterov>), p); break; \
    default: SGP_LAUNCH_ONE((sgp::sgp_rank_update_kernel<VEC, sgp::kUpdAdam>), p);               \
  }
  if (vec) { SGP_LAUNCH_UPDATE(4) } else { SGP_LAUNCH_UPDATE(1) }
#undef SGP_LAUNCH_UPDATE
  SGP_RANK_TRY(r, cudaGetLastError());
  return SGP_OK;
}

int rank_overlap(sgp_rank *r, float *d_x, float *d_w, float *d_m, float *d_v, const float *d_g, float *d_z, int64_t k, int upd,
                 const sgp::UpdateScalars &us, void *stream) {
  if (r->tau < 1) return SGP_ERR_STATE;                  // without a delay the peers' messages are not there yet
  int rc = check_device(r);
  if (rc != SGP_OK) return rc;
  sgp_rank_plan_t plan;
  rc = sgp_rank_plan_period(r->sched, r->rank, k, r->tau, r->send_period, &plan);
  if (rc != SGP_OK) return rc;
  sgp::RankSources s;
  rc = make_sources(r, plan, &s);
  if (rc != SGP_OK) return rc;
  sgp::RankParams p{};
  fill_params(r, &p);
  p.x = d_x;
  p.w = d_w;
  p.m = d_m;
  p.v = d_v;
  p.g = d_g;
  p.z = d_z;
  p.msg = r->block + static_cast<int64_t>(plan.write_slot) * r->slot_floats;
  p.self_weight = plan.self_weight;
  p.us = us;
  const bool vec = aligned16(d_x) && aligned16(d_g) && (d_m == nullptr || aligned16(d_m)) && (d_v == nullptr || aligned16(d_v)) &&
                   (d_z == nullptr || aligned16(d_z));
  cudaStream_t st = static_cast<cudaStream_t>(stream);
#define SGP_LAUNCH_CAPPED(KERNEL, ...) KERNEL<<<stream_grid(r, vec, KERNEL, 4), sgp::kRankThreads, 0, st>>>(__VA_ARGS__)
#define SGP_LAUNCH_OVERLAP(VEC, HZ)                                                                          \
  switch (upd) {                                                                                             \
    case sgp::kUpdSgd: SGP_LAUNCH_CAPPED((sgp::sgp_rank_overlap_kernel<VEC, sgp::kUpdSgd, HZ>), p, s); break;    \
    case sgp::kUpdHeavyBall: SGP_LAUNCH_CAPPED((sgp::sgp_rank_overlap_kernel<VEC, sgp::kUpdHeavyBall, HZ>), p, s); break; \
    case sgp::kUpdNesterov: SGP_LAUNCH_CAPPED((sgp::sgp_rank_overlap_kernel<VEC, sgp::kUpdNesterov, HZ>), p, s); break; \
    default: SGP_LAUNCH_CAPPED((sgp::sgp_rank_overlap_kernel<VEC, sgp::kUpdAdam, HZ>), p, s);                    \
  }
  if (vec) {
    if (d_z) { SGP_LAUNCH_OVERLAP(4, true) } else { SGP_LAUNCH_OVERLAP(4, false) }
  } else {
    if (d_z) { SGP_LAUNCH_OVERLAP(1, true) } else { SGP_LAUNCH_OVERLAP(1, false) }
  }
#undef SGP_LAUNCH_CAPPED
#undef SGP_LAUNCH_OVERLAP
  SGP_RANK_TRY(r, cudaGetLastError());
  return SGP_OK;
}

}  // namespace

extern "C" {

int sgp_rank_update(sgp_rank *r, const float *d_x, float *d_w, float *d_m, const float *d_g, int64_t k, float lr,
                    float momentum, float weight_decay, int nesterov, void *stream) {
  if (r == nullptr || d_x == nullptr || d_w == nullptr || d_g == nullptr || k < 0 || (momentum != 0.0f && d_m == nullptr))
    return SGP_ERR_ARG;
  return rank_update(r, d_x, d_w, momentum != 0.0f ? d_m : nullptr, nullptr, d_g, k, update_kind(momentum, nesterov),
                     sgp::UpdateScalars{lr, momentum, weight_decay, 0.f, 0.f, 0.f, 0.f, 0.f}, stream);
}

int sgp_rank_update_adam(sgp_rank *r, const float *d_x, float *d_w, float *d_m1, float *d_m2, const float *d_g, int64_t k,
                         int64_t t, float lr, float beta1, float beta2, float eps, float weight_decay, void *stream) {
  if (r == nullptr || d_x == nullptr || d_w == nullptr || d_m1 == nullptr || d_m2 == nullptr || d_g == nullptr || k < 0 ||
      !adam_args_ok(t, beta1, beta2, eps))
    return SGP_ERR_ARG;
  return rank_update(r, d_x, d_w, d_m1, d_m2, d_g, k, sgp::kUpdAdam, adam_scalars(lr, beta1, beta2, eps, weight_decay, t), stream);
}

int sgp_rank_mix(sgp_rank *r, float *d_x, float *d_w, float *d_z, int64_t k, void *stream) {
  if (r == nullptr || d_x == nullptr || d_w == nullptr || k < 0) return SGP_ERR_ARG;
  if (r->tau != 0) return SGP_ERR_STATE;                 // with a delay the step is one fused kernel
  int rc = check_device(r);
  if (rc != SGP_OK) return rc;
  sgp_rank_plan_t plan;
  rc = sgp_rank_plan_period(r->sched, r->rank, k, 0, r->send_period, &plan);
  if (rc != SGP_OK) return rc;
  sgp::RankSources s;
  rc = make_sources(r, plan, &s);
  if (rc != SGP_OK) return rc;
  sgp::RankParams p{};
  fill_params(r, &p);
  p.x = d_x;
  p.w = d_w;
  p.z = d_z;
  const bool vec = aligned16(d_x) && (d_z == nullptr || aligned16(d_z));
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (vec) {
    if (d_z) SGP_LAUNCH_ONE((sgp::sgp_rank_mix_kernel<4, true>), p, s);
    else SGP_LAUNCH_ONE((sgp::sgp_rank_mix_kernel<4, false>), p, s);
  } else {
    if (d_z) SGP_LAUNCH_ONE((sgp::sgp_rank_mix_kernel<1, true>), p, s);
    else SGP_LAUNCH_ONE((sgp::sgp_rank_mix_kernel<1, false>), p, s);
  }
  SGP_RANK_TRY(r, cudaGetLastError());
  return SGP_OK;
}

int sgp_rank_step_overlap(sgp_rank *r, float *d_x, float *d_w, float *d_m, const float *d_g, float *d_z, int64_t k,
                          float lr, float momentum, float weight_decay, int nesterov, void *stream) {
  if (r == nullptr || d_x == nullptr || d_w == nullptr || d_g == nullptr || k < 0 || (momentum != 0.0f && d_m == nullptr))
    return SGP_ERR_ARG;
  return rank_overlap(r, d_x, d_w, momentum != 0.0f ? d_m : nullptr, nullptr, d_g, d_z, k, update_kind(momentum, nesterov),
                      sgp::UpdateScalars{lr, momentum, weight_decay, 0.f, 0.f, 0.f, 0.f, 0.f}, stream);
}

int sgp_rank_step_overlap_adam(sgp_rank *r, float *d_x, float *d_w, float *d_m1, float *d_m2, const float *d_g, float *d_z,
                               int64_t k, int64_t t, float lr, float beta1, float beta2, float eps, float weight_decay,
                               void *stream) {
  if (r == nullptr || d_x == nullptr || d_w == nullptr || d_m1 == nullptr || d_m2 == nullptr || d_g == nullptr || k < 0 ||
      !adam_args_ok(t, beta1, beta2, eps))
    return SGP_ERR_ARG;
  return rank_overlap(r, d_x, d_w, d_m1, d_m2, d_g, d_z, k, sgp::kUpdAdam, adam_scalars(lr, beta1, beta2, eps, weight_decay, t),
                      stream);
}

int sgp_rank_device_status(sgp_rank *r, unsigned *status) {
  if (r == nullptr || status == nullptr) return SGP_ERR_ARG;
  SGP_RANK_TRY(r, cudaDeviceSynchronize());
  SGP_RANK_TRY(r, cudaMemcpy(status, r->d_words + 1, sizeof(unsigned), cudaMemcpyDeviceToHost));
  return SGP_OK;
}

int sgp_ipc_export(const void *d_ptr, unsigned char *handle) {
  if (d_ptr == nullptr || handle == nullptr) return SGP_ERR_ARG;
  static_assert(sizeof(cudaIpcMemHandle_t) == SGP_IPC_HANDLE_BYTES, "handle size");
  cudaIpcMemHandle_t hd;
  if (cudaIpcGetMemHandle(&hd, const_cast<void *>(d_ptr)) != cudaSuccess) {
    (void)cudaGetLastError();
    return SGP_ERR_CUDA;
  }
  std::memcpy(handle, &hd, sizeof(hd));
  return SGP_OK;
}

int sgp_ipc_open(const unsigned char *handle, void **d_ptr) {
  if (handle == nullptr || d_ptr == nullptr) return SGP_ERR_ARG;
  cudaIpcMemHandle_t hd;
  std::memcpy(&hd, handle, sizeof(hd));
  if (cudaIpcOpenMemHandle(d_ptr, hd, cudaIpcMemLazyEnablePeerAccess) != cudaSuccess) {
    (void)cudaGetLastError();
    *d_ptr = nullptr;
    return SGP_ERR_CUDA;
  }
  return SGP_OK;
}

int sgp_ipc_close(void *d_ptr) {
  if (d_ptr == nullptr) return SGP_OK;
  if (cudaIpcCloseMemHandle(d_ptr) != cudaSuccess) {
    (void)cudaGetLastError();
    return SGP_ERR_CUDA;
  }
  return SGP_OK;
}

}  // extern "C"
