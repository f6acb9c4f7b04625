// Graph-schedule compiler (host C++, no CUDA): expands one period of the time-varying digraph of
// App. A / App. C into per-step CSR in-neighbour lists with fp32 mixing weights.
//
// Orientation: p_ij is the weight receiver i applies to sender j; CSR row i lists senders j in
// ascending order with the self-loop in its sorted place, so the mix of Alg. 1 line 6 is a
// deterministic left-to-right sum over the row.
#include "schedule.h"

#include <algorithm>
#include <cmath>
#include <new>
#include <utility>

namespace {

// floor(log2(n-1)) + 1 hop distances 2^0 .. 2^floor(log2(n-1)) (App. A); none for a single node.
int exp_cycle_length(int n) {
  int L = 0;
  for (unsigned v = static_cast<unsigned>(n - 1); v != 0; v >>= 1) ++L;
  return n <= 1 ? 0 : L;
}

// splitmix64 finaliser: integer-only, so the random digraph is reproducible bit for bit anywhere.
inline uint64_t mix64(uint64_t x) {
  x ^= x >> 30;
  x *= 0xBF58476D1CE4E5B9ull;
  x ^= x >> 27;
  x *= 0x94D049BB133111EBull;
  x ^= x >> 31;
  return x;
}

inline uint64_t graph_hash(uint64_t seed, uint64_t k, uint32_t i, uint32_t t) {
  const uint64_t a = mix64(seed + 0x9E3779B97F4A7C15ull);
  const uint64_t b = mix64(a ^ k);
  return mix64(b ^ ((static_cast<uint64_t>(i) << 32) | t));
}

using OutLists = std::vector<std::vector<int32_t>>;  // per sender: sorted unique receivers incl. self

void sort_unique(std::vector<int32_t> &v) {
  std::sort(v.begin(), v.end());
  v.erase(std::unique(v.begin(), v.end()), v.end());
}

OutLists exp_out_lists(int n, int64_t k, int peers) {
  const int L = exp_cycle_length(n);
  OutLists out(static_cast<size_t>(n));
  for (int i = 0; i < n; ++i) {
    auto &o = out[static_cast<size_t>(i)];
    o.push_back(i);
    for (int t = 0; t < peers && L > 0; ++t) {
      const int64_t hop = int64_t{1} << ((k + t) % L);
      o.push_back(static_cast<int32_t>((i + hop) % n));
    }
    sort_unique(o);
  }
  return out;
}

// Undirected bipartite exponential graph (App. A, "Undirected exponential graph"): odd node i pairs with the even
// node (i + hop) mod n, hop cycling through 2^1 - 1, 2^2 - 1, ..., 2^floor(log2(n-1)) - 1 (n = 2: the single
// hop 1); the even node answers, so every step is a perfect matching and P is symmetric.
std::vector<int> bipartite_hops(int n) {
  std::vector<int> hops;
  int top = 0;
  for (unsigned v = static_cast<unsigned>(n - 1); v > 1; v >>= 1) ++top;   // floor(log2(n-1))
  for (int j = 1; j <= top; ++j) hops.push_back((1 << j) - 1);
  if (hops.empty()) hops.push_back(1);
  return hops;
}

OutLists bipartite_out_lists(int n, int hop) {
  OutLists out(static_cast<size_t>(n));
  for (int i = 0; i < n; ++i) out[static_cast<size_t>(i)].push_back(i);
  for (int i = 1; i < n; i += 2) {
    const int j = (i + hop) % n;
    out[static_cast<size_t>(i)].push_back(j);
    out[static_cast<size_t>(j)].push_back(i);
  }
  for (auto &o : out) sort_unique(o);
  return out;
}

OutLists complete_out_lists(int n) {
  OutLists out(static_cast<size_t>(n));
  for (auto &o : out) {
    o.resize(static_cast<size_t>(n));
    for (int i = 0; i < n; ++i) o[static_cast<size_t>(i)] = i;
  }
  return out;
}

OutLists random_out_lists(int n, int64_t k, uint64_t seed, int max_outdeg) {
  OutLists out(static_cast<size_t>(n));
  const int cap = std::min(max_outdeg, n - 1);
  for (int i = 0; i < n; ++i) {
    auto &o = out[static_cast<size_t>(i)];
    o.push_back(i);
    if (cap >= 1) {
      const int deg = 1 + static_cast<int>(graph_hash(seed, static_cast<uint64_t>(k), i, 0) % cap);
      uint32_t t = 1;
      while (static_cast<int>(o.size()) < deg + 1) {
        const int32_t c = static_cast<int32_t>(graph_hash(seed, static_cast<uint64_t>(k), i, t++) % n);
        if (std::find(o.begin(), o.end(), c) == o.end()) o.push_back(c);
      }
    }
    std::sort(o.begin(), o.end());
  }
  return out;
}

// Uniform weights 1/|N_out_j| (App. C), transposed into receiver-major CSR.  Senders are visited in
// ascending order, so every row comes out sorted.
SgpStepCsr transpose_uniform(int n, const OutLists &out) {
  SgpStepCsr s;
  s.rowptr.assign(static_cast<size_t>(n) + 1, 0);
  for (const auto &o : out)
    for (int32_t i : o) ++s.rowptr[static_cast<size_t>(i) + 1];
  for (int i = 0; i < n; ++i) {
    s.max_indeg = std::max(s.max_indeg, s.rowptr[static_cast<size_t>(i) + 1]);
    s.rowptr[static_cast<size_t>(i) + 1] += s.rowptr[static_cast<size_t>(i)];
  }
  const size_t nnz = static_cast<size_t>(s.rowptr[static_cast<size_t>(n)]);
  s.col.resize(nnz);
  s.val.resize(nnz);
  std::vector<int32_t> fill(s.rowptr.begin(), s.rowptr.end() - 1);
  for (int j = 0; j < n; ++j) {
    const auto &o = out[static_cast<size_t>(j)];
    const float p = static_cast<float>(1.0 / static_cast<double>(o.size()));
    for (int32_t i : o) {
      const size_t e = static_cast<size_t>(fill[static_cast<size_t>(i)]++);
      s.col[e] = j;
      s.val[e] = p;
    }
  }
  return s;
}

// True when all rows of P are equal: then x_i' = sum_j p_j h_j is the same vector for every receiver.
bool rows_are_uniform(const SgpStepCsr &s, int n) {
  const int32_t len = s.rowptr[1] - s.rowptr[0];
  for (int i = 1; i < n; ++i) {
    const int32_t b = s.rowptr[static_cast<size_t>(i)];
    if (s.rowptr[static_cast<size_t>(i) + 1] - b != len) return false;
    for (int32_t e = 0; e < len; ++e)
      if (s.col[static_cast<size_t>(b + e)] != s.col[static_cast<size_t>(e)] ||
          s.val[static_cast<size_t>(b + e)] != s.val[static_cast<size_t>(e)])
        return false;
  }
  return true;
}

struct Edge {
  int32_t sender, receiver;
  float w;
};

int custom_step(int n, std::vector<Edge> &edges, SgpStepCsr *out) {
  std::sort(edges.begin(), edges.end(), [](const Edge &a, const Edge &b) {
    return a.receiver != b.receiver ? a.receiver < b.receiver : a.sender < b.sender;
  });
  for (size_t e = 1; e < edges.size(); ++e)
    if (edges[e].receiver == edges[e - 1].receiver && edges[e].sender == edges[e - 1].sender)
      return SGP_ERR_GRAPH;  // duplicate edge
  std::vector<double> colsum(static_cast<size_t>(n), 0.0);
  std::vector<int> outdeg(static_cast<size_t>(n), 0);
  std::vector<char> has_self(static_cast<size_t>(n), 0);
  SgpStepCsr s;
  s.rowptr.assign(static_cast<size_t>(n) + 1, 0);
  for (const Edge &e : edges) {
    ++s.rowptr[static_cast<size_t>(e.receiver) + 1];
    colsum[static_cast<size_t>(e.sender)] += static_cast<double>(e.w);
    ++outdeg[static_cast<size_t>(e.sender)];
    if (e.sender == e.receiver) has_self[static_cast<size_t>(e.sender)] = 1;
    s.col.push_back(e.sender);
    s.val.push_back(e.w);
  }
  for (int i = 0; i < n; ++i) {
    if (!has_self[static_cast<size_t>(i)]) return SGP_ERR_GRAPH;
    const double tol = 4.0 * outdeg[static_cast<size_t>(i)] * std::ldexp(1.0, -24);
    if (std::fabs(colsum[static_cast<size_t>(i)] - 1.0) > tol) return SGP_ERR_GRAPH;
    s.max_indeg = std::max(s.max_indeg, s.rowptr[static_cast<size_t>(i) + 1]);
    s.rowptr[static_cast<size_t>(i) + 1] += s.rowptr[static_cast<size_t>(i)];
  }
  *out = std::move(s);
  return SGP_OK;
}

}  // namespace

int sgp_schedule_build(sgp_schedule **out, int n, const sgp_graph_desc *g) {
  if (out == nullptr) return SGP_ERR_ARG;
  *out = nullptr;
  if (g == nullptr || n < 1 || n > SGP_MAX_NODES || g->reserved != 0) return SGP_ERR_ARG;
  sgp_schedule *s = new (std::nothrow) sgp_schedule;
  if (s == nullptr) return SGP_ERR_ALLOC;
  s->n = n;
  int rc = SGP_OK;
  try {
    switch (g->kind) {
      case SGP_GRAPH_EXP_PEERS: {
        if (g->peers < 1 || g->peers > 30) { rc = SGP_ERR_ARG; break; }
        const int period = std::max(1, exp_cycle_length(n));
        for (int k = 0; k < period; ++k) s->steps.push_back(transpose_uniform(n, exp_out_lists(n, k, g->peers)));
        break;
      }
      case SGP_GRAPH_COMPLETE:
        s->steps.push_back(transpose_uniform(n, complete_out_lists(n)));
        break;
      case SGP_GRAPH_BIPARTITE_EXP: {
        if (n < 2 || n % 2 != 0) { rc = SGP_ERR_ARG; break; }     // two halves of equal size
        for (int hop : bipartite_hops(n)) s->steps.push_back(transpose_uniform(n, bipartite_out_lists(n, hop)));
        break;
      }
      case SGP_GRAPH_RANDOM_OUTDEG: {
        if (g->max_outdeg < 1 || g->num_steps < 1 || g->num_steps > (1 << 20)) { rc = SGP_ERR_ARG; break; }
        for (int64_t k = 0; k < g->num_steps; ++k)
          s->steps.push_back(transpose_uniform(n, random_out_lists(n, k, g->seed, g->max_outdeg)));
        break;
      }
      case SGP_GRAPH_CUSTOM: {
        if (g->num_steps < 1 || g->num_steps > (1 << 20) || g->num_edges < 1 || g->edge_step == nullptr ||
            g->edge_sender == nullptr || g->edge_receiver == nullptr || g->edge_weight == nullptr) {
          rc = SGP_ERR_ARG;
          break;
        }
        std::vector<std::vector<Edge>> per_step(static_cast<size_t>(g->num_steps));
        for (int64_t e = 0; e < g->num_edges && rc == SGP_OK; ++e) {
          const int32_t st = g->edge_step[e], j = g->edge_sender[e], i = g->edge_receiver[e];
          const float w = g->edge_weight[e];
          if (st < 0 || st >= g->num_steps || j < 0 || j >= n || i < 0 || i >= n || !std::isfinite(w) || !(w > 0.0f))
            rc = SGP_ERR_GRAPH;
          else
            per_step[static_cast<size_t>(st)].push_back(Edge{j, i, w});
        }
        for (int64_t k = 0; k < g->num_steps && rc == SGP_OK; ++k) {
          SgpStepCsr csr;
          rc = custom_step(n, per_step[static_cast<size_t>(k)], &csr);
          if (rc == SGP_OK) s->steps.push_back(std::move(csr));
        }
        break;
      }
      default:
        rc = SGP_ERR_ARG;
    }
  } catch (const std::bad_alloc &) {
    rc = SGP_ERR_ALLOC;
  }
  if (rc != SGP_OK) {
    delete s;
    return rc;
  }
  for (SgpStepCsr &c : s->steps) c.uniform_rows = n > 1 && rows_are_uniform(c, n);
  *out = s;
  return SGP_OK;
}

SgpStepCsr sgp_identity_step(int n) {
  SgpStepCsr s;
  s.rowptr.resize(static_cast<size_t>(n) + 1);
  s.col.resize(static_cast<size_t>(n));
  s.val.assign(static_cast<size_t>(n), 1.0f);
  for (int i = 0; i <= n; ++i) s.rowptr[static_cast<size_t>(i)] = i;
  for (int i = 0; i < n; ++i) s.col[static_cast<size_t>(i)] = i;
  s.max_indeg = 1;
  s.uniform_rows = false;
  return s;
}

extern "C" {

int sgp_schedule_compile(sgp_schedule **out, int n, const sgp_graph_desc *g) { return sgp_schedule_build(out, n, g); }

int sgp_schedule_destroy(sgp_schedule *s) {
  delete s;
  return SGP_OK;
}

int sgp_schedule_period(const sgp_schedule *s, int64_t *period) {
  if (s == nullptr || period == nullptr) return SGP_ERR_ARG;
  *period = s->period();
  return SGP_OK;
}

int sgp_schedule_nnz(const sgp_schedule *s, int64_t k, int64_t *nnz) {
  if (s == nullptr || nnz == nullptr || k < 0) return SGP_ERR_ARG;
  *nnz = static_cast<int64_t>(s->slot(k).col.size());
  return SGP_OK;
}

int sgp_schedule_get(const sgp_schedule *s, int64_t k, int32_t *rowptr, int32_t *col, float *val, int64_t cap,
                     int64_t *nnz) {
  if (s == nullptr || rowptr == nullptr || col == nullptr || val == nullptr || nnz == nullptr || k < 0)
    return SGP_ERR_ARG;
  const SgpStepCsr &c = s->slot(k);
  *nnz = static_cast<int64_t>(c.col.size());
  if (cap < *nnz) return SGP_ERR_ARG;
  std::copy(c.rowptr.begin(), c.rowptr.end(), rowptr);
  std::copy(c.col.begin(), c.col.end(), col);
  std::copy(c.val.begin(), c.val.end(), val);
  return SGP_OK;
}

}  // extern "C"
