// Graph-schedule compiler: time-varying digraph -> per-step CSR in-neighbour lists (host only).
// Internal C++ view of the opaque sgp_schedule declared in include/sgp.h.
#pragma once
#include <cstdint>
#include <vector>

#include "sgp.h"

struct SgpStepCsr {
  std::vector<int32_t> rowptr;  // n + 1
  std::vector<int32_t> col;     // senders, ascending inside each row
  std::vector<float> val;       // p_ij
  int32_t max_indeg = 0;
  bool uniform_rows = false;    // every receiver has the same in-neighbour list and weights (e.g. the complete graph)
};

struct sgp_schedule {
  int n = 0;
  std::vector<SgpStepCsr> steps;  // one entry per slot of the period
  int64_t period() const { return static_cast<int64_t>(steps.size()); }
  const SgpStepCsr &slot(int64_t k) const { return steps[static_cast<size_t>(k % period())]; }
};

// Returns SGP_OK or an error code; *out is a new object on success.
int sgp_schedule_build(sgp_schedule **out, int n, const sgp_graph_desc *g);

// P = I: the mixing matrix of a step on which no node transmits (Alg. 2 lines 10-11).
SgpStepCsr sgp_identity_step(int n);
