#pragma once
#include <cstdint>
#include <vector>

#include "pasta_plan.h"
#include "pool.hpp"

namespace pasta {

struct PlanLimits {
  int32_t n_q_heads, n_kv_heads, head_dim;
  int32_t max_queries;   // queries of a step
  int32_t max_rows;      // partial rows per layer
  int64_t max_words;     // size of the device copy of the plan
  int32_t grid;          // CTAs the tensor-core kernel may use (one per SM)
  bool tensor_path;      // false: every stream goes to the warp-shuffle kernel
  int32_t tail_percent;  // share of every long run's tiles that is handed out at run time (0: everything is assigned)
  int32_t tail_tiles;    // tiles per unit of that share
};

// Plans the attention of one step: one query per element of `queries`, `slots` parallel to it.
pasta_status_t build_plan(const HostPool &pool, const std::vector<StepQuery> &queries,
                          const std::vector<Slot> &slots, const PlanLimits &lim,
                          std::vector<int32_t> *words);

}  // namespace pasta
