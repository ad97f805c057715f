// Internal definition of the plan object behind mebptt_plan_t.
#pragma once

#include <cstdint>
#include <vector>

#include "mebptt.h"

namespace mebptt {

struct Plan {
  uint64_t id = 0;          // unique per plan object of the process (what cached per-plan data is keyed by)
  int64_t t = 0, m = 0;
  int mode = 0, alpha = 4, beta = 0;
  int sigma = 1;            // size of a hidden state in the unit m is counted in (1 unless planned over byte sizes)
  int64_t cost = 0;         // C(t, m)
  int64_t peak_units = 0;   // paper's accounting
  int64_t arena_units = 0;  // physical hidden-state units the arena must hold
  // row-major [t + 1][m + 1]
  std::vector<int64_t> C;
  std::vector<int32_t> D, D2;
  std::vector<uint8_t> H;
  std::vector<mebptt_op> tape;
};

int build_plan(int64_t t, int64_t m, int mode, int alpha, int beta, Plan** out, int sigma = 1);
int build_chen_plan(int64_t t, int alpha, int beta, Plan** out);
int build_chen_recursive_plan(int64_t t, int k, int alpha, int beta, Plan** out);
int validate_plan(const Plan& p);

}  // namespace mebptt
