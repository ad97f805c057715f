// The environment switches the library reads, all in one place.  None of them is part of the
// interface: they are aids for measuring and for verifying that two ways of doing the same thing
// give the same bits, read once per process.
//
//   MEBPTT_NO_PDL=1           launch without programmatic stream serialization
//   MEBPTT_NO_OVERLAP=1       weight-gradient GEMMs on the caller's stream instead of the side stream;
//                             host-buffer inputs copied in front of the step instead of beside it
//   MEBPTT_PRIORITY=1         the step on a stream of the library's, of the most urgent priority, instead
//                             of the caller's stream itself
//   MEBPTT_NO_ZX_AHEAD=1      input projections in the step's stream, when a run needs them, instead of a
//                             window ahead on a stream of their own
//   MEBPTT_BWD_CLUSTER=0|4|8  backward run kernel: unclustered (what a profiler that cannot launch
//                             clustered cooperative grids can capture), or the cluster size
//   MEBPTT_NO_BWD_GROUPS=1    backward run kernel without groups of batch rows (same bits)
//   MEBPTT_NO_SPLITK=1        no contraction is split along K (other rounding on the step-by-step paths)
//   MEBPTT_STEPWISE_PER_OP=1  step-by-step paths operation by operation instead of in runs (same bits)
//   MEBPTT_PLAN_SCAN=1        the planner scans every split point instead of walking convex columns
//                             (same tables)
//   MEBPTT_DEBUG=1            failed CUDA calls are named on stderr
#pragma once

#include <cstdlib>

namespace mebptt {
namespace env {

inline bool flag(const char* name) {
  const char* v = getenv(name);
  return v != nullptr && v[0] != '\0' && !(v[0] == '0' && v[1] == '\0');
}
// -1 when the variable is not set
inline int integer(const char* name) {
  const char* v = getenv(name);
  return (v && v[0]) ? atoi(v) : -1;
}

inline bool no_pdl() { static const bool v = flag("MEBPTT_NO_PDL"); return v; }
inline bool no_overlap() { static const bool v = flag("MEBPTT_NO_OVERLAP"); return v; }
inline bool priority() { static const bool v = flag("MEBPTT_PRIORITY"); return v; }
inline bool no_zx_ahead() { static const bool v = flag("MEBPTT_NO_ZX_AHEAD"); return v; }
inline int bwd_cluster() { static const int v = integer("MEBPTT_BWD_CLUSTER"); return v; }
inline bool no_bwd_groups() { static const bool v = flag("MEBPTT_NO_BWD_GROUPS"); return v; }
inline bool no_splitk() { static const bool v = flag("MEBPTT_NO_SPLITK"); return v; }
inline bool stepwise_per_op() { return flag("MEBPTT_STEPWISE_PER_OP"); }   // read per call: tests switch it
inline bool plan_scan() { return flag("MEBPTT_PLAN_SCAN"); }               // likewise
inline bool debug() { static const bool v = flag("MEBPTT_DEBUG"); return v; }

}  // namespace env
}  // namespace mebptt
