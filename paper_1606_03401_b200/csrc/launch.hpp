// Kernel launches with programmatic stream serialization: the launched kernel may become
// resident (and run its prologue: barrier set-up, TMEM allocation) while the previous kernel of
// the stream is still running.  Every kernel launched through here calls grid_dep_wait before
// its first access to global memory.  MEBPTT_NO_PDL in the environment turns the attribute off.
#pragma once

#include <cuda_runtime.h>

#include <atomic>
#include <cstdlib>

#include "env.hpp"

namespace mebptt {

inline bool pdl_enabled() { return !env::no_pdl(); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_on(bool pdl, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s,
                             Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = s;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = (pdl && pdl_enabled()) ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s,
                              Args&&... args) {
  return launch_on(true, kernel, grid, block, smem, s, static_cast<Args&&>(args)...);
}

// Cooperative launch (all CTAs co-resident), optionally in clusters of `cluster` CTAs, with
// programmatic stream serialization if the driver accepts the combination: the first refusal
// turns the attribute off for every later cooperative launch of the process.
inline cudaError_t launch_coop(const void* fn, int grid, int block, size_t smem, cudaStream_t s, void** args,
                               int cluster, bool early = true) {
  static std::atomic<int> pdl_state{-1};   // -1 untried, 0 refused, 1 accepted
  for (;;) {
    const bool pdl = early && pdl_enabled() && pdl_state.load() != 0;
    cudaLaunchAttribute at[3];
    int n = 0;
    at[n].id = cudaLaunchAttributeCooperative;
    at[n].val.cooperative = 1;
    ++n;
    if (cluster > 1) {
      at[n].id = cudaLaunchAttributeClusterDimension;
      at[n].val.clusterDim.x = (unsigned)cluster; at[n].val.clusterDim.y = 1; at[n].val.clusterDim.z = 1;
      ++n;
    }
    if (pdl) {
      at[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
      at[n].val.programmaticStreamSerializationAllowed = 1;
      ++n;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid); cfg.blockDim = dim3((unsigned)block); cfg.dynamicSmemBytes = smem; cfg.stream = s;
    cfg.attrs = at; cfg.numAttrs = (unsigned)n;
    const cudaError_t e = cudaLaunchKernelExC(&cfg, fn, args);
    if (e == cudaSuccess) {
      if (pdl) pdl_state.store(1);
      return e;
    }
    if (!pdl || pdl_state.load() == 1) return e;
    cudaGetLastError();
    pdl_state.store(0);
  }
}

}  // namespace mebptt
