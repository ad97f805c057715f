// mebptt_lstm_train_step_static: the training step for callers that may not allocate device
// memory.  Its workspace is a fixed array that lives inside the library image.
//
// The ordinary entry point leaves the workspace to the caller, which normally means a
// cudaMalloc (or a framework allocator on top of one) sized by mebptt_lstm_workspace_bytes().
// Some callers cannot do that at the point where they train: code that runs after the process
// has handed all free device memory to another component, plug-ins that are only given input
// and output buffers by their host application, and set-ups where any allocation would stall
// other streams on the device.  For them the scratch is a fixed array in the library image.
//
// When the array takes up device memory: this file is a module of its own, and with CUDA's
// default lazy module loading a module is placed on a device when something of it is first
// asked for -- here the symbol look-up of the first call on that device (at load time only with
// CUDA_MODULE_LOADING=EAGER).  That first call is therefore a set-up call, to be made while
// device memory is still available; afterwards the array stays until the process exits.
#include <cuda_runtime.h>

#include <cstdint>
#include <mutex>

#include "mebptt.h"

namespace mebptt {
// The training step with a switch for the library-owned side stream (api.cu).
int train_step_impl(const mebptt_lstm_desc* desc, const mebptt_plan_t* plan, const void* W, const void* b,
                    const void* W_out, const void* b_out, const void* x, const void* targets, const void* h0,
                    const void* c0, void* workspace, size_t workspace_bytes, void* stream, float* loss, float* dW,
                    float* db, float* dW_out, float* db_out, float* dx, int64_t* counters, bool side_stream);
}

namespace {

// Every GPU on which the entry point below has been called holds this array until the process exits.
static __device__ __align__(256) unsigned char g_static_workspace[MEBPTT_STATIC_WORKSPACE_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_mutex;
void* g_device_ptr[kMaxDevices] = {};

// The array's name is only a handle on the host side; its device address has to be asked for,
// once per device, with that device current.
int static_workspace(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return MEBPTT_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_mutex);
  if (!g_device_ptr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_workspace) != cudaSuccess || !p) {
      cudaGetLastError();
      return MEBPTT_ERR_CUDA;
    }
    g_device_ptr[dev] = p;
  }
  *out = g_device_ptr[dev];
  return MEBPTT_OK;
}

}  // namespace

extern "C" int mebptt_lstm_train_step_static(const mebptt_lstm_desc* desc, const mebptt_plan_t* plan,
                                             const void* W, const void* b, const void* W_out, const void* b_out,
                                             const void* x, const void* targets, const void* h0, const void* c0,
                                             void* stream, float* loss, float* dW, float* db, float* dW_out,
                                             float* db_out, float* dx, int64_t* counters) {
  // per-launch timing records CUDA events, created on demand: not here
  if (desc && (desc->flags & MEBPTT_FLAG_TIME_RUNS)) return MEBPTT_ERR_ARG;
  const size_t need = mebptt_lstm_workspace_bytes(desc, plan);
  if (need == 0) return MEBPTT_ERR_ARG;                                   // bad descriptor or plan
  if (need > (size_t)MEBPTT_STATIC_WORKSPACE_BYTES) return MEBPTT_ERR_WORKSPACE;  // does not fit the fixed array
  void* ws = nullptr;
  const int rc = static_workspace(&ws);
  if (rc != MEBPTT_OK) return rc;
  // The step itself clears everything in the workspace that has to start at zero (carried
  // gradients, step counters, status word), so what the previous call left behind is harmless.
  // Single-stream execution: the side stream of the ordinary entry point would have to be
  // created on first use, and creating driver objects is a kind of allocation too.
  return mebptt::train_step_impl(desc, plan, W, b, W_out, b_out, x, targets, h0, c0, ws,
                                 (size_t)MEBPTT_STATIC_WORKSPACE_BYTES, stream, loss, dW, db, dW_out, db_out, dx,
                                 counters, false);
}
