// Tensor-core (tcgen05 / TMEM / TMA) kernels: host-callable launchers.
#pragma once

#include <cuda_runtime.h>

#include <cstddef>
#include <cstdint>

#include "mebptt.h"

namespace mebptt {
namespace tc {

// Where a GEMM tile goes.
struct GemmOut {
  enum Kind : int { STORE_F32 = 0, ACCUM_F32 = 1, STORE_BF16 = 2, LOSS_DY = 3 };
  int kind;
  void* ptr;          // [M][ld]
  int64_t ld;         // elements
  const float* bias;  // optional, per column, float32 outputs only
  int perm_h;         // > 0: tile row 4 u + q is written to row q * perm_h + u (undoes the gate permutation)
  // LOSS_DY: the product (plus bias) is the readout y and is not stored.  With d = y - target[m][n],
  // ptr receives dy = 2 d scale in bfloat16 and loss_part[(m / 32) * parts + n / 32] the sum of
  // d * d * scale over that 32 x 32 block, in a fixed order (rows of M in groups of 32).
  const float* target = nullptr;   // [M][ld]
  float* dy32 = nullptr;           // optional: dy in float32 as well, [M][ld] (ptr may then be NULL)
  float* loss_part = nullptr;
  int parts = 0;                   // ceil(N / 32)
  float scale = 0.f;
};

// Caller buffers of one training step (device pointers).
struct StepPtrs {
  const char *W, *W_out, *x, *h0;
  const float *b, *b_out, *targets, *c0;
  char* ws;
  float *loss, *dW, *db, *dW_out, *db_out, *dx;
  int64_t* counters;
  // optional: the targets still lie in host memory at `targets_host`; the step copies them to
  // `targets` on a copy stream while the forward pass runs and waits for them before the first
  // backward run
  const void* targets_host = nullptr;
  size_t targets_bytes = 0;
  // optional, likewise: x still lies in host memory; it is copied to `x` in pieces along the time
  // axis on the copy stream, and each forward run waits only for the pieces it reads
  const void* x_host = nullptr;
  size_t x_bytes = 0;
  // bracket every launch of the two persistent kernels with CUDA events (collected by run_times)
  bool time_runs = false;
  // keep the host copy of the tape in pageable memory (the allocation-free entry point: page-locking
  // memory is an allocation too); its upload may then hold up the calling thread
  bool pageable_tape = false;
};

// Scratch for contractions that are split along K: a product with few output tiles and a long
// contraction index would otherwise stream all of K through a handful of SMs.  Each part writes
// its float32 tile here and a second kernel adds the parts in index order.
struct SplitWs {
  float* partial;        // device, partial_floats floats
  size_t partial_floats;
};

// Where a contraction that was split along K left its parts, for a consumer that adds them itself
// (in index order, starting from zero: the sum the library's own second pass would have stored).
// splits == 0: the product was not split and lies where GemmOut says.
struct SplitParts {
  const float* partial = nullptr;   // [tile][part][128][bn], tile = (m / 128) * tiles_x + n / bn
  int splits = 0, tiles_x = 0, bn = 0;
};
#ifdef __CUDACC__
__device__ __forceinline__ float split_parts_sum(const SplitParts& sp, int m, int n) {
  const int tile = (m >> 7) * sp.tiles_x + n / sp.bn;
  const float* p = sp.partial + (((size_t)tile * sp.splits) * 128 + (size_t)(m & 127)) * sp.bn + (n % sp.bn);
  float acc = 0.f;
  for (int z = 0; z < sp.splits; ++z) acc += p[(size_t)z * 128 * sp.bn];
  return acc;
}
#endif

// Parts gemm_bf16 splits the contraction index into, given scratch for partial_floats floats and
// an output it can split for (a plain float32 store, no bias, rows that take float4); 1 = no
// split, otherwise a second launch adds the parts.
int gemm_split_count(bool a_mn, bool b_mn, int M, int N, int K, size_t partial_floats);

// Parts for a contraction whose adding-up is left to its consumer (gemm_bf16's `defer`): no pass
// of its own has to pay off, so two parts are worth having; always over 128-wide tiles, about a
// wave of CTAs, each part at least 8 blocks of 64 long.
int gemm_split_count_deferred(int M, int N, int K);

// C (+)= A B^T over bfloat16 operands.  a_mn / b_mn: the operand is stored [k][m] instead of
// [m][k]; lda / ldb are row strides in elements (multiples of 8).  `status` (device, nullable)
// receives MEBPTT_ERR_TIMEOUT if a bounded wait expires.  early: the kernel may become resident
// before the previous kernel of the stream has finished (it still waits for it before touching
// memory).
// force_splits > 0: split the contraction index into exactly that many parts (the caller took the
// count from gemm_split_count for a product of another height, so that both sum in the same order).
// defer (optional): if the product is split, the pass that adds the parts is left to the caller's
// next kernel and *defer says where they are (C is then not touched, not even when accumulating:
// the consumer adds the parts to it); if it is not, *defer says so (splits = 0).  With defer and
// force_splits > 1 the tiles are 128 wide whatever the shape.
int gemm_bf16(const void* A, int64_t lda, bool a_mn, const void* B, int64_t ldb, bool b_mn, const GemmOut& out,
              int M, int N, int K, int* status, cudaStream_t s, bool early = true, const SplitWs* split = nullptr,
              int force_splits = 0, SplitParts* defer = nullptr);

}  // namespace tc

struct Layout;
struct Plan;
namespace tc {
// Enqueues one training step on the tensor-core path; returns a status.  With dry = true
// nothing is enqueued and the number of kernel launches is returned instead.
// side_stream: run the weight-gradient GEMMs of a finished chunk on a stream owned by the library,
// concurrently with the backward pass of the next chunk (joined back before the call's last kernel).
int64_t run_step(const Layout& y, const Plan* p, const StepPtrs& io, bool want_dx, cudaStream_t s, bool dry,
                 bool side_stream);


// Testing aid: which bounded waits are made to run out on purpose (0: none).  Bit 0: the step
// counter of the forward run kernel is told to expect one CTA too many; bit 1: likewise for the
// backward run kernels; bit 2: the first stage of a GEMM expects 16 bytes more than its copies
// bring.  The waits then give up after `fault_poll_limit` polls instead of the usual limit, the
// kernels leave through their ordinary exit path, and the status word receives MEBPTT_ERR_TIMEOUT.
int wait_fault_mask();
void set_wait_fault_mask(int mask);
constexpr uint32_t fault_poll_limit = 1u << 14;

// The prepared sets (work items, device tape, kernel variants, tensor maps) that run_step keeps per
// (problem, plan, workspace, device).  forget_plan drops those of a plan that is being freed;
// prepare_host makes (or finds) the host part only and returns its status; prepare_stats fills
// out[0..3] with sets built, sets reused, sets with a page-locked tape, sets held.
void forget_plan(uint64_t plan_id);
int prepare_host(const Layout& y, const Plan* p, bool want_dx);
void prepare_stats(int64_t* out);

// Waits for the event pairs recorded on the current device by steps run with time_runs, adds up
// elapsed milliseconds, launches and operations per class (0: forward runs, 1: backward runs)
// and forgets them.
int run_times(double* ms, int64_t* launches, int64_t* ops);
}  // namespace tc
}  // namespace mebptt
