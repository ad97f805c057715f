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
  enum Kind : int { STORE_F32 = 0, ACCUM_F32 = 1, STORE_BF16 = 2 };
  int kind;
  void* ptr;          // [M][ld]
  int64_t ld;         // elements
  const float* bias;  // optional, per column, float32 outputs only
};

// C (+)= A B^T over bfloat16 operands.  a_mn / b_mn: the operand is stored [k][m] instead of
// [m][k]; lda / ldb are row strides in elements (multiples of 8).  `status` (device, nullable)
// receives MEBPTT_ERR_TIMEOUT if a bounded wait expires.
int gemm_bf16(const void* A, int64_t lda, bool a_mn, const void* B, int64_t ldb, bool b_mn, const GemmOut& out,
              int M, int N, int K, int* status, cudaStream_t s);

}  // namespace tc
}  // namespace mebptt
