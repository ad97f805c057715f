// Batched-over-time contractions on the tensor cores: C[M][N] (+)= sum_k A(m,k) B(n,k) with
// bfloat16 operands and float32 accumulation in TMEM.
//
// These are the parts of the training step that do not sit on the recurrence and can therefore
// be run for many time steps at once:
//   input projection   Zx[(s,b)][g]  = sum_i x[(s,b)][i] W_ih[g][i] + bias[g]         (A, B K-major)
//   readout            y[(s,b)][o]   = sum_j h[(s,b)][j] W_out[o][j]                 (A, B K-major)
//   readout backward   dha[(s,b)][j] = sum_o dy[(s,b)][o] W_out^T[j][o]              (A, B K-major)
//   weight gradients   dW[g][c]     += sum_(s,b) dz[(s,b)][g] in[(s,b)][c]           (A, B MN-major)
// "K-major" means the operand is stored with the contraction index contiguous; "MN-major" that it
// is stored [k][m] (rows are contraction indices), which is how dz and the layer inputs lie in
// memory for the weight gradient, so no transposed copies are made.
//
// One CTA computes one 128 x 128 tile (128 x 32 where C is short and wide: see gemm_bf16).  A single thread feeds a 3- or 6-stage ring of 128-byte
// swizzled shared-memory tiles by TMA (64 contraction indices per stage); a single thread issues
// tcgen05.mma (M = 128, N = 128, K = 16, four per stage) into a 128-column TMEM accumulator and
// releases ring slots with tcgen05.commit; then all four warps read the accumulator with
// tcgen05.ld (warp w owns TMEM lanes 32w .. 32w+31 = tile rows) and write the tile.
// Out-of-range parts of a tile are zero-filled by TMA on the way in and masked on the way out.
// The sum over k runs in one fixed order, so results do not depend on how callers batch steps.
#include <cstdlib>

#include "launch.hpp"
#include "sm100.cuh"
#include "tc.hpp"
#include "tmap.hpp"

namespace mebptt {
namespace tc {

namespace {

using namespace sm100;

constexpr int BM = 128, BK = 64, MAX_STAGES = 6;
constexpr int BN_WIDE = 128, BN_NARROW = 32;   // tile widths; narrow tiles spread a short-and-wide C over more SMs
constexpr int A_BYTES = BM * BK * 2;
constexpr int gemm_smem(int stages, int bn) { return stages * (A_BYTES + bn * BK * 2) + 1024; }  // + slack to align the ring to 1024 B

template <bool A_MN, bool B_MN, int BN = BN_WIDE>
__global__ void __launch_bounds__(128) gemm_bf16_kernel(const __grid_constant__ CUtensorMap tma,
                                                        const __grid_constant__ CUtensorMap tmb, GemmOut out,
                                                        int M, int N, int K, int STAGES, int* status,
                                                        float* partial, int fault) {
  constexpr int B_BYTES = BN * BK * 2, STAGE_BYTES = A_BYTES + B_BYTES;
  static_assert(BN == BN_WIDE || (!A_MN && !B_MN), "narrow tiles exist for K-major operands only");
  extern __shared__ uint8_t smem_raw[];
  __shared__ uint64_t full[MAX_STAGES], empty[MAX_STAGES], done;
  __shared__ uint32_t tmem_slot;
  __shared__ int failed;

  uint8_t* ring = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
  // this CTA's part of the contraction index: blocks [kb_lo, kb_lo + nk) of 64
  const int splits = gridDim.z;
  const int nk_all = (K + BK - 1) / BK;
  const int kb_lo = (int)((int64_t)nk_all * blockIdx.z / splits);
  const int nk = (int)((int64_t)nk_all * (blockIdx.z + 1) / splits) - kb_lo;
  const int tile = blockIdx.y * gridDim.x + blockIdx.x;

  if (threadIdx.x == 0) {
    for (int s = 0; s < MAX_STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    mbar_init(&done, 1);
    failed = 0;
    mbar_fence_init();
    tma_prefetch_desc(&tma);
    tma_prefetch_desc(&tmb);
  }
  if (warp == 1) tmem_alloc(&tmem_slot, BN);
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = tmem_slot;
  grid_dep_wait();     // operands (and, when accumulating, C) come from the kernels before this one
  grid_dep_launch();

  if (warp == 0 && lane == 0) {
    // ---- producer -----------------------------------------------------------------------
    int armed = 0;  // stages whose full barrier still awaits bytes (for the failure path)
    for (int kb = 0; kb < nk; ++kb) {
      const int s = kb % STAGES;
      if (kb >= STAGES && !mbar_wait(&empty[s], ((kb / STAGES) - 1) & 1)) { failed = 1; break; }
      uint8_t* sA = ring + s * STAGE_BYTES;
      uint8_t* sB = sA + A_BYTES;
      // (fault: a testing aid -- the first stage is told to expect 16 bytes that never come, so the
      // issuer's bounded wait runs out and the kernel leaves through its failure path)
      mbar_arrive_expect_tx(&full[s], STAGE_BYTES + ((fault && kb == 0) ? 16u : 0u));
      ++armed;
      if (A_MN) {
        tma_load_2d(sA, &tma, m0, (kb_lo + kb) * BK, &full[s]);
        tma_load_2d(sA + 8192, &tma, m0 + 64, (kb_lo + kb) * BK, &full[s]);
      } else {
        tma_load_2d(sA, &tma, (kb_lo + kb) * BK, m0, &full[s]);
      }
      if (B_MN) {
        tma_load_2d(sB, &tmb, n0, (kb_lo + kb) * BK, &full[s]);
        tma_load_2d(sB + 8192, &tmb, n0 + 64, (kb_lo + kb) * BK, &full[s]);
      } else {
        tma_load_2d(sB, &tmb, (kb_lo + kb) * BK, n0, &full[s]);
      }
    }
    (void)armed;
  } else if (warp == 1) {
    // ---- MMA issuer: the whole warp walks the loop (descriptors stay in uniform registers), one
    // elected lane issues --------------------------------------------------------------------------
    constexpr uint32_t idesc = make_idesc(1, BM, BN, A_MN, B_MN);
    // K-major: 16 contraction indices = 32 B along the row; MN-major: 16 rows of 128 B
    constexpr uint32_t A_STEP = A_MN ? (2048 >> 4) : (32 >> 4), B_STEP = B_MN ? (2048 >> 4) : (32 >> 4);
    const uint32_t ring0 = smem_u32(ring);
    const uint64_t a_desc0 = A_MN ? make_desc_sw128(ring0, 8192, 1024) : make_desc_sw128(ring0, 16, 1024);
    const uint64_t b_desc0 = B_MN ? make_desc_sw128(ring0 + A_BYTES, 8192, 1024) : make_desc_sw128(ring0 + A_BYTES, 16, 1024);
    bool ok = true;
    for (int kb = 0; kb < nk && ok; ++kb) {
      const int s = kb % STAGES;
      if (!mbar_wait(&full[s], (kb / STAGES) & 1)) { failed = 1; ok = false; break; }
      tc_fence_after_sync();
      if (elect_one()) {
        const uint64_t da = a_desc0 + (uint64_t)(s * (STAGE_BYTES >> 4)), db = b_desc0 + (uint64_t)(s * (STAGE_BYTES >> 4));
#pragma unroll
        for (int k4 = 0; k4 < BK / 16; ++k4)
          mma_f16(tmem, da + (uint64_t)(k4 * A_STEP), db + (uint64_t)(k4 * B_STEP), idesc, (kb > 0 || k4 > 0) ? 1u : 0u);
        mma_commit(&empty[s]);  // the slot may be refilled once these MMAs have read it
      }
      __syncwarp();
    }
    if (elect_one()) mma_commit(&done);
    __syncwarp();
  }

  // ---- epilogue: all four warps ---------------------------------------------------------
  __syncwarp();
  bool ok = mbar_wait(&done, 0);
  tc_fence_after_sync();
  bool finish = ok && !failed;
  if (finish && splits > 1) {
    // a part of a contraction split along K: the raw float32 tile goes to the scratch, and a
    // second kernel adds the parts in index order
    float* mine = partial + (((size_t)tile * splits + blockIdx.z) * BM + (size_t)(warp * 32 + lane)) * BN;
#pragma unroll 1
    for (int c = 0; c < BN / 32; ++c) {
      uint32_t r[32];
      tmem_ld_32x32(tmem + ((uint32_t)(warp * 32) << 16) + (uint32_t)(c * 32), r);
      tmem_ld_wait();
#pragma unroll
      for (int j = 0; j < 8; ++j)
        *(reinterpret_cast<float4*>(mine + c * 32) + j) =
            make_float4(__uint_as_float(r[4 * j]), __uint_as_float(r[4 * j + 1]), __uint_as_float(r[4 * j + 2]),
                        __uint_as_float(r[4 * j + 3]));
    }
    finish = false;
  }
  auto load_acc = [&](int c, uint32_t (&r)[32]) {
    tmem_ld_32x32(tmem + ((uint32_t)(warp * 32) << 16) + (uint32_t)(c * 32), r);
    tmem_ld_wait();
  };
  if (finish) {
    // Float32 tiles whose rows can be written as aligned float4: each warp parks its 32 x 128
    // block of the accumulator in the (now idle) operand ring, then writes -- or adds to -- one
    // whole 512-byte row of C per instruction.  Everything else takes the per-thread path below.
    const bool wide = BN == BN_WIDE && out.kind != GemmOut::STORE_BF16 && out.kind != GemmOut::LOSS_DY && (out.ld % 4 == 0) &&
                      ((reinterpret_cast<uintptr_t>(out.ptr) & 15) == 0) && (n0 % 4 == 0) &&
                      ((reinterpret_cast<uintptr_t>(out.bias) & 15) == 0);
    if (wide) {
      constexpr int PITCH = BN + 4;   // floats; keeps both the parking and the row reads conflict-free
      float* park = reinterpret_cast<float*>(ring) + (size_t)warp * 32 * PITCH;
#pragma unroll 1
      for (int c = 0; c < BN / 32; ++c) {
        uint32_t r[32];
        load_acc(c, r);
        float4* dst = reinterpret_cast<float4*>(park + (size_t)lane * PITCH + c * 32);
#pragma unroll
        for (int j = 0; j < 8; ++j)
          dst[j] = make_float4(__uint_as_float(r[4 * j]), __uint_as_float(r[4 * j + 1]), __uint_as_float(r[4 * j + 2]),
                               __uint_as_float(r[4 * j + 3]));
      }
      __syncwarp();
      const int col = n0 + lane * 4;
      const bool col_ok = col + 3 < N;       // N % 4 == 0 is implied by ld % 4 == 0 only for ld == N: check
      float4 bv = make_float4(0.f, 0.f, 0.f, 0.f);
      if (out.bias && col_ok) bv = *reinterpret_cast<const float4*>(out.bias + col);
      float* base = reinterpret_cast<float*>(out.ptr);
#pragma unroll 1
      for (int r0 = 0; r0 < 32; r0 += 8) {
        float4 old[8];
        size_t off[8];
        bool live[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const int row = m0 + warp * 32 + r0 + j;
          const int row_o = out.perm_h ? ((row & 3) * out.perm_h + (row >> 2)) : row;
          live[j] = row < M && col_ok;
          off[j] = (size_t)row_o * out.ld + col;
          old[j] = make_float4(0.f, 0.f, 0.f, 0.f);
          if (live[j] && out.kind == GemmOut::ACCUM_F32) old[j] = *reinterpret_cast<const float4*>(base + off[j]);
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          if (!live[j]) continue;
          const float4 v = *reinterpret_cast<const float4*>(park + (size_t)(r0 + j) * PITCH + lane * 4);
          *reinterpret_cast<float4*>(base + off[j]) =
              make_float4(v.x + bv.x + old[j].x, v.y + bv.y + old[j].y, v.z + bv.z + old[j].z, v.w + bv.w + old[j].w);
        }
      }
      // columns of a ragged right edge (N not a multiple of 4 inside this tile)
      if (!col_ok && col < N) {
        for (int r0 = 0; r0 < 32; ++r0) {
          const int row = m0 + warp * 32 + r0;
          if (row >= M) break;
          const int row_o = out.perm_h ? ((row & 3) * out.perm_h + (row >> 2)) : row;
          for (int j = 0; j < 4 && col + j < N; ++j) {
            float v = park[(size_t)r0 * PITCH + lane * 4 + j];
            if (out.bias) v += out.bias[col + j];
            float* q = base + (size_t)row_o * out.ld + col + j;
            if (out.kind == GemmOut::ACCUM_F32) v += *q;
            *q = v;
          }
        }
      }
    } else {
    const int row = m0 + warp * 32 + lane;
    const int row_o = out.perm_h ? ((row & 3) * out.perm_h + (row >> 2)) : row;
#pragma unroll 1
    for (int c = 0; c < BN / 32; ++c) {
      uint32_t r[32];
      load_acc(c, r);
      const int col0 = n0 + c * 32;
      if (out.kind == GemmOut::LOSS_DY) {
        // squared-error loss fused into the readout: this lane's row against its targets, columns in
        // ascending order, then the 32 rows of the warp in a fixed butterfly order
        float sq = 0.f;
        if (row < M) {
          const float* tp = out.target + (size_t)row * out.ld + col0;
          __nv_bfloat16* dp = reinterpret_cast<__nv_bfloat16*>(out.ptr) + (size_t)row * out.ld + col0;
          const float two = 2.f * out.scale;
          float* d32 = out.dy32 ? out.dy32 + (size_t)row * out.ld + col0 : nullptr;
          if (col0 + 32 <= N && ((reinterpret_cast<uintptr_t>(tp) & 15) == 0) && ((reinterpret_cast<uintptr_t>(dp) & 15) == 0) &&
              ((reinterpret_cast<uintptr_t>(out.bias) & 15) == 0) && ((reinterpret_cast<uintptr_t>(d32) & 15) == 0)) {
            float4 t4[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) t4[j] = *reinterpret_cast<const float4*>(tp + 4 * j);
            uint32_t packed[16];
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              float4 bv = make_float4(0.f, 0.f, 0.f, 0.f);
              if (out.bias) bv = *reinterpret_cast<const float4*>(out.bias + col0 + 4 * j);
              const float d0 = (__uint_as_float(r[4 * j]) + bv.x) - t4[j].x;
              const float d1 = (__uint_as_float(r[4 * j + 1]) + bv.y) - t4[j].y;
              const float d2 = (__uint_as_float(r[4 * j + 2]) + bv.z) - t4[j].z;
              const float d3 = (__uint_as_float(r[4 * j + 3]) + bv.w) - t4[j].w;
              sq = fmaf(d0, d0, sq); sq = fmaf(d1, d1, sq); sq = fmaf(d2, d2, sq); sq = fmaf(d3, d3, sq);
              packed[2 * j] = pack_bf16x2(d0 * two, d1 * two);
              packed[2 * j + 1] = pack_bf16x2(d2 * two, d3 * two);
              if (d32) *reinterpret_cast<float4*>(d32 + 4 * j) = make_float4(d0 * two, d1 * two, d2 * two, d3 * two);
            }
            if (out.ptr) {
#pragma unroll
              for (int j = 0; j < 4; ++j)
                *reinterpret_cast<uint4*>(dp + 8 * j) = make_uint4(packed[4 * j], packed[4 * j + 1], packed[4 * j + 2], packed[4 * j + 3]);
            }
          } else {
#pragma unroll
            for (int j = 0; j < 32; ++j)
              if (col0 + j < N) {
                const float d = (__uint_as_float(r[j]) + (out.bias ? out.bias[col0 + j] : 0.f)) - tp[j];
                sq = fmaf(d, d, sq);
                if (out.ptr) dp[j] = __float2bfloat16_rn(d * two);
                if (d32) d32[j] = d * two;
              }
          }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
        if (lane == 0 && m0 + warp * 32 < M && col0 < N)
          out.loss_part[(size_t)((m0 + warp * 32) / 32) * out.parts + col0 / 32] = sq * out.scale;
      } else if (row < M) {
        if (out.kind == GemmOut::STORE_BF16) {
          __nv_bfloat16* p = reinterpret_cast<__nv_bfloat16*>(out.ptr) + (size_t)row_o * out.ld + col0;
#pragma unroll
          for (int j = 0; j < 32; ++j)
            if (col0 + j < N) p[j] = __float2bfloat16_rn(__uint_as_float(r[j]));
        } else {
          float* p = reinterpret_cast<float*>(out.ptr) + (size_t)row_o * out.ld + col0;
          const bool vec = (col0 + 32 <= N) && ((reinterpret_cast<uintptr_t>(p) & 15) == 0) &&
                           ((reinterpret_cast<uintptr_t>(out.bias) & 15) == 0);
          if (vec) {
            // all eight loads of the old values first, so that their latencies overlap
            float4 o[8];
            if (out.kind == GemmOut::ACCUM_F32) {
#pragma unroll
              for (int j = 0; j < 8; ++j) o[j] = *reinterpret_cast<const float4*>(p + 4 * j);
            } else {
#pragma unroll
              for (int j = 0; j < 8; ++j) o[j] = make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              float4 v = make_float4(__uint_as_float(r[4 * j]), __uint_as_float(r[4 * j + 1]),
                                     __uint_as_float(r[4 * j + 2]), __uint_as_float(r[4 * j + 3]));
              if (out.bias) {
                const float4 bv = *reinterpret_cast<const float4*>(out.bias + col0 + 4 * j);
                v.x += bv.x; v.y += bv.y; v.z += bv.z; v.w += bv.w;
              }
              v.x += o[j].x; v.y += o[j].y; v.z += o[j].z; v.w += o[j].w;
              *reinterpret_cast<float4*>(p + 4 * j) = v;
            }
          } else {
#pragma unroll
            for (int j = 0; j < 32; ++j)
              if (col0 + j < N) {
                float v = __uint_as_float(r[j]);
                if (out.bias) v += out.bias[col0 + j];
                if (out.kind == GemmOut::ACCUM_F32) v += p[j];
                p[j] = v;
              }
          }
        }
      }
    }
    }
  } else if ((!ok || failed) && status && threadIdx.x == 0) {
    *status = MEBPTT_ERR_TIMEOUT;
  }
  // On the failure path the producer may still have loads in flight: give them a bounded
  // chance to land before the shared memory goes away.
  if (failed && warp == 0 && lane == 0)
    for (int s = 0; s < STAGES; ++s) (void)mbar_wait(&full[s], 0);
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem, BN);
}

// C[m][n] = sum over the parts, in index order, of a contraction that was split along K.
// partial: [tile][part][128][bn] with tile = (m / 128) * tiles_x + n / bn.  One thread per four
// adjacent columns.
__global__ void splitk_reduce(const float* partial, int splits, int M, int N, int tiles_x, int bn, float* out, int64_t ld) {
  grid_dep_wait();
  grid_dep_launch();
  const int n4 = (N + 3) / 4;
  const size_t total = (size_t)M * n4;
  for (size_t e = blockIdx.x * (size_t)blockDim.x + threadIdx.x; e < total; e += (size_t)gridDim.x * blockDim.x) {
    const int m = (int)(e / n4), n = (int)(e % n4) * 4;
    const int tile = (m / BM) * tiles_x + n / bn;
    const float* p = partial + (((size_t)tile * splits) * BM + (size_t)(m % BM)) * bn + (n % bn);
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int z = 0; z < splits; ++z) {
      const float4 v = *reinterpret_cast<const float4*>(p + (size_t)z * BM * bn);
      acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
    }
    float* q = out + (size_t)m * ld + n;
    if (n + 3 < N) *reinterpret_cast<float4*>(q) = acc;
    else {
      const float a[4] = {acc.x, acc.y, acc.z, acc.w};
      for (int j = 0; j < 4 && n + j < N; ++j) q[j] = a[j];
    }
  }
}

}  // namespace

// Few tiles and a long contraction index: split K so that about a wave of CTAs streams the
// operands, each part at least 8 blocks of 64 long; a second kernel adds the parts.  Only where at
// least four parts come out of it: below that the extra pass costs more than it saves.
int gemm_split_count(bool a_mn, bool b_mn, int M, int N, int K, size_t partial_floats) {
  if (env::no_splitk()) return 1;
  const int wide_tiles = ((N + BN_WIDE - 1) / BN_WIDE) * ((M + BM - 1) / BM);
  const bool narrow = !a_mn && !b_mn && wide_tiles <= 37 && N >= 2 * BN_NARROW;
  const int BN = narrow ? BN_NARROW : BN_WIDE;
  const int tiles = ((N + BN - 1) / BN) * ((M + BM - 1) / BM);
  const int nk = (K + BK - 1) / BK;
  int want = 148 / tiles;
  if (want > nk / 8) want = nk / 8;
  if (want > 16) want = 16;
  while (want > 1 && (size_t)tiles * want * BM * BN > partial_floats) --want;
  return want >= 4 ? want : 1;
}

int gemm_split_count_deferred(int M, int N, int K) {
  if (env::no_splitk()) return 1;
  const int tiles = ((N + BN_WIDE - 1) / BN_WIDE) * ((M + BM - 1) / BM);
  const int nk = (K + BK - 1) / BK;
  int want = 148 / tiles;
  if (want > nk / 8) want = nk / 8;
  if (want > 16) want = 16;
  return want >= 2 ? want : 1;
}

int gemm_bf16(const void* A, int64_t lda, bool a_mn, const void* B, int64_t ldb, bool b_mn, const GemmOut& out,
              int M, int N, int K, int* status, cudaStream_t s, bool early, const SplitWs* split, int force_splits,
              SplitParts* defer) {
  if (M <= 0 || N <= 0 || K <= 0) return MEBPTT_ERR_ARG;
  // A short-and-wide product over K-major operands (a few steps' worth of rows against a whole
  // weight matrix) gives few 128-wide tiles, each streaming all of K through one SM: 32-wide tiles
  // put four times as many SMs to work on the same bytes.
  const int wide_tiles = ((N + BN_WIDE - 1) / BN_WIDE) * ((M + BM - 1) / BM);
  const bool narrow = !a_mn && !b_mn && wide_tiles <= 37 && N >= 2 * BN_NARROW && !(defer && force_splits > 1);
  const int BN = narrow ? BN_NARROW : BN_WIDE;
  CUtensorMap ta, tb;
  // K-major: tensor is [M][K], box 64 (k) x tile rows.  MN-major: tensor is [K][M], box 64 (m) x 64 rows.
  bool ok = a_mn ? make_tmap_2d(&ta, A, 2, (uint64_t)M, (uint64_t)K, (uint64_t)lda * 2, 64, 64)
                 : make_tmap_2d(&ta, A, 2, (uint64_t)K, (uint64_t)M, (uint64_t)lda * 2, 64, 128);
  ok = ok && (b_mn ? make_tmap_2d(&tb, B, 2, (uint64_t)N, (uint64_t)K, (uint64_t)ldb * 2, 64, 64)
                   : make_tmap_2d(&tb, B, 2, (uint64_t)K, (uint64_t)N, (uint64_t)ldb * 2, 64, (uint32_t)BN));
  if (!ok) return MEBPTT_ERR_UNSUPPORTED;
  dim3 grid((N + BN - 1) / BN, (M + BM - 1) / BM);
  int splits = 1;
  if (split && split->partial && (out.kind == GemmOut::STORE_F32 || (defer && out.kind == GemmOut::ACCUM_F32)) &&
      !out.bias && !out.perm_h && out.ld % 4 == 0 && (reinterpret_cast<uintptr_t>(out.ptr) & 15) == 0)
    splits = force_splits > 0 ? force_splits : gemm_split_count(a_mn, b_mn, M, N, K, split->partial_floats);
  else if (force_splits > 1)
    return MEBPTT_ERR_ARG;
  if (splits > 1 && (size_t)grid.x * grid.y * splits * BM * BN > split->partial_floats) return MEBPTT_ERR_WORKSPACE;
  grid.z = splits;
  static const bool attrs = [] {
    const int most = gemm_smem(MAX_STAGES, BN_WIDE);
    cudaFuncSetAttribute(gemm_bf16_kernel<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, most);
    cudaFuncSetAttribute(gemm_bf16_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, most);
    cudaFuncSetAttribute(gemm_bf16_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, most);
    cudaFuncSetAttribute(gemm_bf16_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, most);
    cudaFuncSetAttribute(gemm_bf16_kernel<false, false, BN_NARROW>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                         gemm_smem(MAX_STAGES, BN_NARROW));
    return true;
  }();
  (void)attrs;
  // Large grids: 3 stages, two CTAs per SM, so that one CTA's epilogue overlaps the other's main
  // loop.  Grids of at most one wave: 6 stages, more loads in flight per CTA to hide their latency.
  const int stages = (grid.x * grid.y * grid.z <= 148) ? MAX_STAGES : 3;
  const int GEMM_SMEM = gemm_smem(stages, BN);
  auto* fn = narrow ? gemm_bf16_kernel<false, false, BN_NARROW>
             : a_mn ? (b_mn ? gemm_bf16_kernel<true, true> : gemm_bf16_kernel<true, false>)
                    : (b_mn ? gemm_bf16_kernel<false, true> : gemm_bf16_kernel<false, false>);
  const cudaError_t e = launch_on(early, fn, grid, dim3(128), (size_t)GEMM_SMEM, s, ta, tb, out, M, N, K, stages, status,
                                  splits > 1 ? split->partial : nullptr, (wait_fault_mask() & 4) ? 1 : 0);
  if (e != cudaSuccess) {
    cudaGetLastError();
    return MEBPTT_ERR_CUDA;
  }
  if (defer) *defer = splits > 1 ? SplitParts{split->partial, splits, (int)grid.x, BN} : SplitParts{};
  if (splits > 1 && !defer) {
    const size_t quads = (size_t)M * ((N + 3) / 4);
    const int blocks = (int)((quads + 255) / 256 > 1184 ? 1184 : (quads + 255) / 256);
    const cudaError_t e2 = launch_on(early, splitk_reduce, dim3(blocks), dim3(256), 0, s, (const float*)split->partial,
                                     splits, M, N, (int)grid.x, BN, reinterpret_cast<float*>(out.ptr), out.ld);
    if (e2 != cudaSuccess) {
      cudaGetLastError();
      return MEBPTT_ERR_CUDA;
    }
  }
  return MEBPTT_OK;
}

}  // namespace tc
}  // namespace mebptt
