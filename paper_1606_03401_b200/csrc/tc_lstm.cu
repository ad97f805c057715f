// The LSTM recurrence on the tensor cores (bfloat16 operands, float32 accumulation and cell
// state), one layer.
//
// What sits on the recurrence, and therefore cannot be batched over time, is only the
// product with the recurrent weights: z_t = Zx_t + h_{t-1} W_hh^T going forward and
// dh_{t-1} = dz_t W_hh going backward.  Both run in persistent kernels that walk a run of
// consecutive tape operations with W_hh resident in shared memory:
//
//   fwd_run_kernel   CTA c owns hidden units 8c .. 8c+7, i.e. the 32 gate rows {i,f,g,o} x 8 of
//                    W_hh, permuted so that the four gates of a unit are adjacent columns.  Per
//                    step: TMA streams h_{t-1} ([B][H], 64 columns at a time) through a ring,
//                    one thread issues tcgen05.mma (M = 64 or 128 batch rows, N = 32, K = 16)
//                    into TMEM, then each thread owning a batch row reads its 32 accumulators,
//                    adds the batched input projection Zx_t (bias included), applies the gates
//                    and updates c_t, h_t for its 8 units -- c_t and h_t stay in registers from
//                    step to step -- and writes the state where the tape says (scratch, a slot
//                    of the arena, or a whole internal state).
//   bwd_run_kernel   same ownership.  Per step each thread forms dz for its 8 units x 4 gates
//                    from dh (read back from TMEM), dc (registers), the stored gates and cell
//                    states, writes dz (bfloat16) to the staging chunk, and the CTA then
//                    contracts the whole dz_t ([B][4H]) against its 8 rows of W_hh^T
//                    (M = batch, N = 8, K = 16) to get its slice of dh_{t-1}.
//
// Between steps every CTA needs all of h_t (or dz_t): a grid-wide counter in global memory is
// bumped by each CTA after its stores (release) and polled by the one thread that issues the
// next step's TMA loads (acquire), with a proxy fence on both sides because the loads go
// through the async proxy.  The kernels are launched cooperatively, so all CTAs are resident
// and the wait cannot deadlock; it is bounded all the same.
//
// Everything off the recurrence is batched over S consecutive time steps and done by the
// tensor-core GEMM: input projections before a forward run; readout, its gradient, and -- once
// the backward pass has completed a chunk of S steps aligned to absolute time -- the weight
// gradients.  Chunks are tied to time indices, not to run boundaries, and backward steps always
// come in the order t .. 1, so every sum runs in the same order under every plan.
#include <atomic>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <memory>
#include <mutex>
#include <vector>

#include "launch.hpp"
#include "layout.hpp"
#include "sm100.cuh"
#include "tc.hpp"
#include "tmap.hpp"

namespace mebptt {
namespace tc {

namespace {

using namespace sm100;

constexpr int NU = 8;            // hidden units per CTA
constexpr int NG = 4 * NU;       // gate columns per CTA
constexpr int NST = 8;           // ring stages of 64 contraction indices
constexpr int LOSS_PARTS = 64;   // partial sums per step of the loss

// Tape entry as the kernels see it.  Offsets are in units of 16 bytes from the workspace base.
struct DevOp {
  int32_t k;
  int32_t fmt;
  uint32_t h_src, c_src;   // FWD: state k-1.            BWD: h_{k-1}, c_{k-1}
  uint32_t h_dst, c_dst;   // FWD: where h_k, c_k go.    BWD: h_k, c_k of the stored internal state
  uint32_t gates;          // FWD: gate planes to write, 0 = none.   BWD: gate planes to read
  uint32_t in_copy;        // FWD: hidden block receiving the copy of state k-1, 0 = none
};
static_assert(sizeof(DevOp) == 32, "DevOp layout");

__device__ __forceinline__ float sigmoid_fast(float x) { return __fdividef(1.f, 1.f + __expf(-x)); }
__device__ __forceinline__ float tanh_fast(float x) {
  float y;
  asm("tanh.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ bool wait_or_fail(uint64_t* bar, uint32_t parity, volatile int* failed) {
  for (uint32_t i = 0; i < kSpinLimit; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if (i > 256) {
      if (*failed) return false;
      __nanosleep(64);
    }
  }
  *failed = 1;
  return false;
}
__device__ __forceinline__ bool wait_counter(const uint32_t* ctr, uint32_t target, volatile int* failed,
                                             uint32_t limit = kSpinLimit >> 1) {
  for (uint32_t i = 0; i < limit; ++i) {
    if (ld_acquire(ctr) >= target) return true;
    if (i > 4096 && *failed) return false;
  }
  *failed = 1;
  return false;
}
__device__ __forceinline__ float bf16_lo(uint32_t v) { return __uint_as_float(v << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t v) { return __uint_as_float(v & 0xFFFF0000u); }

// ------------------------------------------------------------------------------------------
// forward run
// ------------------------------------------------------------------------------------------
// A step of the recurrence is bound by latency, not by bytes or flops: h_{k-1} has to get from the
// SMs that produce it to every SM that holds a part of W_hh (stores, release of a step counter, a
// poll with acquire, the fetch), and one thread must then issue an MMA per 16 contraction indices.
// What the kernel does about it:
//
//   * The batch rows of an LSTM never mix, so the grid is cut into groups of CTAs that each own
//     FB = 32 batch rows: a CTA pulls only its group's rows of h_{k-1}, and groups synchronise
//     among themselves only (a step counter per group, in a cache line of its own).  CTA c of a
//     group owns hidden units 16 c .. 16 c + 15.
//   * The product is taken transposed: the CTA's 64 gate rows of W_hh (resident in shared memory,
//     rows permuted to 4 u + q) are the M side of the MMA and the 32 batch rows the N side, so that
//     a tile of full height serves a batch slice of 32.
//   * The TMA unit accepts one copy request at a time and takes ~100 ns for each, whatever its
//     size: sixteen tile copies are a microsecond and a half before the last tile even starts.
//     h_{k-1} is therefore fetched with two copies (one per half of the contraction index) over a
//     3-D tensor map that sees a row as blocks of 64 columns, which land as consecutive swizzled
//     tiles.
//   * The contraction is summed in two parts (two TMEM accumulators; the MMAs of the first are
//     issued while the second half of h_{k-1} is still arriving):  z = (Zx + part 0) + part 1, Zx
//     being the batched input projection, bias included.  The batched GEMMs of a leaf batch
//     accumulate in the same order, so both give the same bits.
//   * The accumulators [64 gate rows][32 batch rows] leave TMEM one gate row per thread and are
//     handed over through shared memory; each of the 128 epilogue threads then owns four hidden
//     units of one batch row -- four threads side by side cover 32 bytes of a row, so a warp's
//     store is 8 full sectors instead of 32 quarter sectors, and the stores are what the release
//     that follows waits for.  The thread applies the gates and updates c_t, h_t (which stay in
//     registers from step to step) and writes the state where the tape says (scratch, a slot of
//     the arena, or a whole internal state).
//
// Measured and dropped (config 3, microseconds per forward operation against 4.47 for this
// kernel): clusters of two CTAs that split the contraction index and exchange partial tiles
// through distributed shared memory, by ordinary remote stores with a release/acquire barrier
// (5.0) or by asynchronous stores that count on the receiver's barrier (exchange 0.66 of the
// 4.5 us step); h_k as its own signal -- a ring of exchange slots whose words hold an impossible
// bit pattern until h_k is written with strong stores, polled with strong 16-byte loads into
// registers and staged into the swizzled tiles by the epilogue warps, the step counter kept off
// the critical path for the reuse of slots only -- which removes the 1.5 us signalling round but
// loses as much to the staging and to waiting for the slowest producer (5.3).
//
// Warps 0-3: epilogue; warp 4: TMA producer; warp 5: MMA issuer.  All of h_{k-1} a CTA needs is
// resident in shared memory for the step (H <= 1024), so the producer never waits for a free slot.
constexpr int FU = 16;          // hidden units per CTA
constexpr int FG = 4 * FU;      // gate rows per CTA
constexpr int FB = 32;          // batch rows per group of CTAs: the N of the MMA
constexpr int PART_LD = FG + 4; // row stride of an accumulator handed over in shared memory, [batch row][gate row] (floats)
constexpr int SYNC_STRIDE = 32; // words between the step counters of two groups (one 128-byte line each)

struct FwdRunArgs {
  const DevOp* ops;      // this launch's operations (consecutive forward operations)
  int n;
  char* ws;              // workspace base
  const float* zx;       // [n][B][4H]: input projection + bias, gate columns permuted (4 u + q)
  uint32_t* sync;        // step counters of this launch, one per group (zero on entry)
  int* status;
  int64_t* counters;
  int B, H;
  int ncg;               // CTAs per group
  int bb;                // K tiles (64 contraction indices each) per barrier and, in slab mode, per copy
  int slab;              // 1: tm_h is a blocked 3-D map and one copy brings bb tiles; 0: one 2-D copy per tile
  uint32_t expect;       // signals a step is complete with: ncg (a testing aid may ask for one too many)
  uint32_t poll_limit;   // polls of the step counter before the wait gives up
  uint32_t plane16;      // distance between gate planes, in 16-byte units
  uint32_t hsz16;        // distance from h to c inside a hidden block, in 16-byte units
};

// 64-wide blocks of the contraction index in the first part of the split (all of them if there is
// one part only: below 640 columns the second accumulator and its hand-over cost more than starting
// the MMAs half a fetch earlier saves)
__host__ __device__ inline int fwd_first_part_blocks(int H) {
  const int KB = (H + 63) / 64;
  return KB >= 10 ? (KB + 1) / 2 : KB;
}

// State update of one thread: batch row b, hidden units j0 .. j0 + 3.  z[u] holds the four
// pre-activations (i, f, g, o) of unit j0 + u; writes h_k at once and the rest of the state after
// `signal` has told the other CTAs that h_k is there.
struct FwdCell {
  float c[4];
  uint2 hprev;
  float4 zx[4];
};
__device__ __forceinline__ void fwd_cell_init(FwdCell& st, const FwdRunArgs& a, bool owner, int b, int j0, size_t e0) {
#pragma unroll
  for (int u = 0; u < 4; ++u) { st.c[u] = 0.f; st.zx[u] = make_float4(0.f, 0.f, 0.f, 0.f); }
  st.hprev = make_uint2(0, 0);
  if (!owner) return;
  const DevOp op0 = a.ops[0];
  const float4 c0 = *(reinterpret_cast<const float4*>(a.ws + (size_t)op0.c_src * 16) + e0 / 4);
  st.c[0] = c0.x; st.c[1] = c0.y; st.c[2] = c0.z; st.c[3] = c0.w;
  st.hprev = *reinterpret_cast<const uint2*>(reinterpret_cast<const __nv_bfloat16*>(a.ws + (size_t)op0.h_src * 16) + e0);
  const float4* zp = reinterpret_cast<const float4*>(a.zx + (size_t)b * 4 * a.H + (size_t)4 * j0);
#pragma unroll
  for (int v = 0; v < 4; ++v) st.zx[v] = zp[v];
}
struct FwdCellOut {
  uint2 hnew, gi, gf, gg, go;
  float cin[4];
};
__device__ __forceinline__ void fwd_cell_gates(FwdCell& st, const float4 (&z)[4], FwdCellOut& o) {
  float hv[4], iv[4], fv[4], gv[4], ov[4];
#pragma unroll
  for (int u = 0; u < 4; ++u) {
    iv[u] = sigmoid_fast(z[u].x);
    fv[u] = sigmoid_fast(z[u].y);
    gv[u] = tanh_fast(z[u].z);
    ov[u] = sigmoid_fast(z[u].w);
    o.cin[u] = st.c[u];
    st.c[u] = fmaf(fv[u], st.c[u], iv[u] * gv[u]);
    hv[u] = ov[u] * tanh_fast(st.c[u]);
  }
  o.hnew = make_uint2(pack_bf16x2(hv[0], hv[1]), pack_bf16x2(hv[2], hv[3]));
  o.gi = make_uint2(pack_bf16x2(iv[0], iv[1]), pack_bf16x2(iv[2], iv[3]));
  o.gf = make_uint2(pack_bf16x2(fv[0], fv[1]), pack_bf16x2(fv[2], fv[3]));
  o.gg = make_uint2(pack_bf16x2(gv[0], gv[1]), pack_bf16x2(gv[2], gv[3]));
  o.go = make_uint2(pack_bf16x2(ov[0], ov[1]), pack_bf16x2(ov[2], ov[3]));
}
// The part of the state that is not on the critical path of the recurrence, and the input
// projection of the next step (which does not depend on the recurrence either).
__device__ __forceinline__ void fwd_cell_rest(FwdCell& st, const FwdRunArgs& a, const DevOp& op, const FwdCellOut& o,
                                              int i, int b, int j0, size_t e0) {
  char* ws = a.ws;
  *(reinterpret_cast<float4*>(ws + (size_t)op.c_dst * 16) + e0 / 4) = make_float4(st.c[0], st.c[1], st.c[2], st.c[3]);
  if (op.gates) {
    __nv_bfloat16* gp = reinterpret_cast<__nv_bfloat16*>(ws + (size_t)op.gates * 16) + e0;
    const size_t pl = (size_t)a.plane16 * 8;   // elements
    *reinterpret_cast<uint2*>(gp) = o.gi;
    *reinterpret_cast<uint2*>(gp + pl) = o.gf;
    *reinterpret_cast<uint2*>(gp + 2 * pl) = o.gg;
    *reinterpret_cast<uint2*>(gp + 3 * pl) = o.go;
  }
  if (op.in_copy) {
    char* blk = ws + (size_t)op.in_copy * 16;
    *reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(blk) + e0) = st.hprev;
    *(reinterpret_cast<float4*>(blk + (size_t)a.hsz16 * 16) + e0 / 4) = make_float4(o.cin[0], o.cin[1], o.cin[2], o.cin[3]);
  }
  st.hprev = o.hnew;
  if (i + 1 < a.n) {
    const float4* zp = reinterpret_cast<const float4*>(a.zx + ((size_t)(i + 1) * a.B + b) * 4 * a.H + (size_t)4 * j0);
#pragma unroll
    for (int v = 0; v < 4; ++v) st.zx[v] = zp[v];
  }
}
// z = (Zx + part 0) + part 1 for the 16 gate rows of this thread: p0 / p1 point at its 16 floats
// (gate rows 4 u + q of its four units) in the handed-over accumulators.
__device__ __forceinline__ void fwd_cell_sum(const FwdCell& st, const float* p0, const float* p1, float4 (&z)[4]) {
#pragma unroll
  for (int u = 0; u < 4; ++u) {
    const float4 x = *reinterpret_cast<const float4*>(p0 + 4 * u);
    z[u] = make_float4(st.zx[u].x + x.x, st.zx[u].y + x.y, st.zx[u].z + x.z, st.zx[u].w + x.w);
    if (p1) {
      const float4 y = *reinterpret_cast<const float4*>(p1 + 4 * u);
      z[u].x += y.x; z[u].y += y.y; z[u].z += y.z; z[u].w += y.w;
    }
  }
}

// One CTA per 16 hidden units and group; both halves of the contraction, into two accumulators.
__global__ void __launch_bounds__(192, 1) fwd_run_kernel(const __grid_constant__ CUtensorMap tm_h,
                                                         const __grid_constant__ CUtensorMap tm_w,
                                                         const FwdRunArgs a) {
  constexpr uint32_t W_TILE = FG * 128;   // [64 gate rows][64 contraction indices]
  constexpr uint32_t H_TILE = FB * 128;   // [32 batch rows][64 contraction indices]
  extern __shared__ uint8_t smem_raw[];
  __shared__ uint64_t wfull, full[4], acc;
  __shared__ uint32_t tmem_slot;
  __shared__ int failed;

  uint8_t* sm = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int KB = (a.H + 63) / 64;      // <= 16
  const int KB0 = fwd_first_part_blocks(a.H);
  uint8_t* sW = sm;                    // KB tiles: this CTA's rows of W_hh
  uint8_t* tiles = sm + KB * W_TILE;   // KB tiles: the group's rows of h_{k-1}
  const int NQ = KB0 < KB ? 2 : 1;     // parts of the contraction: one barrier, one copy (slab mode), one accumulator each
  float* part = reinterpret_cast<float*>(tiles + NQ * KB0 * H_TILE);   // [2][FB][PART_LD]

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int grp = blockIdx.x / a.ncg, cta = blockIdx.x % a.ncg;
  uint32_t* const sync = a.sync + grp * SYNC_STRIDE;

  if (tid == 0) {
    mbar_init(&wfull, 1);
    for (int s = 0; s < 4; ++s) mbar_init(&full[s], 1);
    mbar_init(&acc, 1);
    failed = 0;
    mbar_fence_init();
    tma_prefetch_desc(&tm_h);
    tma_prefetch_desc(&tm_w);
  }
  if (warp == 4) tmem_alloc(&tmem_slot, 64);
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = tmem_slot;
  const uint32_t row_bytes = (uint32_t)a.H * 2u;
  grid_dep_wait();   // everything above touched no global memory; everything below may

  if (warp == 4) {
    // ---- producer: lane 0 watches the group's step counter, then h_{k-1} is requested.  A copy
    // instruction takes the TMA unit ~80-120 ns to accept whatever its size, and the unit takes one
    // at a time: 16 tiles requested one by one are a microsecond.  In slab mode one copy (a 3-D box
    // over a map that sees the row as blocks of 64 columns) brings a whole part of the split. ------
    if (lane == 0) {
      mbar_arrive_expect_tx(&wfull, (uint32_t)KB * W_TILE);
      for (int kb = 0; kb < KB; ++kb) tma_load_2d(sW + kb * W_TILE, &tm_w, kb * 64, cta * FG, &wfull);
    }
    int armed = -1;   // last step whose loads were requested (for the failure path)
    for (int i = 0; i < a.n; ++i) {
      const DevOp op = a.ops[i];
      // rows of the group inside the block of h_{k-1}; rows past the batch are never used (they
      // only reach accumulator columns that no thread reads)
      const int32_t row = (int32_t)(((uint64_t)op.h_src * 16u) / row_bytes) + grp * FB;
      int go = 1;
      if (lane == 0) go = !failed && (i == 0 || wait_counter(sync, (uint32_t)i * a.expect, &failed, a.poll_limit)) && !failed;
      go = __shfl_sync(0xffffffffu, go, 0);
      if (!go) continue;
      // the acquire of lane 0 reaches the other lanes through the shuffle; the proxy fence then orders
      // a lane's TMA read after the h_k written by the other CTAs
      if (a.slab) {
        if (lane < NQ) {
          fence_proxy_async_global();
          mbar_arrive_expect_tx(&full[lane], (uint32_t)KB0 * H_TILE);   // a box counts in full, also where it is filled with zeros
          tma_load_3d(tiles + lane * KB0 * H_TILE, &tm_h, 0, row, lane * KB0, &full[lane]);
        }
      } else if (lane < KB) {
        fence_proxy_async_global();
        const int q = lane >= KB0 ? 1 : 0;
        if (lane == q * KB0) mbar_arrive_expect_tx(&full[q], (uint32_t)(q ? KB - KB0 : KB0) * H_TILE);
        tma_load_2d(tiles + lane * H_TILE, &tm_h, lane * 64, row, &full[q]);
      }
      armed = i;
      if (i == a.n - 1 && lane == 0) grid_dep_launch();   // last step under way: the next kernel may set itself up
      __syncwarp();
    }
    if (failed && lane == 0) {
      // loads that were requested may still be landing: give them a bounded chance
      (void)mbar_wait(&wfull, 0);
      if (armed >= 0)
        for (int q = 0; q < NQ; ++q) (void)mbar_wait(&full[q], (uint32_t)armed & 1);
    }
  } else if (warp == 5) {
    // ---- MMA issuer: the whole warp walks the loop (so that addresses and descriptors stay in
    // uniform registers), one elected lane issues ------------------------------------------------
    constexpr uint32_t idesc = make_idesc(1, FG, FB, false, false);
    bool ok = wait_or_fail(&wfull, 0, &failed);
    const uint64_t w_desc0 = make_desc_sw128(smem_u32(sW), 16, 1024);
    const uint64_t h_desc0 = make_desc_sw128(smem_u32(tiles), 16, 1024);
    for (int i = 0; i < a.n; ++i) {
      // descriptors advance by plain additions to their address field: 2 (32 bytes) per K = 16
      // inside a tile, one tile (8 KB of W, 4 KB of h) per 64 contraction indices
      uint64_t dw = w_desc0, dh = h_desc0;
      for (int q = 0; q < NQ && ok; ++q) {
        ok = wait_or_fail(&full[q], (uint32_t)i & 1, &failed);
        if (!ok) break;
        tc_fence_after_sync();
        const int nkb = q ? KB - KB0 : KB0;   // part q of the split, into accumulator q
        if (elect_one()) {
          for (int kb = 0; kb < nkb; ++kb)
            mma_f16_x4(tmem + (uint32_t)(q * FB), dw + (uint64_t)(kb * (W_TILE >> 4)), dh + (uint64_t)(kb * (H_TILE >> 4)),
                       idesc, kb ? 1u : 0u);
        }
        __syncwarp();
        dw += (uint64_t)KB0 * (W_TILE >> 4);
        dh += (uint64_t)KB0 * (H_TILE >> 4);
      }
      if (elect_one()) mma_commit(&acc);   // always: the epilogue counts on one arrival per step
      __syncwarp();
    }
  } else {
    // ---- gates and state update ------------------------------------------------------------------
    // as a reader of TMEM: warp w, lanes 0 .. 15 hold accumulator rows (gate rows) 16 w .. 16 w + 15;
    // as an owner of state: batch row tid / 4 of the group, hidden units 4 (tid % 4) .. + 3 of the CTA
    const int zrow = 16 * warp + lane;
    const int bl = tid >> 2, u0 = 4 * (tid & 3);        // batch row inside the group, first unit inside the CTA
    const int b = grp * FB + bl;                        // batch row
    const int j0 = cta * FU + u0;                       // first hidden unit
    const bool owner = b < a.B && j0 < a.H;
    const size_t e0 = (size_t)b * a.H + j0;             // element index of (b, j0) in a [B][H] array
    const bool two = KB0 < KB;
    FwdCell st;
    fwd_cell_init(st, a, owner, b, j0, e0);
    for (int i = 0; i < a.n; ++i) {
      const DevOp op = a.ops[i];
      const bool got = wait_or_fail(&acc, (uint32_t)i & 1, &failed);
      tc_fence_after_sync();
      for (int h = 0; h < (two ? 2 : 1); ++h) {
        uint32_t r[32];
        tmem_ld_32x32(tmem + ((uint32_t)(32 * warp) << 16) + (uint32_t)(h * FB), r);
        tmem_ld_wait();
        if (lane < 16) {
          float* dst = part + (size_t)h * FB * PART_LD + zrow;
#pragma unroll
          for (int n = 0; n < FB; ++n) dst[n * PART_LD] = __uint_as_float(r[n]);
        }
      }
      tc_fence_before_sync();
      named_barrier(1, 128);   // the accumulators of every gate row are in shared memory
      FwdCellOut out;
      if (got && owner) {
        float4 z[4];
        const float* p0 = part + (size_t)bl * PART_LD + 4 * u0;
        fwd_cell_sum(st, p0, two ? p0 + FB * PART_LD : nullptr, z);
        fwd_cell_gates(st, z, out);
        // h_k first: it is what the other CTAs wait for
        *reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(a.ws + (size_t)op.h_dst * 16) + e0) = out.hnew;
      }
      named_barrier(1, 128);   // all of this CTA's h_k stores precede the release below; the parts are free again
      if (tid == 0) red_release_add(sync, 1u);
      if (got && owner) fwd_cell_rest(st, a, op, out, i, b, j0, e0);
    }
  }

  tc_fence_before_sync();
  __syncthreads();
  if (tid == 0) {
    if (failed) *a.status = MEBPTT_ERR_TIMEOUT;
    else if (blockIdx.x == 0) a.counters[0] += a.n;
  }
  if (warp == 4) tmem_dealloc(tmem, 64);
}

// ------------------------------------------------------------------------------------------
// backward run
// ------------------------------------------------------------------------------------------
struct BwdRunArgs {
  const DevOp* ops;        // consecutive backward operations, k descending, all in one chunk
  int n;
  char* ws;
  const float* dha;        // [S][B][H]: gradient entering h_k from the readout, row block (k-1) % S
  __nv_bfloat16* dz;       // [S][B][4H] staging, row block (k-1) % S, gate columns permuted
  float* dh;               // [B][H] carried dL/dh (in: from step k_hi + 1; out: for step k_lo - 1)
  float* dc;               // [B][H] carried dL/dc
  const float* loss_part;  // [S][loss_parts]
  float* loss_t;           // [t]
  uint32_t* sync;
  int* status;
  int64_t* counters;
  int B, H, S;
  uint32_t plane16, hsz16;
  const float* zleaf;      // leaf batch: [S][B][4H] pre-activations z_k (gate columns permuted); NULL otherwise
  int loss_parts;          // partial sums of the loss per step
  int tb;                  // clustered kernel: K tiles per barrier and, in slab mode, per copy
  int slab;                // clustered kernel: 1: tm_dz is a blocked 3-D map and one copy brings tb tiles
  uint32_t expect;         // signals a step is complete with: the grid size (a testing aid may ask for one too many)
  uint32_t poll_limit;     // polls of the step counter before the wait gives up
};

// What the gate derivatives of one batch row and 8 hidden units read from memory at one step: the
// stored gates and cell states and the readout gradient.  None of it depends on the recurrence,
// so it can be fetched while the exchange of the previous step is still in flight.
struct GateInputs {
  uint4 qi, qf, qg, qo;
  float4 t0, t1, p0, p1, d0, d1;
};
__device__ __forceinline__ GateInputs load_gate_inputs(const BwdRunArgs& a, const DevOp& op, int sidx, int b, int cta,
                                                       size_t e0, size_t pl) {
  GateInputs in;
  const char* ws = a.ws;
  const float* dha = a.dha + ((size_t)sidx * a.B) * a.H + e0;
  in.d0 = *reinterpret_cast<const float4*>(dha);
  in.d1 = *reinterpret_cast<const float4*>(dha + 4);
  const float* cpp = reinterpret_cast<const float*>(ws + (size_t)op.c_src * 16) + e0;
  in.p0 = *reinterpret_cast<const float4*>(cpp);
  in.p1 = *reinterpret_cast<const float4*>(cpp + 4);
  if (a.zleaf) {
    // A leaf of the recursion: no internal state was stored.  Its forward operation is redone
    // here from the pre-activations, with exactly the arithmetic of the forward kernel (gates
    // rounded to bfloat16 as they would have been stored, c_k from the unrounded gates).
    const float4* zp = reinterpret_cast<const float4*>(a.zleaf + ((size_t)sidx * a.B + b) * 4 * a.H + (size_t)cta * NG);
    const float cp[NU] = {in.p0.x, in.p0.y, in.p0.z, in.p0.w, in.p1.x, in.p1.y, in.p1.z, in.p1.w};
    float ct[NU];
    uint32_t gi[4], gf[4], gg[4], go[4];
#pragma unroll
    for (int u = 0; u < NU; u += 2) {
      float iv[2], fv[2], gv[2], ov[2];
#pragma unroll
      for (int d = 0; d < 2; ++d) {
        const float4 z = zp[u + d];
        iv[d] = sigmoid_fast(z.x);
        fv[d] = sigmoid_fast(z.y);
        gv[d] = tanh_fast(z.z);
        ov[d] = sigmoid_fast(z.w);
        ct[u + d] = fmaf(fv[d], cp[u + d], iv[d] * gv[d]);
      }
      gi[u / 2] = pack_bf16x2(iv[0], iv[1]);
      gf[u / 2] = pack_bf16x2(fv[0], fv[1]);
      gg[u / 2] = pack_bf16x2(gv[0], gv[1]);
      go[u / 2] = pack_bf16x2(ov[0], ov[1]);
    }
    in.qi = make_uint4(gi[0], gi[1], gi[2], gi[3]);
    in.qf = make_uint4(gf[0], gf[1], gf[2], gf[3]);
    in.qg = make_uint4(gg[0], gg[1], gg[2], gg[3]);
    in.qo = make_uint4(go[0], go[1], go[2], go[3]);
    in.t0 = make_float4(ct[0], ct[1], ct[2], ct[3]);
    in.t1 = make_float4(ct[4], ct[5], ct[6], ct[7]);
    return in;
  }
  const __nv_bfloat16* g = reinterpret_cast<const __nv_bfloat16*>(ws + (size_t)op.gates * 16) + e0;
  in.qi = *reinterpret_cast<const uint4*>(g);
  in.qf = *reinterpret_cast<const uint4*>(g + pl);
  in.qg = *reinterpret_cast<const uint4*>(g + 2 * pl);
  in.qo = *reinterpret_cast<const uint4*>(g + 3 * pl);
  const float* ctp = reinterpret_cast<const float*>(ws + (size_t)op.c_dst * 16) + e0;
  in.t0 = *reinterpret_cast<const float4*>(ctp);
  in.t1 = *reinterpret_cast<const float4*>(ctp + 4);
  return in;
}

// Gate derivatives from the fetched inputs and the carried (dh, dc); writes dz (bfloat16, columns
// 4 u + q) to the staging chunk and leaves dc = dc_t * f for the next (earlier) step.
__device__ __forceinline__ void compute_gates(const BwdRunArgs& a, const GateInputs& in, int sidx, int b, int cta,
                                              const float (&dh)[NU], float (&dc)[NU]) {
  const int G = 4 * a.H;
  const float dhav[NU] = {in.d0.x, in.d0.y, in.d0.z, in.d0.w, in.d1.x, in.d1.y, in.d1.z, in.d1.w};
  const uint32_t wi[4] = {in.qi.x, in.qi.y, in.qi.z, in.qi.w}, wf[4] = {in.qf.x, in.qf.y, in.qf.z, in.qf.w};
  const uint32_t wg[4] = {in.qg.x, in.qg.y, in.qg.z, in.qg.w}, wo[4] = {in.qo.x, in.qo.y, in.qo.z, in.qo.w};
  const float ct[NU] = {in.t0.x, in.t0.y, in.t0.z, in.t0.w, in.t1.x, in.t1.y, in.t1.z, in.t1.w};
  const float cp[NU] = {in.p0.x, in.p0.y, in.p0.z, in.p0.w, in.p1.x, in.p1.y, in.p1.z, in.p1.w};
  uint32_t out[NG / 2];
#pragma unroll
  for (int u = 0; u < NU; ++u) {
    const int w = u >> 1;
    const bool hi = (u & 1) != 0;
    const float gi = hi ? bf16_hi(wi[w]) : bf16_lo(wi[w]);
    const float gf = hi ? bf16_hi(wf[w]) : bf16_lo(wf[w]);
    const float gg = hi ? bf16_hi(wg[w]) : bf16_lo(wg[w]);
    const float go = hi ? bf16_hi(wo[w]) : bf16_lo(wo[w]);
    const float dht = dhav[u] + dh[u];
    const float th = tanh_fast(ct[u]);
    const float d_o = dht * th;
    const float dct = fmaf(dht * go, 1.f - th * th, dc[u]);
    const float zi = dct * gg * gi * (1.f - gi);
    const float zf = dct * cp[u] * gf * (1.f - gf);
    const float zg = dct * gi * (1.f - gg * gg);
    const float zo = d_o * go * (1.f - go);
    dc[u] = dct * gf;
    out[2 * u] = pack_bf16x2(zi, zf);
    out[2 * u + 1] = pack_bf16x2(zg, zo);
  }
  uint4* dzp = reinterpret_cast<uint4*>(a.dz + ((size_t)sidx * a.B + b) * G + (size_t)cta * NG);
#pragma unroll
  for (int v = 0; v < NG / 8; ++v) dzp[v] = make_uint4(out[4 * v], out[4 * v + 1], out[4 * v + 2], out[4 * v + 3]);
}

__device__ __forceinline__ void backward_gates(const BwdRunArgs& a, const DevOp& op, int sidx, int b, int cta,
                                               size_t e0, size_t pl, const float (&dh)[NU], float (&dc)[NU]) {
  const GateInputs in = load_gate_inputs(a, op, sidx, b, cta, e0, pl);
  compute_gates(a, in, sidx, b, cta, dh, dc);
}

template <int BM>
__global__ void __launch_bounds__(128, 1) bwd_run_kernel(const __grid_constant__ CUtensorMap tm_dz,
                                                         const __grid_constant__ CUtensorMap tm_wt,
                                                         const BwdRunArgs a) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ uint64_t wfull, full[NST], empty[NST], acc;
  __shared__ uint32_t tmem_slot;
  __shared__ int failed;

  uint8_t* sm = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int KB = (4 * a.H + 63) / 64;
  uint8_t* sW = sm;                    // KB tiles of [8 rows][128 B]: rows 8c .. 8c+7 of W_hh^T
  uint8_t* ring = sm + KB * 1024;
  constexpr uint32_t A_TILE = BM * 128;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int cta = blockIdx.x, ncta = gridDim.x;
  const bool is_p = (tid == 0), is_mma = (tid == 32);

  if (tid == 0) {
    mbar_init(&wfull, 1);
    for (int s = 0; s < NST; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    mbar_init(&acc, 1);
    failed = 0;
    mbar_fence_init();
    tma_prefetch_desc(&tm_dz);
    tma_prefetch_desc(&tm_wt);
  }
  if (warp == 1) tmem_alloc(&tmem_slot, 32);
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = tmem_slot;
  grid_dep_wait();
  if (tid == 0) grid_dep_launch();

  if (is_p) {
    mbar_arrive_expect_tx(&wfull, (uint32_t)KB * 1024u);
    for (int kb = 0; kb < KB; ++kb) tma_load_2d(sW + kb * 1024, &tm_wt, kb * 64, cta * NU, &wfull);
  }

  const int b = (BM == 64) ? (16 * warp + lane) : (32 * warp + lane);
  const bool owner = ((BM == 64) ? (lane < 16) : true) && b < a.B;
  const int j0 = cta * NU;
  const size_t e0 = (size_t)b * a.H + j0;
  const size_t pl = (size_t)a.plane16 * 8;
  float dh[NU], dc[NU];
  if (owner) {
    const float4 a0 = *reinterpret_cast<const float4*>(a.dh + e0), a1 = *reinterpret_cast<const float4*>(a.dh + e0 + 4);
    const float4 c0 = *reinterpret_cast<const float4*>(a.dc + e0), c1 = *reinterpret_cast<const float4*>(a.dc + e0 + 4);
    dh[0] = a0.x; dh[1] = a0.y; dh[2] = a0.z; dh[3] = a0.w; dh[4] = a1.x; dh[5] = a1.y; dh[6] = a1.z; dh[7] = a1.w;
    dc[0] = c0.x; dc[1] = c0.y; dc[2] = c0.z; dc[3] = c0.w; dc[4] = c1.x; dc[5] = c1.y; dc[6] = c1.z; dc[7] = c1.w;
  } else {
#pragma unroll
    for (int u = 0; u < NU; ++u) { dh[u] = 0.f; dc[u] = 0.f; }
  }

  uint32_t issued = 0, consumed = 0;
  constexpr uint32_t idesc = make_idesc(1, BM, NU, false, false);

  for (int i = 0; i < a.n; ++i) {
    const DevOp op = a.ops[i];
    const int sidx = (op.k - 1) % a.S;
    if (i > 0) {
      // dh for this step = the slice of dz_{k+1} W_hh this CTA computed in the previous iteration
      const bool got = wait_or_fail(&acc, (uint32_t)(i - 1) & 1, &failed);
      tc_fence_after_sync();
      uint32_t r[NU];
      tmem_ld_32x8(tmem + ((uint32_t)(32 * warp) << 16), r);
      tmem_ld_wait();
      if (got) {
#pragma unroll
        for (int u = 0; u < NU; ++u) dh[u] = __uint_as_float(r[u]);
      }
    }
    if (owner && !failed) backward_gates(a, op, sidx, b, cta, e0, pl, dh, dc);
    if (cta == 0 && tid == 0) {
      // loss term of this step: its partial sums in a fixed order
      float s = 0.f;
      for (int p = 0; p < a.loss_parts; ++p) s += a.loss_part[sidx * a.loss_parts + p];
      a.loss_t[op.k - 1] = s;
    }
    fence_proxy_async();
    tc_fence_before_sync();
    __syncthreads();
    if (tid == 0) red_release_add(a.sync, 1u);
    if (failed) break;

    if (is_p) {
      // ---- producer: all of dz_k through the ring -----------------------------------------
      bool ok = wait_counter(a.sync, (uint32_t)(i + 1) * a.expect, &failed, a.poll_limit);
      if (ok) {
        fence_proxy_async();
        const int32_t row = sidx * a.B;
        for (int kb = 0; kb < KB && ok; ++kb, ++issued) {
          const uint32_t s = issued % NST, it = issued / NST;
          if (it > 0) ok = wait_or_fail(&empty[s], (it - 1) & 1, &failed);
          if (!ok) break;
          mbar_arrive_expect_tx(&full[s], A_TILE);
          tma_load_2d(ring + s * A_TILE, &tm_dz, kb * 64, row, &full[s]);
        }
      }
    } else if (is_mma) {
      bool ok = true;
      if (i == 0) ok = wait_or_fail(&wfull, 0, &failed);
      for (int kb = 0; kb < KB && ok; ++kb, ++consumed) {
        const uint32_t s = consumed % NST, it = consumed / NST;
        ok = wait_or_fail(&full[s], it & 1, &failed);
        if (!ok) break;
        tc_fence_after_sync();
        const uint32_t a0 = smem_u32(ring + s * A_TILE), b0 = smem_u32(sW + kb * 1024);
#pragma unroll
        for (int k4 = 0; k4 < 4; ++k4)
          mma_f16(tmem, make_desc_sw128(a0 + k4 * 32, 16, 1024), make_desc_sw128(b0 + k4 * 32, 16, 1024), idesc,
                  (kb > 0 || k4 > 0) ? 1u : 0u);
        mma_commit(&empty[s]);
      }
      mma_commit(&acc);
    }
    __syncwarp();
  }

  if (!failed) {
    // the gradient that leaves the run: dh from the last product, dc from registers
    const bool got = wait_or_fail(&acc, (uint32_t)(a.n - 1) & 1, &failed);
    tc_fence_after_sync();
    uint32_t r[NU];
    tmem_ld_32x8(tmem + ((uint32_t)(32 * warp) << 16), r);
    tmem_ld_wait();
    if (got && owner) {
      *reinterpret_cast<float4*>(a.dh + e0) = make_float4(__uint_as_float(r[0]), __uint_as_float(r[1]),
                                                           __uint_as_float(r[2]), __uint_as_float(r[3]));
      *reinterpret_cast<float4*>(a.dh + e0 + 4) = make_float4(__uint_as_float(r[4]), __uint_as_float(r[5]),
                                                               __uint_as_float(r[6]), __uint_as_float(r[7]));
      *reinterpret_cast<float4*>(a.dc + e0) = make_float4(dc[0], dc[1], dc[2], dc[3]);
      *reinterpret_cast<float4*>(a.dc + e0 + 4) = make_float4(dc[4], dc[5], dc[6], dc[7]);
    }
  }
  tc_fence_before_sync();
  __syncthreads();
  if (failed) {
    if (tid == 0) *a.status = MEBPTT_ERR_TIMEOUT;
    if (is_p) {
      for (uint32_t q = (issued > NST ? issued - NST : 0); q < issued; ++q)
        (void)mbar_wait(&full[q % NST], (q / NST) & 1);
      (void)mbar_wait(&wfull, 0);
    }
    __syncthreads();
  } else if (cta == 0 && tid == 0) {
    a.counters[1] += a.n;
  }
  if (warp == 1) tmem_dealloc(tmem, 32);
}

// ------------------------------------------------------------------------------------------
// backward run, split over thread-block clusters
// ------------------------------------------------------------------------------------------
// The product dh_{k-1} = dz_k W_hh has K = 4H: a CTA that wants its 8 columns on its own must
// pull all of dz_k (B x 4H) through shared memory every step.  Here CS neighbouring CTAs (one
// cluster, 8 CS hidden units) share the work along K instead: CTA r multiplies the K-slice
// [r G/CS, (r+1) G/CS) of dz_k by the matching [8 CS x G/CS] block of W_hh^T, resident in its
// shared memory, into a partial [B x 8 CS] tile; the partial tiles go to shared memory, the
// cluster synchronises, and each owner thread adds the CS partial values of its 8 columns in the
// order r = 0 .. CS-1, reading its peers' tiles through distributed shared memory.
template <int CS>
__global__ void __launch_bounds__(192, 1) bwd_run_cluster_kernel(const __grid_constant__ CUtensorMap tm_dz,
                                                                 const __grid_constant__ CUtensorMap tm_wt,
                                                                 const BwdRunArgs a) {
  constexpr int BM = 64;
  constexpr int NC = NU * CS;              // columns of dh the cluster produces
  constexpr uint32_t A_TILE = BM * 128;
  constexpr uint32_t W_TILE = NC * 128;
  extern __shared__ uint8_t smem_raw[];
  __shared__ uint64_t wfull, full[4], acc, pready[2];
  __shared__ uint32_t tmem_slot;
  __shared__ int failed;

  uint8_t* sm = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int G = 4 * a.H;
  const int KBS = (G / 64) / CS;           // 64-wide K blocks in this CTA's slice (<= 16)
  const int TB = a.tb;                     // K tiles per barrier
  const int NQ = (KBS + TB - 1) / TB;      // <= 4
  uint8_t* sW = sm;                        // KBS tiles [NC rows][128 B]
  uint8_t* ring = sW + KBS * W_TILE;       // KBS tiles [64 rows][128 B], all of the slice at once
  // partial sums received from the cluster: [2 buffers][CS senders][64 rows][8 columns]
  float* recv = reinterpret_cast<float*>(ring + NQ * TB * A_TILE);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int cta = blockIdx.x, ncta = gridDim.x;
  const uint32_t rank = cluster_ctarank();
  const int cl = cta / CS;

  if (tid == 0) {
    mbar_init(&wfull, 1);
    for (int s = 0; s < 4; ++s) mbar_init(&full[s], 1);
    mbar_init(&acc, 1);
    mbar_init(&pready[0], CS);
    mbar_init(&pready[1], CS);
    failed = 0;
    mbar_fence_init();
    tma_prefetch_desc(&tm_dz);
    tma_prefetch_desc(&tm_wt);
  }
  if (warp == 4) tmem_alloc(&tmem_slot, 64);
  tc_fence_before_sync();
  cluster_sync();                          // peers arrive on each other's barriers: all must be initialised
  tc_fence_after_sync();
  const uint32_t tmem = tmem_slot;
  grid_dep_wait();

  if (warp == 4) {
    // ---- producer: this CTA's K-slice of dz_k, all of it in flight at once; lane 0 watches the
    // step counter, lanes 0 .. NQ-1 each request one block of four K tiles -------------------------
    if (lane == 0) {
      mbar_arrive_expect_tx(&wfull, (uint32_t)KBS * W_TILE);
      for (int kb = 0; kb < KBS; ++kb)
        tma_load_2d(sW + kb * W_TILE, &tm_wt, ((int)rank * KBS + kb) * 64, cl * NC, &wfull);
    }
    int armed = -1;
    for (int i = 0; i < a.n; ++i) {
      const int sidx = (a.ops[i].k - 1) % a.S;
      if (cta == 0 && lane == 31) {
        // loss term of this step: its partial sums in a fixed order (on a lane that is off the
        // critical path of the recurrence)
        float sum = 0.f;
        for (int p = 0; p < a.loss_parts; ++p) sum += a.loss_part[sidx * a.loss_parts + p];
        a.loss_t[a.ops[i].k - 1] = sum;
      }
      int go = 1;
      if (lane == 0) go = !failed && wait_counter(a.sync, (uint32_t)(i + 1) * a.expect, &failed, a.poll_limit) && !failed;
      go = __shfl_sync(0xffffffffu, go, 0);
      if (!go) continue;
      if (lane < NQ) {
        // (the TMA unit takes its copy requests one at a time, ~100 ns each: in slab mode one copy over
        // a map that sees a row as blocks of 64 columns brings the TB tiles of a barrier)
        fence_proxy_async_global();
        const int32_t row = sidx * a.B;
        const int q = lane;
        const int kb0 = TB * q, kb1 = (kb0 + TB < KBS) ? kb0 + TB : KBS;
        if (a.slab) {
          mbar_arrive_expect_tx(&full[q], (uint32_t)TB * A_TILE);   // a box counts in full
          tma_load_3d(ring + kb0 * A_TILE, &tm_dz, 0, row, (int)rank * KBS + kb0, &full[q]);
        } else {
          mbar_arrive_expect_tx(&full[q], (uint32_t)(kb1 - kb0) * A_TILE);
          for (int kb = kb0; kb < kb1; ++kb)
            tma_load_2d(ring + kb * A_TILE, &tm_dz, ((int)rank * KBS + kb) * 64, row, &full[q]);
        }
      }
      armed = i;
      if (i == a.n - 1 && lane == 0) grid_dep_launch();
      __syncwarp();
    }
    if (failed && lane == 0) {
      (void)mbar_wait(&wfull, 0);
      if (armed >= 0)
        for (int q = 0; q < NQ; ++q) (void)mbar_wait(&full[q], (uint32_t)armed & 1);
    }
  } else if (warp == 5) {
    // ---- MMA issuer: the whole warp walks the loop, one elected lane issues --------------------
    constexpr uint32_t idesc = make_idesc(1, BM, NC, false, false);
    bool ok = wait_or_fail(&wfull, 0, &failed);
    const uint64_t a_desc0 = make_desc_sw128(smem_u32(ring), 16, 1024);
    const uint64_t b_desc0 = make_desc_sw128(smem_u32(sW), 16, 1024);
    for (int i = 0; i < a.n; ++i) {
      uint64_t da = a_desc0, db = b_desc0;
      for (int q = 0; q < NQ && ok; ++q) {
        ok = wait_or_fail(&full[q], (uint32_t)i & 1, &failed);
        if (!ok) break;
        tc_fence_after_sync();
        const int nkb = (TB * q + TB < KBS) ? TB : KBS - TB * q;
        if (elect_one()) {
          for (int kb = 0; kb < nkb; ++kb)
            mma_f16_x4(tmem, da + (uint64_t)(kb * (A_TILE >> 4)), db + (uint64_t)(kb * (W_TILE >> 4)), idesc,
                       (q > 0 || kb > 0) ? 1u : 0u);
        }
        __syncwarp();
        da += (uint64_t)TB * (A_TILE >> 4);
        db += (uint64_t)TB * (W_TILE >> 4);
      }
      if (elect_one()) mma_commit(&acc);   // always: the epilogue counts on one arrival per step
      __syncwarp();
    }
  } else {
    // ---- gate derivatives: warp w owns tile rows 16w .. 16w+15 ----------------------------------
    const int b = 16 * warp + lane;
    const bool row_thread = lane < 16;             // holds an accumulator row in TMEM
    const bool owner = row_thread && b < a.B;
    const int j0 = cta * NU;
    const size_t e0 = (size_t)b * a.H + j0;
    const size_t pl = (size_t)a.plane16 * 8;
    float dh[NU], dc[NU];
    if (owner) {
      const float4 a0 = *reinterpret_cast<const float4*>(a.dh + e0), a1 = *reinterpret_cast<const float4*>(a.dh + e0 + 4);
      const float4 c0 = *reinterpret_cast<const float4*>(a.dc + e0), c1 = *reinterpret_cast<const float4*>(a.dc + e0 + 4);
      dh[0] = a0.x; dh[1] = a0.y; dh[2] = a0.z; dh[3] = a0.w; dh[4] = a1.x; dh[5] = a1.y; dh[6] = a1.z; dh[7] = a1.w;
      dc[0] = c0.x; dc[1] = c0.y; dc[2] = c0.z; dc[3] = c0.w; dc[4] = c1.x; dc[5] = c1.y; dc[6] = c1.z; dc[7] = c1.w;
    } else {
#pragma unroll
      for (int u = 0; u < NU; ++u) { dh[u] = 0.f; dc[u] = 0.f; }
    }

    // Reduces the partial tiles of product number `it` into this thread's dh.  Each row thread
    // reads its row of this CTA's partial tile from TMEM and sends the 8 columns that belong to
    // CTA p straight into p's shared memory; once all CS senders have signalled, the owner adds
    // the CS partial values of its columns in the order of the ranks.
    auto reduce_partials = [&](int it) {
      float* buf = recv + (size_t)(it & 1) * CS * BM * NU;
      const bool got = wait_or_fail(&acc, (uint32_t)it & 1, &failed);
      tc_fence_after_sync();
#pragma unroll
      for (int c0 = 0; c0 < NC; c0 += 32) {
        uint32_t r[32];
        tmem_ld_32x32(tmem + ((uint32_t)(32 * warp) << 16) + (uint32_t)c0, r);
        tmem_ld_wait();
        if (row_thread) {
#pragma unroll
          for (int pp = 0; pp < 4; ++pp) {   // 32 columns = the columns of four CTAs
            float* dst = buf + ((size_t)rank * BM + b) * NU;      // slot of sender `rank`, row b
            const uint32_t peer = (uint32_t)(c0 / NU + pp);
            st_peer_f4(dst, peer, make_float4(__uint_as_float(r[8 * pp]), __uint_as_float(r[8 * pp + 1]),
                                              __uint_as_float(r[8 * pp + 2]), __uint_as_float(r[8 * pp + 3])));
            st_peer_f4(dst + 4, peer, make_float4(__uint_as_float(r[8 * pp + 4]), __uint_as_float(r[8 * pp + 5]),
                                                  __uint_as_float(r[8 * pp + 6]), __uint_as_float(r[8 * pp + 7])));
          }
        }
      }
      tc_fence_before_sync();
      named_barrier(1, 128);
      if (tid < CS) mbar_arrive_peer(&pready[it & 1], (uint32_t)tid);   // release: the stores above are visible
      bool all = false;
      for (uint32_t spin = 0; spin < kSpinLimit; ++spin) {
        if (mbar_try_wait_cluster(&pready[it & 1], (uint32_t)(it >> 1) & 1)) { all = true; break; }
        if (spin > 256) {
          if (failed) break;
          __nanosleep(64);
        }
      }
      if (!all) failed = 1;
      if (got && all && owner) {
        float sum[NU];
#pragma unroll
        for (int u = 0; u < NU; ++u) sum[u] = 0.f;
#pragma unroll
        for (int p = 0; p < CS; ++p) {
          const float4* src = reinterpret_cast<const float4*>(buf + ((size_t)p * BM + b) * NU);
          const float4 v0 = src[0], v1 = src[1];
          sum[0] += v0.x; sum[1] += v0.y; sum[2] += v0.z; sum[3] += v0.w;
          sum[4] += v1.x; sum[5] += v1.y; sum[6] += v1.z; sum[7] += v1.w;
        }
#pragma unroll
        for (int u = 0; u < NU; ++u) dh[u] = sum[u];
      }
    };

    GateInputs gin;
    if (owner) gin = load_gate_inputs(a, a.ops[0], (a.ops[0].k - 1) % a.S, b, cta, e0, pl);
    for (int i = 0; i < a.n; ++i) {
      const DevOp op = a.ops[i];
      const int sidx = (op.k - 1) % a.S;
      if (i > 0) reduce_partials(i - 1);
      if (owner && !failed) compute_gates(a, gin, sidx, b, cta, dh, dc);
      named_barrier(1, 128);   // all of this CTA's dz stores precede the release below
      if (tid == 0) red_release_add(a.sync, 1u);
      // the inputs of the next (earlier) step do not depend on the recurrence: fetch them while the
      // exchange of this step is in flight
      if (owner && i + 1 < a.n) gin = load_gate_inputs(a, a.ops[i + 1], (a.ops[i + 1].k - 1) % a.S, b, cta, e0, pl);
    }
    reduce_partials(a.n - 1);
    if (owner && !failed) {
      *reinterpret_cast<float4*>(a.dh + e0) = make_float4(dh[0], dh[1], dh[2], dh[3]);
      *reinterpret_cast<float4*>(a.dh + e0 + 4) = make_float4(dh[4], dh[5], dh[6], dh[7]);
      *reinterpret_cast<float4*>(a.dc + e0) = make_float4(dc[0], dc[1], dc[2], dc[3]);
      *reinterpret_cast<float4*>(a.dc + e0 + 4) = make_float4(dc[4], dc[5], dc[6], dc[7]);
    }
  }

  tc_fence_before_sync();
  cluster_sync();   // no CTA leaves while a peer may still read its partial tiles or signal it
  if (tid == 0) {
    if (failed) *a.status = MEBPTT_ERR_TIMEOUT;
    else if (cta == 0) a.counters[1] += a.n;
  }
  if (warp == 4) tmem_dealloc(tmem, 64);
}

// ------------------------------------------------------------------------------------------
// backward run, clusters inside groups of batch rows
// ------------------------------------------------------------------------------------------
// The same split along K as above (clusters of four CTAs, partial tiles reduced in rank order), with
// what the forward kernel does about latency: the grid is cut into groups of CTAs that each own
// FB = 32 batch rows and have a step counter of their own, so that a CTA pulls half the bytes of
// dz_k and a step is signalled by half the CTAs; the product is taken transposed (the cluster's 64
// columns of dh, as rows of W_hh^T resident in shared memory, are the M side of the MMA, the 32
// batch rows the N side); and all 128 epilogue threads take part in the gate derivatives, each with
// four hidden units of one batch row.  CTA c of a group owns hidden units 16 c .. 16 c + 15; the
// partial sums of a column are added in the order of the ranks as above, so both kernels give the
// same bits.
struct GateInputs4 {
  uint2 qi, qf, qg, qo;
  float4 t, p, d;
};
__device__ __forceinline__ GateInputs4 load_gate_inputs4(const BwdRunArgs& a, const DevOp& op, int sidx, int b, int j0,
                                                         size_t e0, size_t pl) {
  GateInputs4 in;
  const char* ws = a.ws;
  in.d = *reinterpret_cast<const float4*>(a.dha + ((size_t)sidx * a.B) * a.H + e0);
  in.p = *reinterpret_cast<const float4*>(reinterpret_cast<const float*>(ws + (size_t)op.c_src * 16) + e0);
  if (a.zleaf) {
    // a leaf of the recursion: its forward operation redone from the pre-activations, with the
    // arithmetic of the forward kernel
    const float4* zp = reinterpret_cast<const float4*>(a.zleaf + ((size_t)sidx * a.B + b) * 4 * a.H + (size_t)4 * j0);
    const float cp[4] = {in.p.x, in.p.y, in.p.z, in.p.w};
    float ct[4], iv[4], fv[4], gv[4], ov[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const float4 z = zp[u];
      iv[u] = sigmoid_fast(z.x);
      fv[u] = sigmoid_fast(z.y);
      gv[u] = tanh_fast(z.z);
      ov[u] = sigmoid_fast(z.w);
      ct[u] = fmaf(fv[u], cp[u], iv[u] * gv[u]);
    }
    in.qi = make_uint2(pack_bf16x2(iv[0], iv[1]), pack_bf16x2(iv[2], iv[3]));
    in.qf = make_uint2(pack_bf16x2(fv[0], fv[1]), pack_bf16x2(fv[2], fv[3]));
    in.qg = make_uint2(pack_bf16x2(gv[0], gv[1]), pack_bf16x2(gv[2], gv[3]));
    in.qo = make_uint2(pack_bf16x2(ov[0], ov[1]), pack_bf16x2(ov[2], ov[3]));
    in.t = make_float4(ct[0], ct[1], ct[2], ct[3]);
    return in;
  }
  const __nv_bfloat16* g = reinterpret_cast<const __nv_bfloat16*>(ws + (size_t)op.gates * 16) + e0;
  in.qi = *reinterpret_cast<const uint2*>(g);
  in.qf = *reinterpret_cast<const uint2*>(g + pl);
  in.qg = *reinterpret_cast<const uint2*>(g + 2 * pl);
  in.qo = *reinterpret_cast<const uint2*>(g + 3 * pl);
  in.t = *reinterpret_cast<const float4*>(reinterpret_cast<const float*>(ws + (size_t)op.c_dst * 16) + e0);
  return in;
}

// The arithmetic of compute_gates for four hidden units.
__device__ __forceinline__ void compute_gates4(const BwdRunArgs& a, const GateInputs4& in, int sidx, int b, int j0,
                                               const float (&dh)[4], float (&dc)[4]) {
  const int G = 4 * a.H;
  const float dhav[4] = {in.d.x, in.d.y, in.d.z, in.d.w};
  const uint32_t wi[2] = {in.qi.x, in.qi.y}, wf[2] = {in.qf.x, in.qf.y}, wg[2] = {in.qg.x, in.qg.y}, wo[2] = {in.qo.x, in.qo.y};
  const float ct[4] = {in.t.x, in.t.y, in.t.z, in.t.w};
  const float cp[4] = {in.p.x, in.p.y, in.p.z, in.p.w};
  uint32_t out[8];
#pragma unroll
  for (int u = 0; u < 4; ++u) {
    const int w = u >> 1;
    const bool hi = (u & 1) != 0;
    const float gi = hi ? bf16_hi(wi[w]) : bf16_lo(wi[w]);
    const float gf = hi ? bf16_hi(wf[w]) : bf16_lo(wf[w]);
    const float gg = hi ? bf16_hi(wg[w]) : bf16_lo(wg[w]);
    const float go = hi ? bf16_hi(wo[w]) : bf16_lo(wo[w]);
    const float dht = dhav[u] + dh[u];
    const float th = tanh_fast(ct[u]);
    const float d_o = dht * th;
    const float dct = fmaf(dht * go, 1.f - th * th, dc[u]);
    const float zi = dct * gg * gi * (1.f - gi);
    const float zf = dct * cp[u] * gf * (1.f - gf);
    const float zg = dct * gi * (1.f - gg * gg);
    const float zo = d_o * go * (1.f - go);
    dc[u] = dct * gf;
    out[2 * u] = pack_bf16x2(zi, zf);
    out[2 * u + 1] = pack_bf16x2(zg, zo);
  }
  uint4* dzp = reinterpret_cast<uint4*>(a.dz + ((size_t)sidx * a.B + b) * G + (size_t)4 * j0);
  dzp[0] = make_uint4(out[0], out[1], out[2], out[3]);
  dzp[1] = make_uint4(out[4], out[5], out[6], out[7]);
}

constexpr int GCS = 4;           // CTAs per cluster
constexpr int RECV_LD = FB + 4;  // row stride of a received partial tile, [dh column][batch row] (floats)

__global__ void __launch_bounds__(192, 1) bwd_run_group_kernel(const __grid_constant__ CUtensorMap tm_dz,
                                                               const __grid_constant__ CUtensorMap tm_wt,
                                                               const BwdRunArgs a) {
  constexpr int NC = FU * GCS;             // columns of dh the cluster produces: the M of the MMA
  constexpr uint32_t W_TILE = NC * 128;    // [64 columns of dh][64 contraction indices]
  constexpr uint32_t A_TILE = FB * 128;    // [32 batch rows][64 contraction indices]
  extern __shared__ uint8_t smem_raw[];
  __shared__ uint64_t wfull, full[4], acc, pready[2];
  __shared__ uint32_t tmem_slot;
  __shared__ int failed;

  uint8_t* sm = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int G = 4 * a.H;
  const int KBS = (G / 64) / GCS;          // 64-wide K blocks in this CTA's slice (<= 16)
  const int TB = a.tb;                     // K tiles per barrier and per copy
  const int NQ = (KBS + TB - 1) / TB;      // <= 4
  uint8_t* sW = sm;                        // KBS tiles of W_hh^T
  uint8_t* ring = sW + KBS * W_TILE;       // KBS tiles of dz_k, all of the slice at once
  // partial sums received from the cluster: [2 buffers][GCS senders][16 columns][RECV_LD]
  float* recv = reinterpret_cast<float*>(ring + NQ * TB * A_TILE);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int ncg = (int)gridDim.x / ((a.B > FB) ? 2 : 1);   // CTAs per group
  const int grp = blockIdx.x / ncg, cta = blockIdx.x % ncg;
  const uint32_t rank = cluster_ctarank();
  const int cl = cta / GCS;
  uint32_t* const sync = a.sync + grp * SYNC_STRIDE;

  if (tid == 0) {
    mbar_init(&wfull, 1);
    for (int s = 0; s < 4; ++s) mbar_init(&full[s], 1);
    mbar_init(&acc, 1);
    mbar_init(&pready[0], GCS);
    mbar_init(&pready[1], GCS);
    failed = 0;
    mbar_fence_init();
    tma_prefetch_desc(&tm_dz);
    tma_prefetch_desc(&tm_wt);
  }
  if (warp == 4) tmem_alloc(&tmem_slot, 32);
  tc_fence_before_sync();
  cluster_sync();                          // peers arrive on each other's barriers: all must be initialised
  tc_fence_after_sync();
  const uint32_t tmem = tmem_slot;
  grid_dep_wait();

  if (warp == 4) {
    // ---- producer: this CTA's K-slice of the group's rows of dz_k; lane 0 watches the group's step
    // counter, lanes 0 .. NQ-1 each request one block of TB tiles -------------------------------------
    if (lane == 0) {
      mbar_arrive_expect_tx(&wfull, (uint32_t)KBS * W_TILE);
      for (int kb = 0; kb < KBS; ++kb)
        tma_load_2d(sW + kb * W_TILE, &tm_wt, ((int)rank * KBS + kb) * 64, cl * NC, &wfull);
    }
    int armed = -1;
    for (int i = 0; i < a.n; ++i) {
      const int sidx = (a.ops[i].k - 1) % a.S;
      if (blockIdx.x == 0 && lane == 31) {
        // loss term of this step: its partial sums in a fixed order (on a lane that is off the
        // critical path of the recurrence)
        float sum = 0.f;
        for (int p = 0; p < a.loss_parts; ++p) sum += a.loss_part[sidx * a.loss_parts + p];
        a.loss_t[a.ops[i].k - 1] = sum;
      }
      int go = 1;
      if (lane == 0) go = !failed && wait_counter(sync, (uint32_t)(i + 1) * a.expect, &failed, a.poll_limit) && !failed;
      go = __shfl_sync(0xffffffffu, go, 0);
      if (!go) continue;
      if (lane < NQ) {
        fence_proxy_async_global();
        // rows past the batch are never used: they only reach accumulator columns that no thread reads
        const int32_t row = sidx * a.B + grp * FB;
        mbar_arrive_expect_tx(&full[lane], (uint32_t)TB * A_TILE);   // a box counts in full
        tma_load_3d(ring + TB * lane * A_TILE, &tm_dz, 0, row, (int)rank * KBS + TB * lane, &full[lane]);
      }
      armed = i;
      if (i == a.n - 1 && lane == 0) grid_dep_launch();
      __syncwarp();
    }
    if (failed && lane == 0) {
      (void)mbar_wait(&wfull, 0);
      if (armed >= 0)
        for (int q = 0; q < NQ; ++q) (void)mbar_wait(&full[q], (uint32_t)armed & 1);
    }
  } else if (warp == 5) {
    // ---- MMA issuer: the whole warp walks the loop, one elected lane issues --------------------
    constexpr uint32_t idesc = make_idesc(1, NC, FB, false, false);
    bool ok = wait_or_fail(&wfull, 0, &failed);
    const uint64_t w_desc0 = make_desc_sw128(smem_u32(sW), 16, 1024);
    const uint64_t z_desc0 = make_desc_sw128(smem_u32(ring), 16, 1024);
    for (int i = 0; i < a.n; ++i) {
      uint64_t dw = w_desc0, dzd = z_desc0;
      for (int q = 0; q < NQ && ok; ++q) {
        ok = wait_or_fail(&full[q], (uint32_t)i & 1, &failed);
        if (!ok) break;
        tc_fence_after_sync();
        const int nkb = (TB * q + TB < KBS) ? TB : KBS - TB * q;
        if (elect_one()) {
          for (int kb = 0; kb < nkb; ++kb)
            mma_f16_x4(tmem, dw + (uint64_t)(kb * (W_TILE >> 4)), dzd + (uint64_t)(kb * (A_TILE >> 4)), idesc,
                       (q > 0 || kb > 0) ? 1u : 0u);
        }
        __syncwarp();
        dw += (uint64_t)TB * (W_TILE >> 4);
        dzd += (uint64_t)TB * (A_TILE >> 4);
      }
      if (elect_one()) mma_commit(&acc);   // always: the epilogue counts on one arrival per step
      __syncwarp();
    }
  } else {
    // ---- gate derivatives -------------------------------------------------------------------------
    // as a reader of TMEM: warp w, lanes 0 .. 15 hold accumulator rows 16 w .. 16 w + 15, the columns
    // of dh that CTA w of the cluster owns; as an owner of state: batch row tid / 4 of the group,
    // hidden units 4 (tid % 4) .. + 3 of the CTA
    const int bl = tid >> 2, u0 = 4 * (tid & 3);
    const int b = grp * FB + bl;
    const int j0 = cta * FU + u0;
    const bool owner = b < a.B;
    const size_t e0 = (size_t)b * a.H + j0;
    const size_t pl = (size_t)a.plane16 * 8;
    float dh[4], dc[4];
    if (owner) {
      const float4 a0 = *reinterpret_cast<const float4*>(a.dh + e0), c0 = *reinterpret_cast<const float4*>(a.dc + e0);
      dh[0] = a0.x; dh[1] = a0.y; dh[2] = a0.z; dh[3] = a0.w;
      dc[0] = c0.x; dc[1] = c0.y; dc[2] = c0.z; dc[3] = c0.w;
    } else {
#pragma unroll
      for (int u = 0; u < 4; ++u) { dh[u] = 0.f; dc[u] = 0.f; }
    }

    // Reduces the partial tiles of product number `it` into this thread's dh: each row thread reads
    // its row of this CTA's partial tile from TMEM (one column of dh, 32 batch rows) and sends it
    // into the shared memory of the CTA that owns the column; once all senders have signalled, an
    // owner adds the partial values of its columns in the order of the ranks.
    auto reduce_partials = [&](int it) {
      float* buf = recv + (size_t)(it & 1) * GCS * FU * RECV_LD;
      const bool got = wait_or_fail(&acc, (uint32_t)it & 1, &failed);
      tc_fence_after_sync();
      uint32_t r[32];
      tmem_ld_32x32(tmem + ((uint32_t)(32 * warp) << 16), r);
      tmem_ld_wait();
      if (lane < 16) {
        float* dst = buf + ((size_t)rank * FU + lane) * RECV_LD;      // slot of sender `rank`, column `lane` of CTA `warp`
#pragma unroll
        for (int v = 0; v < FB / 4; ++v)
          st_peer_f4(dst + 4 * v, (uint32_t)warp, make_float4(__uint_as_float(r[4 * v]), __uint_as_float(r[4 * v + 1]),
                                                              __uint_as_float(r[4 * v + 2]), __uint_as_float(r[4 * v + 3])));
      }
      tc_fence_before_sync();
      named_barrier(1, 128);
      if (tid < GCS) mbar_arrive_peer(&pready[it & 1], (uint32_t)tid);   // release: the stores above are visible
      bool all = false;
      for (uint32_t spin = 0; spin < kSpinLimit; ++spin) {
        if (mbar_try_wait_cluster(&pready[it & 1], (uint32_t)(it >> 1) & 1)) { all = true; break; }
        if (spin > 256) {
          if (failed) break;
          __nanosleep(64);
        }
      }
      if (!all) failed = 1;
      if (got && all && owner) {
        float sum[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int p = 0; p < GCS; ++p) {
          const float* src = buf + ((size_t)p * FU + u0) * RECV_LD + bl;
#pragma unroll
          for (int u = 0; u < 4; ++u) sum[u] += src[u * RECV_LD];
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) dh[u] = sum[u];
      }
    };

    GateInputs4 gin;
    if (owner) gin = load_gate_inputs4(a, a.ops[0], (a.ops[0].k - 1) % a.S, b, j0, e0, pl);
    for (int i = 0; i < a.n; ++i) {
      const DevOp op = a.ops[i];
      const int sidx = (op.k - 1) % a.S;
      if (i > 0) reduce_partials(i - 1);
      if (owner && !failed) compute_gates4(a, gin, sidx, b, j0, dh, dc);
      named_barrier(1, 128);   // all of this CTA's dz stores precede the release below
      if (tid == 0) red_release_add(sync, 1u);
      // the inputs of the next (earlier) step do not depend on the recurrence: fetch them while the
      // exchange of this step is in flight
      if (owner && i + 1 < a.n) gin = load_gate_inputs4(a, a.ops[i + 1], (a.ops[i + 1].k - 1) % a.S, b, j0, e0, pl);
    }
    reduce_partials(a.n - 1);
    if (owner && !failed) {
      *reinterpret_cast<float4*>(a.dh + e0) = make_float4(dh[0], dh[1], dh[2], dh[3]);
      *reinterpret_cast<float4*>(a.dc + e0) = make_float4(dc[0], dc[1], dc[2], dc[3]);
    }
  }

  tc_fence_before_sync();
  cluster_sync();   // no CTA leaves while a peer may still read its partial tiles or signal it
  if (tid == 0) {
    if (failed) *a.status = MEBPTT_ERR_TIMEOUT;
    else if (blockIdx.x == 0) a.counters[1] += a.n;
  }
  if (warp == 4) tmem_dealloc(tmem, 32);
}

// ------------------------------------------------------------------------------------------
// small kernels off the recurrence
// ------------------------------------------------------------------------------------------
// Packs the weights once per training step: gate rows permuted to 4 u + q (the four gates of
// hidden unit u adjacent), W_ih and W_hh split, their transposes for the backward products, the
// transposed readout matrix, and the permuted bias.  Element by element: for widths that are not
// multiples of 8 (the tiled kernel below serves the rest).
__global__ void pack_weights_scalar(const __nv_bfloat16* W, const float* bias, const __nv_bfloat16* W_out, int I, int H,
                                    int O, __nv_bfloat16* wp_ih, __nv_bfloat16* wp_hh, __nv_bfloat16* wpT_hh,
                                    __nv_bfloat16* wpT_ih, float* bias_p, __nv_bfloat16* woutT) {
  grid_dep_wait();
  grid_dep_launch();
  const int G = 4 * H, K = I + H;
  const size_t nW = (size_t)G * K;
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  for (size_t e = blockIdx.x * (size_t)blockDim.x + threadIdx.x; e < nW; e += stride) {
    const int g = (int)(e / K), col = (int)(e % K);
    const int q = g / H, u = g % H, gp = 4 * u + q;
    const __nv_bfloat16 v = W[e];
    if (col < I) {
      wp_ih[(size_t)gp * I + col] = v;
      if (wpT_ih) wpT_ih[(size_t)col * G + gp] = v;
    } else {
      wp_hh[(size_t)gp * H + (col - I)] = v;
      wpT_hh[(size_t)(col - I) * G + gp] = v;
    }
  }
  for (size_t e = blockIdx.x * (size_t)blockDim.x + threadIdx.x; e < (size_t)G; e += stride) {
    const int q = (int)e / H, u = (int)e % H;
    bias_p[4 * u + q] = bias[e];
  }
  for (size_t e = blockIdx.x * (size_t)blockDim.x + threadIdx.x; e < (size_t)O * H; e += stride) {
    const int o = (int)(e / H), j = (int)(e % H);
    woutT[(size_t)j * O + o] = W_out[e];
  }
}

// The same in tiles of 64 x 64 through shared memory, 16 bytes per access on both sides of a
// transpose (I, H, O multiples of 8).  A block of 256 threads takes tiles in turn: first those of
// W (tile row = 64 permuted gate rows, i.e. 16 hidden units), then those of W_out.
__global__ void __launch_bounds__(256) pack_weights(const __nv_bfloat16* W, const float* bias, const __nv_bfloat16* W_out, int I,
                                                    int H, int O, __nv_bfloat16* wp_ih, __nv_bfloat16* wp_hh,
                                                    __nv_bfloat16* wpT_hh, __nv_bfloat16* wpT_ih, float* bias_p,
                                                    __nv_bfloat16* woutT) {
  __shared__ __align__(16) __nv_bfloat16 tile[64][72];   // 144-byte rows: 16-byte accesses stay aligned
  grid_dep_wait();
  grid_dep_launch();
  const int G = 4 * H, K = I + H;
  const int tid = threadIdx.x;
  const int r = tid >> 2, seg = (tid & 3) * 16;   // this thread's row of a tile and its 16 columns
  const int tc_w = (K + 63) / 64, tr_w = (G + 63) / 64;
  const int tc_o = (H + 63) / 64, tr_o = (O + 63) / 64;
  const int n_w = tc_w * tr_w, n_o = tc_o * tr_o;
  for (int t = blockIdx.x; t < n_w + n_o; t += gridDim.x) {
    const bool is_w = t < n_w;
    const int tt = is_w ? t : t - n_w;
    const int r0 = (tt / (is_w ? tc_w : tc_o)) * 64, c0 = (tt % (is_w ? tc_w : tc_o)) * 64;
    const int rows = is_w ? G : O, cols = is_w ? K : H;
    // ---- in: row r0 + r of the (permuted) source, columns c0 + seg .. + 15
    const int pr = r0 + r;   // permuted gate row, or row of W_out
    uint4 v[2] = {make_uint4(0, 0, 0, 0), make_uint4(0, 0, 0, 0)};
    if (pr < rows) {
      const size_t src_row = is_w ? (size_t)((pr & 3) * H + (pr >> 2)) : (size_t)pr;
      const __nv_bfloat16* src = (is_w ? W : W_out) + src_row * cols;
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int c = c0 + seg + 8 * h;
        if (c < cols) v[h] = *reinterpret_cast<const uint4*>(src + c);
      }
    }
#pragma unroll
    for (int h = 0; h < 2; ++h) *reinterpret_cast<uint4*>(&tile[r][seg + 8 * h]) = v[h];
    if (is_w && pr < rows) {
      // the row-major copies, split at column I (a multiple of 8, so no 16-byte piece straddles it)
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int c = c0 + seg + 8 * h;
        if (c >= cols) continue;
        if (c < I) *reinterpret_cast<uint4*>(wp_ih + (size_t)pr * I + c) = v[h];
        else *reinterpret_cast<uint4*>(wp_hh + (size_t)pr * H + (c - I)) = v[h];
      }
    }
    __syncthreads();
    // ---- out, transposed: column c0 + r of the tile, rows r0 + seg .. + 15
    const int c = c0 + r;
    if (c < cols) {
      __nv_bfloat16* dst = is_w ? (c < I ? (wpT_ih ? wpT_ih + (size_t)c * G : nullptr) : wpT_hh + (size_t)(c - I) * G)
                                : woutT + (size_t)c * O;
      if (dst) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const int rr = seg + 8 * h;
          if (r0 + rr >= rows) continue;   // rows is a multiple of 8
          __align__(16) __nv_bfloat16 o[8];
#pragma unroll
          for (int j = 0; j < 8; ++j) o[j] = tile[rr + j][r];
          *reinterpret_cast<uint4*>(dst + r0 + rr) = *reinterpret_cast<const uint4*>(o);
        }
      }
    }
    __syncthreads();
  }
  for (size_t e = blockIdx.x * (size_t)blockDim.x + tid; e < (size_t)G; e += (size_t)gridDim.x * blockDim.x) {
    const int q = (int)e / H, u = (int)e % H;
    bias_p[4 * u + q] = bias[e];
  }
}

// Copies h_k and h_{k-1} of each step of a backward run from wherever the internal state lies
// into the staging chunk (row block (k-1) % S), 16 bytes per thread per access.
__global__ void gather_states(const DevOp* ops, int n, const char* ws, uint4* hk, uint4* hprev, int S,
                              size_t block16) {  // block16: B*H*2/16
  grid_dep_wait();
  grid_dep_launch();
  const DevOp op = ops[blockIdx.y];
  const int sidx = (op.k - 1) % S;
  const uint4* src_k = reinterpret_cast<const uint4*>(ws + (size_t)op.h_dst * 16);
  const uint4* src_p = reinterpret_cast<const uint4*>(ws + (size_t)op.h_src * 16);
  uint4* dk = hk + (size_t)sidx * block16;
  uint4* dp = hprev + (size_t)sidx * block16;
  for (size_t e = blockIdx.x * (size_t)blockDim.x + threadIdx.x; e < block16; e += (size_t)gridDim.x * blockDim.x) {
    if (hk) dk[e] = src_k[e];   // leaf batches have no stored h_k: leaf_forward writes it
    dp[e] = src_p[e];
  }
}

// The forward operations of a batch of leaves, after the batched GEMMs have produced their
// pre-activations z (row block (k-1) % S, gate columns 4 u + q): h_k = o tanh(f c_{k-1} + i g),
// written to the staging chunk for the readout and the weight gradients.  Same arithmetic as the
// epilogue of the forward run kernel; the gates themselves are redone by the backward kernel.
__global__ void leaf_forward(const DevOp* ops, int n, const char* ws, const float* z, __nv_bfloat16* hk, int S, int B,
                             int H, int64_t* counters) {
  grid_dep_wait();
  grid_dep_launch();
  const DevOp op = ops[blockIdx.y];
  const int sidx = (op.k - 1) % S;
  const size_t bh = (size_t)B * H;
  const float* cprev = reinterpret_cast<const float*>(ws + (size_t)op.c_src * 16);
  const float4* zs = reinterpret_cast<const float4*>(z + (size_t)sidx * bh * 4);
  __nv_bfloat16* out = hk + (size_t)sidx * bh;
  for (size_t e = blockIdx.x * (size_t)blockDim.x + threadIdx.x; e < bh; e += (size_t)gridDim.x * blockDim.x) {
    const float4 zz = zs[e];   // (b, u): columns 4 u .. 4 u + 3 of row b
    const float iv = sigmoid_fast(zz.x), fv = sigmoid_fast(zz.y), gv = tanh_fast(zz.z), ov = sigmoid_fast(zz.w);
    const float c = fmaf(fv, cprev[e], iv * gv);
    out[e] = __float2bfloat16_rn(ov * tanh_fast(c));
  }
  if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) counters[0] += n;
}

// y (float32, readout with bias) -> dy = 2 (y - target) / (B O) in bfloat16, and LOSS_PARTS
// partial sums of the squared error per step (each a fixed-order sum over a fixed slice).
__global__ void loss_dy(const DevOp* ops, const float* y, const float* targets, __nv_bfloat16* dy, float* loss_part,
                        int S, int B, int O) {
  __shared__ float red[256];
  grid_dep_wait();
  grid_dep_launch();
  const DevOp op = ops[blockIdx.y];
  const int sidx = (op.k - 1) % S;
  const size_t n = (size_t)B * O;
  const size_t per = (n + LOSS_PARTS - 1) / LOSS_PARTS;
  const size_t lo = blockIdx.x * per, hi = (lo + per < n) ? lo + per : n;
  const float* yp = y + (size_t)sidx * n;
  const float* tp = targets + (size_t)(op.k - 1) * n;
  __nv_bfloat16* dp = dy + (size_t)sidx * n;
  const float inv = 1.f / ((float)B * (float)O);
  float s = 0.f;
  for (size_t e = lo + threadIdx.x; e < hi; e += blockDim.x) {
    const float d = yp[e] - tp[e];
    dp[e] = __float2bfloat16_rn(2.f * d * inv);
    s = fmaf(d, d, s);
  }
  red[threadIdx.x] = s;
  __syncthreads();
  for (int w = 128; w > 0; w >>= 1) {
    if ((int)threadIdx.x < w) red[threadIdx.x] += red[threadIdx.x + w];
    __syncthreads();
  }
  if (threadIdx.x == 0) loss_part[sidx * LOSS_PARTS + blockIdx.x] = red[0] * inv;
}

// out[map(n)] += sum_r v[r][n]; perm_h > 0 maps column 4 u + q to q perm_h + u.  A block of
// 32 x 32 threads sums 64 columns: thread (x, g) takes the rows g, g + 32, ... of columns 2 x and
// 2 x + 1 into four running sums (row g + 32 i goes to sum i mod 4, so that four loads are in
// flight), adds them as (0 + 1) + (2 + 3), and the 32 partial sums of a column are added in the
// order g = 0 .. 31: fixed, whatever the plan.
__global__ void __launch_bounds__(1024) colsum_bf16(const __nv_bfloat16* v, int rows, int N, float* out, int perm_h) {
  __shared__ float2 part[32][33];
  grid_dep_wait();
  grid_dep_launch();
  const int n = (blockIdx.x * 32 + threadIdx.x) * 2, g = threadIdx.y;
  float2 acc[4];
#pragma unroll
  for (int j = 0; j < 4; ++j) acc[j] = make_float2(0.f, 0.f);
  if (n < N) {
    const bool pair = (N & 1) == 0;   // then column n + 1 exists and the two lie in one aligned word
    auto load = [&](int r) {
      const __nv_bfloat16* q = v + (size_t)r * N + n;
      if (pair) return __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(q));
      return make_float2(__bfloat162float(q[0]), n + 1 < N ? __bfloat162float(q[1]) : 0.f);
    };
    int r = g;
    for (; r + 96 < rows; r += 128) {
      float2 x[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) x[j] = load(r + 32 * j);
#pragma unroll
      for (int j = 0; j < 4; ++j) { acc[j].x += x[j].x; acc[j].y += x[j].y; }
    }
#pragma unroll
    for (int j = 0; j < 3; ++j)   // at most three rows are left
      if (r + 32 * j < rows) {
        const float2 x = load(r + 32 * j);
        acc[j].x += x.x; acc[j].y += x.y;
      }
  }
  part[g][threadIdx.x] = make_float2((acc[0].x + acc[1].x) + (acc[2].x + acc[3].x), (acc[0].y + acc[1].y) + (acc[2].y + acc[3].y));
  __syncthreads();
  if (g < 2 && n + g < N) {
    float tot = 0.f;
#pragma unroll
    for (int i = 0; i < 32; ++i) tot += g ? part[i][threadIdx.x].y : part[i][threadIdx.x].x;
    const int c = n + g;
    const int o = perm_h ? ((c & 3) * perm_h + (c >> 2)) : c;
    out[o] += tot;
  }
}

__global__ void finalize_tc(const float* loss_t, int64_t t, float* loss, int64_t* counters, int64_t peak_units,
                            const int* status) {
  grid_dep_wait();
  grid_dep_launch();
  float s = 0.f;
  for (int64_t i = threadIdx.x; i < t; i += 32) s += loss_t[i];
  for (int o = 16; o > 0; o >>= 1) s += __shfl_down_sync(0xffffffffu, s, o);
  if (threadIdx.x == 0) {
    *loss = s;
    counters[2] = peak_units;
    counters[3] = *status;
  }
}

__global__ void copy16_tc(uint4* dst, const uint4* src, size_t n) {
  grid_dep_wait();
  grid_dep_launch();
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x)
    dst[i] = src[i];
}

inline uint32_t off16(size_t byte_off) { return (uint32_t)(byte_off >> 4); }

// With MEBPTT_DEBUG set in the environment, failed CUDA calls are named on stderr.
inline bool cuda_ok(cudaError_t e, const char* what) {
  if (e == cudaSuccess) return true;
  if (env::debug()) fprintf(stderr, "mebptt: %s failed: %s\n", what, cudaGetErrorString(e));
  return false;
}

}  // namespace

// ------------------------------------------------------------------------------------------
// host: one training step
// ------------------------------------------------------------------------------------------
// A second stream and four events per device, created on first use and kept for the life of the
// process.  The side stream has lower priority than any stream a caller is likely to pass, so
// that the cooperative kernels of the recurrence get their SMs first and the GEMMs fill the rest.
constexpr int X_PIECES = 8;
struct SideStream {
  cudaStream_t stream = nullptr;
  cudaStream_t main = nullptr;                 // the step itself, at the most urgent priority
  cudaEvent_t fork = nullptr, join = nullptr;  // the caller's stream -> main, main -> the caller's stream
  cudaStream_t zx = nullptr;                   // input projections of the window after the one in use
  cudaEvent_t zx_free[2] = {nullptr, nullptr};   // copy b of the window buffer has no reader left (recorded on the step's stream)
  cudaEvent_t zx_ready[2] = {nullptr, nullptr};  // copy b holds its window (recorded on the zx stream)
  cudaEvent_t ready[2] = {nullptr, nullptr};   // stages of parity p are complete (recorded on the caller's stream)
  cudaEvent_t done[2] = {nullptr, nullptr};    // GEMMs reading parity p have finished (recorded on the side stream)
  cudaStream_t copy = nullptr;                 // host-to-device copies that overlap the forward pass
  cudaEvent_t copy_from = nullptr, copy_done = nullptr;
  cudaEvent_t x_ready[X_PIECES] = {};          // pieces of x (along time) have arrived
  cudaEvent_t t_ready[X_PIECES] = {};          // pieces of the targets have arrived (copied last piece first)
  bool ok = false;
};
SideStream* side_stream_for_current_device() {
  static std::mutex mu;
  static SideStream table[64];
  static bool tried[64] = {};
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  std::lock_guard<std::mutex> lock(mu);
  SideStream& t = table[dev];
  if (!tried[dev]) {
    tried[dev] = true;
    int lo = 0, hi = 0;
    cudaDeviceGetStreamPriorityRange(&lo, &hi);   // lo = numerically largest = least urgent
    bool ok = cudaStreamCreateWithPriority(&t.stream, cudaStreamNonBlocking, lo) == cudaSuccess &&
              cudaStreamCreateWithPriority(&t.main, cudaStreamNonBlocking, hi) == cudaSuccess &&
              cudaEventCreateWithFlags(&t.fork, cudaEventDisableTiming) == cudaSuccess &&
              cudaEventCreateWithFlags(&t.join, cudaEventDisableTiming) == cudaSuccess &&
              cudaStreamCreateWithPriority(&t.zx, cudaStreamNonBlocking, (lo + hi) / 2) == cudaSuccess;
    for (int i = 0; i < 2 && ok; ++i) {
      ok = cudaEventCreateWithFlags(&t.zx_free[i], cudaEventDisableTiming) == cudaSuccess &&
           cudaEventCreateWithFlags(&t.zx_ready[i], cudaEventDisableTiming) == cudaSuccess;
    }
    for (int i = 0; i < 2 && ok; ++i) {
      ok = cudaEventCreateWithFlags(&t.ready[i], cudaEventDisableTiming) == cudaSuccess &&
           cudaEventCreateWithFlags(&t.done[i], cudaEventDisableTiming) == cudaSuccess;
    }
    ok = ok && cudaStreamCreateWithFlags(&t.copy, cudaStreamNonBlocking) == cudaSuccess &&
         cudaEventCreateWithFlags(&t.copy_from, cudaEventDisableTiming) == cudaSuccess &&
         cudaEventCreateWithFlags(&t.copy_done, cudaEventDisableTiming) == cudaSuccess;
    for (int i = 0; i < X_PIECES && ok; ++i)
      ok = cudaEventCreateWithFlags(&t.x_ready[i], cudaEventDisableTiming) == cudaSuccess &&
           cudaEventCreateWithFlags(&t.t_ready[i], cudaEventDisableTiming) == cudaSuccess;
    if (!ok) cudaGetLastError();
    t.ok = ok;
  }
  return t.ok ? &t : nullptr;
}

// Event pairs around the launches of the persistent kernels, per device; filled only by steps
// that ask for it.
struct RunTimer {
  struct Span { cudaEvent_t e0, e1; int cls; int ops; };
  std::mutex mu;
  std::vector<Span> spans;
  std::vector<cudaEvent_t> pool;
  cudaEvent_t get() {
    if (!pool.empty()) { cudaEvent_t e = pool.back(); pool.pop_back(); return e; }
    cudaEvent_t e = nullptr;
    if (cudaEventCreate(&e) != cudaSuccess) { cudaGetLastError(); return nullptr; }
    return e;
  }
};
RunTimer* run_timer_for_current_device() {
  static RunTimer table[64];
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  return &table[dev];
}
// Records the start of a span on `s`; the returned index is closed by span_end.
int span_begin(RunTimer* rt, int cls, int ops, cudaStream_t s) {
  if (!rt) return -1;
  std::lock_guard<std::mutex> lock(rt->mu);
  RunTimer::Span sp{rt->get(), rt->get(), cls, ops};
  if (!sp.e0 || !sp.e1) return -1;
  cudaEventRecord(sp.e0, s);
  rt->spans.push_back(sp);
  return (int)rt->spans.size() - 1;
}
void span_end(RunTimer* rt, int idx, cudaStream_t s) {
  if (!rt || idx < 0) return;
  std::lock_guard<std::mutex> lock(rt->mu);
  cudaEventRecord(rt->spans[idx].e1, s);
}

int run_times(double* ms, int64_t* launches, int64_t* ops) {
  RunTimer* rt = run_timer_for_current_device();
  if (!rt || !ms || !launches || !ops) return MEBPTT_ERR_ARG;
  for (int c = 0; c < 2; ++c) { ms[c] = 0.0; launches[c] = 0; ops[c] = 0; }
  std::lock_guard<std::mutex> lock(rt->mu);
  int rc = MEBPTT_OK;
  for (const RunTimer::Span& sp : rt->spans) {
    float t = 0.f;
    if (cudaEventSynchronize(sp.e1) != cudaSuccess || cudaEventElapsedTime(&t, sp.e0, sp.e1) != cudaSuccess) {
      cudaGetLastError();
      rc = MEBPTT_ERR_CUDA;
    } else {
      ms[sp.cls] += t; launches[sp.cls] += 1; ops[sp.cls] += sp.ops;
    }
    rt->pool.push_back(sp.e0);
    rt->pool.push_back(sp.e1);
  }
  rt->spans.clear();
  return rc;
}

// Inputs that are still in host memory, copied on the library's copy stream beside the forward
// pass: x in X_PIECES pieces along the time axis (event x_ready[p] marks piece p), then the
// targets, likewise in pieces but from the last one to the first (event t_ready[p]): the backward
// pass starts at the end of the sequence and reaches the early targets long after they arrive.
// Ordered after everything already in `s`: the previous step on `s` may still read the destinations.
struct LateCopies {
  SideStream* side = nullptr;
  int x_pieces = 0;            // 0: x was not copied here
  int64_t steps_per_piece = 0;
  int t_pieces = 0;            // 0: the targets were not copied here
  int64_t t_steps_per_piece = 0;
  bool targets = false;
};
LateCopies start_late_copies(const StepPtrs& io, int64_t t, cudaStream_t s) {
  LateCopies lc;
  SideStream* side = side_stream_for_current_device();
  if (!side || (!io.x_host && !io.targets_host)) return lc;
  lc.side = side;
  cudaEventRecord(side->copy_from, s);
  cudaStreamWaitEvent(side->copy, side->copy_from, 0);
  if (io.x_host) {
    const size_t per_step = io.x_bytes / (size_t)t;
    lc.steps_per_piece = (t + X_PIECES - 1) / X_PIECES;
    lc.x_pieces = (int)((t + lc.steps_per_piece - 1) / lc.steps_per_piece);
    for (int p = 0; p < lc.x_pieces; ++p) {
      const int64_t lo = p * lc.steps_per_piece, hi = (lo + lc.steps_per_piece < t) ? lo + lc.steps_per_piece : t;
      cudaMemcpyAsync(const_cast<char*>(io.x) + (size_t)lo * per_step, (const char*)io.x_host + (size_t)lo * per_step,
                      (size_t)(hi - lo) * per_step, cudaMemcpyHostToDevice, side->copy);
      cudaEventRecord(side->x_ready[p], side->copy);
    }
  }
  if (io.targets_host) {
    const size_t per_step = io.targets_bytes / (size_t)t;
    lc.t_steps_per_piece = (t + X_PIECES - 1) / X_PIECES;
    lc.t_pieces = (int)((t + lc.t_steps_per_piece - 1) / lc.t_steps_per_piece);
    for (int p = lc.t_pieces - 1; p >= 0; --p) {
      const int64_t lo = p * lc.t_steps_per_piece, hi = (lo + lc.t_steps_per_piece < t) ? lo + lc.t_steps_per_piece : t;
      cudaMemcpyAsync(reinterpret_cast<char*>(const_cast<float*>(io.targets)) + (size_t)lo * per_step,
                      (const char*)io.targets_host + (size_t)lo * per_step, (size_t)(hi - lo) * per_step,
                      cudaMemcpyHostToDevice, side->copy);
      cudaEventRecord(side->t_ready[p], side->copy);
    }
    cudaEventRecord(side->copy_done, side->copy);
    lc.targets = true;
  }
  return lc;
}

// ------------------------------------------------------------------------------------------
// What a step needs besides the caller's pointers, prepared once and kept
// ------------------------------------------------------------------------------------------
// Everything here follows from the descriptor, the plan and the workspace address alone: the work
// items the tape is cut into, where each forward run finds its input projections, the tape as the
// kernels read it (in page-locked host memory, so that its upload is an asynchronous copy that
// does not hold up the calling thread), the kernel variants the device can keep resident and the
// tensor maps.  A step looks its set up in a small cache, most recently used first; freeing a
// plan drops the entries made for it.
struct Prepared {
  // key
  uint64_t plan_id = 0;
  int I = 0, H = 0, O = 0, B = 0;
  int64_t t = 0;
  bool want_dx = false;
  char* ws = nullptr;      // nullptr: host part only (no tensor maps)
  int device = -1;
  // host part
  std::vector<WorkItem> items;
  std::vector<int> zx_next;  // per item that opens a window: the item that opens the next one (-1: none)
  std::vector<int> zx_hi;  // per item: a forward run that projects its inputs anew does so up to this step (exclusive); 0: the window in place serves it
  DevOp* tape = nullptr;   // [2 nops]: the tape, then the compacted leaves of leaf batches
  size_t tape_entries = 0;
  bool pinned = false;
  // device part
  CUtensorMap tm_h, tm_w, tm_dz[2], tm_wt, tm_dz_b[2], tm_wt_c;
  int bwd_cs = 0, bwdc_smem = 0;   // cluster size of the backward kernel (0: one CTA per 8 columns, unclustered)
  int bwd_tb = 4;                  // its K tiles per barrier
  bool bwd_slab = false;           // its slice of dz by one copy per barrier instead of one per K tile
  bool bwd_grp = false;            // the backward kernel with groups of batch rows (then bwd_cs is its cluster size)
  int bwdg_smem = 0, bwdg_tb = 8, bwdg_ncg = 0;
  CUtensorMap tm_dz_g[2], tm_wt_g;
  int fwd_ncg = 0, fwd_smem = 0, fwd_bb = 0;
  bool fwd_slab = false;
  int rc = MEBPTT_OK;

  Prepared() = default;
  Prepared(const Prepared&) = delete;
  Prepared& operator=(const Prepared&) = delete;
  ~Prepared() {
    if (tape && pinned) cudaFreeHost(tape);
    else if (tape) free(tape);
  }
};

namespace {
std::mutex g_prep_mu;
std::vector<std::shared_ptr<Prepared>> g_prep;     // most recently used first
constexpr size_t kPrepCapacity = 8;
std::atomic<int64_t> g_prep_stats[3];               // sets built, sets reused, sets whose tape lies in page-locked memory

void build_host_part(Prepared& P, const Layout& y, const Plan* p, bool allow_pinned) {
  auto block_off = [&](int32_t loc) -> size_t {
    switch (loc) {
      case MEBPTT_LOC_INIT: return y.off_init;
      case MEBPTT_LOC_PING: return y.off_ping;
      case MEBPTT_LOC_PONG: return y.off_pong;
      case MEBPTT_LOC_CORE: return y.off_core;
      default: return y.off_arena + (size_t)loc * y.loc_bytes;
    }
  };
  const int S = y.S;
  const size_t nops = p->tape.size();
  P.items = work_items(p, S);
  // Input projections Zx: computed for the S steps from the start of a forward run on, unless the
  // buffer already holds them: recomputation sweeps keep returning to the same stored state, so one
  // projection serves many short runs.  (The values do not depend on how steps are batched.)  The
  // tape is known, so the window ends where the last run that will still find its steps in it ends
  // (the first forward run that does not fit in the S steps from the window's start on replaces it).
  P.zx_hi.assign(P.items.size(), 0);
  int zx_lo = 0, zx_hi = 0;
  for (size_t item = 0; item < P.items.size(); ++item) {
    const WorkItem& wi = P.items[item];
    if (wi.kind != WorkItem::FWD) continue;
    const int k0 = p->tape[wi.i].k, n = wi.n;
    if (k0 >= zx_lo && k0 + n <= zx_hi) continue;
    zx_lo = k0;
    const int cap = (int)((int64_t)k0 + S <= y.t + 1 ? k0 + S : y.t + 1);
    zx_hi = k0 + n;
    for (size_t j = item + 1; j < P.items.size(); ++j) {
      if (P.items[j].kind != WorkItem::FWD) continue;
      const int kj = p->tape[P.items[j].i].k, ej = kj + P.items[j].n;
      if (kj < k0 || ej > cap) break;
      if (ej > zx_hi) zx_hi = ej;
    }
    P.zx_hi[item] = zx_hi;
  }
  P.zx_next.assign(P.items.size(), -1);
  for (int item = (int)P.items.size() - 1, next = -1; item >= 0; --item)
    if (P.zx_hi[item]) { P.zx_next[item] = next; next = item; }
  // the tape as the kernels read it
  P.tape_entries = 2 * nops;
  const size_t bytes = (P.tape_entries ? P.tape_entries : 1) * sizeof(DevOp);
  void* mem = nullptr;
  if (allow_pinned && cudaHostAlloc(&mem, bytes, cudaHostAllocDefault) == cudaSuccess) {
    P.pinned = true;
  } else {
    if (allow_pinned) cudaGetLastError();
    mem = malloc(bytes);
  }
  P.tape = static_cast<DevOp*>(mem);
  if (!P.tape) { P.rc = MEBPTT_ERR_OOM; return; }
  memset(P.tape, 0, bytes);
  for (size_t i = 0; i < nops; ++i) {
    const mebptt_op& op = p->tape[i];
    DevOp d{};
    d.k = op.k;
    d.fmt = op.dst_fmt;
    if (op.kind == MEBPTT_OP_FWD) {
      const size_t src = block_off(op.src), dst = block_off(op.dst);
      d.h_src = off16(src); d.c_src = off16(src + y.hsz);
      d.h_dst = off16(dst); d.c_dst = off16(dst + y.hsz);
      d.gates = (op.dst_fmt != MEBPTT_FMT_HIDDEN) ? off16(dst + y.rec_gates) : 0;
      d.in_copy = (op.dst_fmt == MEBPTT_FMT_INTERNAL) ? off16(dst + y.rec_in) : 0;
    } else {
      const size_t rec = block_off(op.src);
      const size_t prev = (op.dst_fmt == MEBPTT_FMT_INTERNAL) ? rec + y.rec_in : block_off(op.aux);
      d.h_dst = off16(rec); d.c_dst = off16(rec + y.hsz);
      d.h_src = off16(prev); d.c_src = off16(prev + y.hsz);
      d.gates = off16(rec + y.rec_gates);
    }
    P.tape[i] = d;
  }
  for (const WorkItem& it : P.items) {
    if (it.kind != WorkItem::LEAF) continue;
    for (int j = 0; j < it.n; ++j) {
      const mebptt_op& f = p->tape[it.i + 2 * (size_t)j];   // the leaf's forward operation
      const size_t src = block_off(f.src);
      DevOp d{};
      d.k = f.k;
      d.h_src = off16(src); d.c_src = off16(src + y.hsz);   // state k-1, memorised
      P.tape[nops + it.i + (size_t)j] = d;
    }
  }
}

// Kernel variants and tensor maps for the workspace at `ws` on the current device.
void build_device_part(Prepared& P, const Layout& y, char* ws) {
  const int B = y.B, H = y.H, S = y.S, G = 4 * H;
  const int BM = 64;  // batch rows per MMA tile (B <= 64)
  const int ncta = H / NU;
  __nv_bfloat16* dz = reinterpret_cast<__nv_bfloat16*>(ws + y.off_dz);
  __nv_bfloat16* wp_hh = reinterpret_cast<__nv_bfloat16*>(ws + y.off_wp_hh);
  __nv_bfloat16* wpT_hh = reinterpret_cast<__nv_bfloat16*>(ws + y.off_wpT_hh);
  const int KBh = (H + 63) / 64;
  const int KB0 = fwd_first_part_blocks(H);       // 64-wide blocks of the recurrent contraction in its first part
  const int fwd_groups = B > FB ? 2 : 1;          // groups of CTAs that each own FB batch rows
  const int fwd_parts = KB0 < KBh ? 2 : 1;
  P.fwd_ncg = (H + FU - 1) / FU;                  // CTAs per group
  P.fwd_smem = (KBh * FG + fwd_parts * KB0 * FB) * 128 + 2 * FB * PART_LD * 4 + 1024;
  P.fwd_slab = false;                             // h_{k-1} by one copy per part instead of one per K tile
  P.fwd_bb = KB0;                                 // K tiles per barrier
  P.bwd_cs = 0; P.bwdc_smem = 0;
  {
    // function attributes belong to the device that is current
    const int big = 220 * 1024;  // the kernels also hold a few static barriers
    cudaFuncSetAttribute(fwd_run_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, big);
    cudaFuncSetAttribute(bwd_run_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, big);
  }
  // the whole workspace as rows of H bfloat16: any h block starts at a whole row
  const uint64_t rows = y.total / ((size_t)H * 2);
  bool ok = make_tmap_2d(&P.tm_h, ws, 2, (uint64_t)H, rows, (uint64_t)H * 2, 64, FB);
  ok = ok && make_tmap_2d(&P.tm_w, wp_hh, 2, (uint64_t)H, (uint64_t)G, (uint64_t)H * 2, 64, FG);
  if (ok && H % 64 == 0) {
    CUtensorMap blocked;
    if (make_tmap_blocks64(&blocked, ws, (uint64_t)H, rows, (uint64_t)H * 2, FB, (uint32_t)P.fwd_bb)) {
      P.tm_h = blocked;
      P.fwd_slab = true;
    }
  }
  for (int pb = 0; pb < 2; ++pb)
    ok = ok && make_tmap_2d(&P.tm_dz[pb], dz + (size_t)pb * S * B * G, 2, (uint64_t)G, (uint64_t)S * B, (uint64_t)G * 2, 64,
                            (uint32_t)BM);
  ok = ok && make_tmap_2d(&P.tm_wt, wpT_hh, 2, (uint64_t)G, (uint64_t)H, (uint64_t)G * 2, 64, NU);
  if (!ok) { P.rc = MEBPTT_ERR_UNSUPPORTED; return; }
  // the clustered backward kernel, if the device can keep enough clusters resident
  // (a switch in the environment can override the choice: env.hpp)
  const int force = env::bwd_cluster();
  for (int cs : {8, 4}) {
    if (force >= 0 && force != cs) continue;
    if (G % 64 != 0 || (G / 64) % cs != 0 || ncta % cs != 0 || (G / 64) / cs > 16) continue;
    const int kbs = (G / 64) / cs;
    const int tb = kbs > 8 ? 8 : 4;   // K tiles per barrier: at most four barriers, two where the slice is long
    const int smem = kbs * (NU * cs * 128) + ((kbs + tb - 1) / tb) * tb * BM * 128 + 2 * cs * BM * NU * 4 + 1024;
    if (smem > 220 * 1024) continue;
    const void* fn = cs == 8 ? (const void*)bwd_run_cluster_kernel<8> : (const void*)bwd_run_cluster_kernel<4>;
    cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(ncta); cfg.blockDim = dim3(192); cfg.dynamicSmemBytes = smem;
    cudaLaunchAttribute at1[1];
    at1[0].id = cudaLaunchAttributeClusterDimension;
    at1[0].val.clusterDim.x = cs; at1[0].val.clusterDim.y = 1; at1[0].val.clusterDim.z = 1;
    cfg.attrs = at1; cfg.numAttrs = 1;
    int nclusters = 0;
    if (cudaOccupancyMaxActiveClusters(&nclusters, fn, &cfg) != cudaSuccess) { cudaGetLastError(); continue; }
    if (nclusters * cs < ncta) continue;
    P.bwd_cs = cs; P.bwdc_smem = smem; P.bwd_tb = tb;
    break;
  }
  // the kernel with groups of batch rows, where the batch fills two groups and the driver takes a
  // map that sees the staging chunk as [columns / 64][rows][64]
  if (P.bwd_cs && force < 0 && !env::no_bwd_groups() && B > FB && B <= 2 * FB && H % (FU * GCS) == 0 &&
      (G / 64) % GCS == 0 && (G / 64) / GCS <= 16) {
    const int kbs = (G / 64) / GCS;
    const int tb = kbs > 8 ? 8 : 4;
    const int nq = (kbs + tb - 1) / tb;
    const int smem = kbs * (FU * GCS * 128) + nq * tb * FB * 128 + 2 * GCS * FU * RECV_LD * 4 + 1024;
    const int ncg = H / FU;
    bool g_ok = smem <= 220 * 1024;
    const void* fn = (const void*)bwd_run_group_kernel;
    if (g_ok) {
      cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
      cudaLaunchConfig_t cfg = {};
      cfg.gridDim = dim3(2 * ncg); cfg.blockDim = dim3(192); cfg.dynamicSmemBytes = smem;
      cudaLaunchAttribute at1[1];
      at1[0].id = cudaLaunchAttributeClusterDimension;
      at1[0].val.clusterDim.x = GCS; at1[0].val.clusterDim.y = 1; at1[0].val.clusterDim.z = 1;
      cfg.attrs = at1; cfg.numAttrs = 1;
      int nclusters = 0;
      if (cudaOccupancyMaxActiveClusters(&nclusters, fn, &cfg) != cudaSuccess) { cudaGetLastError(); g_ok = false; }
      else g_ok = nclusters * GCS >= 2 * ncg;
    }
    for (int pb = 0; pb < 2 && g_ok; ++pb)
      g_ok = make_tmap_blocks64(&P.tm_dz_g[pb], dz + (size_t)pb * S * B * G, (uint64_t)G, (uint64_t)S * B, (uint64_t)G * 2, FB,
                                (uint32_t)tb);
    g_ok = g_ok && make_tmap_2d(&P.tm_wt_g, wpT_hh, 2, (uint64_t)G, (uint64_t)H, (uint64_t)G * 2, 64, FU * GCS);
    if (g_ok) { P.bwd_grp = true; P.bwdg_smem = smem; P.bwdg_tb = tb; P.bwdg_ncg = ncg; }
  }
  if (P.bwd_cs) {
    // the staging chunk as [columns / 64][rows][64] if the driver takes such a map, else tile by tile
    P.bwd_slab = true;
    for (int pb = 0; pb < 2; ++pb)
      P.bwd_slab = P.bwd_slab && make_tmap_blocks64(&P.tm_dz_b[pb], dz + (size_t)pb * S * B * G, (uint64_t)G, (uint64_t)S * B,
                                                   (uint64_t)G * 2, 64, (uint32_t)P.bwd_tb);
    if (!P.bwd_slab)
      for (int pb = 0; pb < 2; ++pb)
        ok = ok && make_tmap_2d(&P.tm_dz_b[pb], dz + (size_t)pb * S * B * G, 2, (uint64_t)G, (uint64_t)S * B,
                                (uint64_t)G * 2, 64, 64);
    ok = ok && make_tmap_2d(&P.tm_wt_c, wpT_hh, 2, (uint64_t)G, (uint64_t)H, (uint64_t)G * 2, 64, (uint32_t)(NU * P.bwd_cs));
    if (!ok) { P.rc = MEBPTT_ERR_UNSUPPORTED; return; }
  }

}

// The set for (problem, plan, workspace, device): from the cache, or built and put there.  ws may
// be null: then only the host part is made (what counting launches needs, or a machine without a GPU).
std::shared_ptr<Prepared> prepare(const Layout& y, const Plan* p, bool want_dx, char* ws, bool allow_pinned) {
  int dev = -1;
  if (ws && cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); dev = -1; }
  {
    std::lock_guard<std::mutex> lock(g_prep_mu);
    for (size_t i = 0; i < g_prep.size(); ++i) {
      const Prepared& q = *g_prep[i];
      if (q.plan_id == p->id && q.I == y.I && q.H == y.H && q.O == y.O && q.B == y.B && q.t == y.t &&
          q.want_dx == want_dx && q.ws == ws && q.device == dev) {
        std::shared_ptr<Prepared> hit = g_prep[i];
        g_prep.erase(g_prep.begin() + (long)i);
        g_prep.insert(g_prep.begin(), hit);
        g_prep_stats[1]++;
        return hit;
      }
    }
  }
  // built outside the lock (two threads may build the same set at the same time: both are valid)
  std::shared_ptr<Prepared> P = std::make_shared<Prepared>();
  P->plan_id = p->id; P->I = y.I; P->H = y.H; P->O = y.O; P->B = y.B; P->t = y.t;
  P->want_dx = want_dx; P->ws = ws; P->device = dev;
  build_host_part(*P, y, p, allow_pinned && ws != nullptr);
  if (P->rc == MEBPTT_OK && ws) build_device_part(*P, y, ws);
  g_prep_stats[0]++;
  if (P->pinned) g_prep_stats[2]++;
  if (P->rc == MEBPTT_OK) {
    std::lock_guard<std::mutex> lock(g_prep_mu);
    g_prep.insert(g_prep.begin(), P);
    if (g_prep.size() > kPrepCapacity) g_prep.pop_back();
  }
  return P;
}
}  // namespace

namespace {
std::atomic<int> g_wait_fault{0};
}
int wait_fault_mask() { return g_wait_fault.load(); }
void set_wait_fault_mask(int mask) { g_wait_fault.store(mask); }

void forget_plan(uint64_t plan_id) {
  std::lock_guard<std::mutex> lock(g_prep_mu);
  for (size_t i = g_prep.size(); i-- > 0;)
    if (g_prep[i]->plan_id == plan_id) g_prep.erase(g_prep.begin() + (long)i);
}

void prepare_stats(int64_t* out) {
  for (int i = 0; i < 3; ++i) out[i] = g_prep_stats[i].load();
  std::lock_guard<std::mutex> lock(g_prep_mu);
  out[3] = (int64_t)g_prep.size();
}

int prepare_host(const Layout& y, const Plan* p, bool want_dx) { return prepare(y, p, want_dx, nullptr, false)->rc; }

int64_t run_step(const Layout& y, const Plan* p, const StepPtrs& io, bool want_dx, cudaStream_t caller, bool dry,
                 bool side_stream) {
  const int B = y.B, H = y.H, I = y.I, O = y.O, S = y.S, G = 4 * H, K = I + H;
  const int BM = 64;  // batch rows per MMA tile (B <= 64)
  const int ncta = H / NU;
  int64_t launches = 0;
  char* ws = io.ws;
  auto at = [&](size_t off) { return ws + off; };

  // ---- the prepared set of this (problem, plan, workspace) --------------------------------------
  const std::shared_ptr<Prepared> prep = prepare(y, p, want_dx, dry ? nullptr : ws, !io.pageable_tape);
  if (prep->rc != MEBPTT_OK) return prep->rc;
  const Prepared& P = *prep;
  const size_t nops = p->tape.size();
  const std::vector<WorkItem>& items = P.items;
  const DevOp* dops = reinterpret_cast<const DevOp*>(at(y.off_tape));
  uint32_t* sync = reinterpret_cast<uint32_t*>(at(y.off_sync));
  int* status = reinterpret_cast<int*>(at(y.off_status));
  float* loss_t = reinterpret_cast<float*>(at(y.off_loss_t));
  float* dh = reinterpret_cast<float*>(at(y.off_dh));
  float* dc = reinterpret_cast<float*>(at(y.off_dc));
  float* zx = reinterpret_cast<float*>(at(y.off_zx));
  __nv_bfloat16* dz = reinterpret_cast<__nv_bfloat16*>(at(y.off_dz));
  __nv_bfloat16* hprev = reinterpret_cast<__nv_bfloat16*>(at(y.off_hprev));
  __nv_bfloat16* hk = reinterpret_cast<__nv_bfloat16*>(at(y.off_hk));
  float* yv = reinterpret_cast<float*>(at(y.off_y));
  __nv_bfloat16* dyv = reinterpret_cast<__nv_bfloat16*>(at(y.off_dy));
  float* dha = reinterpret_cast<float*>(at(y.off_dha));
  float* loss_part = reinterpret_cast<float*>(at(y.off_loss_part));
  __nv_bfloat16* wp_ih = reinterpret_cast<__nv_bfloat16*>(at(y.off_wp_ih));
  __nv_bfloat16* wp_hh = reinterpret_cast<__nv_bfloat16*>(at(y.off_wp_hh));
  __nv_bfloat16* wpT_hh = reinterpret_cast<__nv_bfloat16*>(at(y.off_wpT_hh));
  __nv_bfloat16* wpT_ih = want_dx ? reinterpret_cast<__nv_bfloat16*>(at(y.off_wpT_ih)) : nullptr;
  float* bias_p = reinterpret_cast<float*>(at(y.off_bias_p));
  __nv_bfloat16* woutT = reinterpret_cast<__nv_bfloat16*>(at(y.off_woutT));

  const int KBh = (H + 63) / 64;
  const int KB0 = fwd_first_part_blocks(H);       // 64-wide blocks of the recurrent contraction in its first part
  const int fwd_groups = B > FB ? 2 : 1;          // groups of CTAs that each own FB batch rows
  const int bwd_smem = ((G + 63) / 64) * 1024 + NST * BM * 128 + 1024;
  const CUtensorMap &tm_h = P.tm_h, &tm_w = P.tm_w, &tm_wt = P.tm_wt, &tm_wt_c = P.tm_wt_c;
  const CUtensorMap* tm_dz = P.tm_dz;
  const CUtensorMap* tm_dz_b = P.tm_dz_b;
  const int bwd_cs = P.bwd_cs, bwdc_smem = P.bwdc_smem, fwd_ncg = P.fwd_ncg, fwd_smem = P.fwd_smem, fwd_bb = P.fwd_bb;
  const bool fwd_slab = P.fwd_slab;
  // On request (a switch in the environment) the step runs on a stream of the library's, of the most
  // urgent priority, ordered after what the caller's stream holds and joined to it at the end: the
  // caller's stream is of the least urgent priority as a rule, like the stream of the weight-gradient
  // GEMMs, whose grids then take free SMs as readily as the kernels of the recurrence do.  Measured
  // at config 3: 0.46 ms faster at MSM m = 100, 0.4 to 0.7 ms slower at m = 10, m = 32 and with full
  // memory (the gradient GEMMs fall behind and the step ends waiting for them).  Off by default.
  SideStream* side = (!dry && side_stream) ? side_stream_for_current_device() : nullptr;
  cudaStream_t s = caller;
  if (side && env::priority()) {
    cudaEventRecord(side->fork, caller);
    cudaStreamWaitEvent(side->main, side->fork, 0);
    s = side->main;
  }
  if (!dry) {
    cudaMemsetAsync(dh, 0, (size_t)B * H * 4, s);
    cudaMemsetAsync(dc, 0, (size_t)B * H * 4, s);
    cudaMemsetAsync(io.dW, 0, (size_t)G * K * 4, s);
    cudaMemsetAsync(io.db, 0, (size_t)G * 4, s);
    cudaMemsetAsync(io.dW_out, 0, (size_t)O * H * 4, s);
    cudaMemsetAsync(io.db_out, 0, (size_t)O * 4, s);
    cudaMemsetAsync(io.counters, 0, 8 * sizeof(int64_t), s);
    cudaMemsetAsync(sync, 0, y.n_sync * 4, s);
    cudaMemsetAsync(status, 0, 256, s);
    // (from page-locked memory: an asynchronous copy proper; from pageable memory, which only the
    // allocation-free entry point uses, the call may wait for the stream to reach the copy)
    cudaMemcpyAsync(at(y.off_tape), P.tape, P.tape_entries * sizeof(DevOp), cudaMemcpyHostToDevice, s);
    launch_pdl((I % 8 == 0 && H % 8 == 0 && O % 8 == 0) ? pack_weights : pack_weights_scalar, dim3(592), dim3(256), 0, s,
               reinterpret_cast<const __nv_bfloat16*>(io.W), io.b, reinterpret_cast<const __nv_bfloat16*>(io.W_out), I, H, O,
               wp_ih, wp_hh, wpT_hh, wpT_ih, bias_p, woutT);
    // Peek of the initial state: the caller's (h0, c0) as a hidden block inside the workspace
    launch_pdl(copy16_tc, dim3(64), dim3(256), 0, s, reinterpret_cast<uint4*>(at(y.off_init)),
               reinterpret_cast<const uint4*>(io.h0), (size_t)B * H * 2 / 16);
    launch_pdl(copy16_tc, dim3(64), dim3(256), 0, s, reinterpret_cast<uint4*>(at(y.off_init + y.hsz)),
               reinterpret_cast<const uint4*>(io.c0), (size_t)B * H * 4 / 16);
  }
  launches += 3;
  // The targets, if they are still on the host: requested after every other host-to-device copy of
  // this step (the copy engine serves requests in order), on a stream of their own.
  LateCopies late;
  if (!dry && (io.targets_host || io.x_host)) {
    late = start_late_copies(io, y.t, s);
    if (io.x_host && !late.x_pieces)
      cudaMemcpyAsync(const_cast<char*>(io.x), io.x_host, io.x_bytes, cudaMemcpyHostToDevice, s);
    if (io.targets_host && !late.targets)
      cudaMemcpyAsync(const_cast<float*>(io.targets), io.targets_host, io.targets_bytes, cudaMemcpyHostToDevice, s);
  }
  int x_waited = 0, x_waited_zx = 0;   // pieces of x the step's stream (the zx stream) has already waited for
  auto need_x_on = [&](cudaStream_t st, int& waited, int64_t steps) {   // time steps [0, steps) of x are about to be read on `st`
    while (waited < late.x_pieces && (int64_t)waited * late.steps_per_piece < steps)
      cudaStreamWaitEvent(st, late.side->x_ready[waited++], 0);
  };
  auto need_x = [&](int64_t steps) { need_x_on(s, x_waited, steps); };

  int t_waited = 0;   // pieces of the targets, counted from the last, the caller's stream has waited for
  auto need_targets = [&](int64_t k_lo) {   // the targets of time steps k_lo .. t are about to be read on `s`
    if (!late.t_pieces) return;
    const int first_piece = (int)((k_lo - 1) / late.t_steps_per_piece);
    while (t_waited < late.t_pieces - first_piece) {
      cudaStreamWaitEvent(s, late.side->t_ready[late.t_pieces - 1 - t_waited], 0);
      ++t_waited;
    }
  };

  int launch_id = 0;
  int rc = MEBPTT_OK;
  const int fault = wait_fault_mask();   // testing aid, 0 outside the tests of the bounded waits
  if (!dry && !cuda_ok(cudaGetLastError(), "set-up (memsets, tape upload, weight packing)")) rc = MEBPTT_ERR_CUDA;
  auto gemm_on = [&](cudaStream_t st, const void* A, int64_t lda, bool amn, const void* Bm, int64_t ldb, bool bmn,
                     GemmOut out, int M, int N, int Kc) {
    ++launches;
    if (dry || rc != MEBPTT_OK) return;
    // on the side stream a kernel that is resident early only takes room from the one that runs
    rc = gemm_bf16(A, lda, amn, Bm, ldb, bmn, out, M, N, Kc, status, st, st == s);
    if (rc != MEBPTT_OK) cuda_ok(cudaErrorUnknown, "batched contraction");
  };
  auto gemm = [&](const void* A, int64_t lda, bool amn, const void* Bm, int64_t ldb, bool bmn, GemmOut out, int M,
                  int N, int Kc) { gemm_on(s, A, lda, amn, Bm, ldb, bmn, out, M, N, Kc); };
  bool side_busy[2] = {false, false};   // GEMMs reading the stages of this parity were put on the side stream

  RunTimer* timer = (!dry && io.time_runs) ? run_timer_for_current_device() : nullptr;
  bool targets_waited = false;
  int zx_lo = 0, zx_hi = 0;   // time steps [zx_lo, zx_hi) whose input projections the Zx buffer holds
  float* zleaf = reinterpret_cast<float*>(at(y.off_zleaf));
  const bool zx_ahead = side && !env::no_zx_ahead();
  int zx_w = -1;          // windows opened so far, less one
  float* zx_cur = zx;     // the copy of the buffer that holds the window in use
  auto project_window = [&](size_t it, int w) {
    const int k0 = p->tape[items[it].i].k, hi = P.zx_hi[it];
    cudaEventRecord(side->zx_free[w & 1], s);
    cudaStreamWaitEvent(side->zx, side->zx_free[w & 1], 0);
    need_x_on(side->zx, x_waited_zx, hi - 1);
    const __nv_bfloat16* xk = reinterpret_cast<const __nv_bfloat16*>(io.x) + (size_t)(k0 - 1) * B * I;
    gemm_on(side->zx, xk, I, false, wp_ih, I, false,
            GemmOut{GemmOut::STORE_F32, zx + (size_t)(w & 1) * S * B * G, G, bias_p, 0}, (hi - k0) * B, G, I);
    cudaEventRecord(side->zx_ready[w & 1], side->zx);
  };
  for (size_t item = 0; item < items.size() && rc == MEBPTT_OK; ++item) {
    const WorkItem& wi = items[item];
    const size_t i = wi.i;
    const mebptt_op& first = p->tape[i];
    if (wi.kind == WorkItem::FWD) {
      // a forward run: consecutive operations k, k+1, ... each starting from the state the
      // previous one wrote; at most S of them per launch
      const int n = wi.n;
      // input projections Zx, unless the window in place holds those of this run
      const int k0 = first.k;
      if (P.zx_hi[item]) {
        zx_lo = k0;
        zx_hi = P.zx_hi[item];
        if (!zx_ahead) {
          const __nv_bfloat16* xk = reinterpret_cast<const __nv_bfloat16*>(io.x) + (size_t)(k0 - 1) * B * I;
          need_x(zx_hi - 1);
          gemm(xk, I, false, wp_ih, I, false, GemmOut{GemmOut::STORE_F32, zx, G, bias_p, 0}, (zx_hi - zx_lo) * B, G, I);
        } else {
          // Windows alternate between the two copies of the buffer.  The projections of a window
          // depend on x alone: those of the next window are put on a stream of their own as soon
          // as its copy has no reader left (every run of the window before this one is in the
          // step's stream by now), so that they run beside this window's runs and what follows
          // them, on the SMs the persistent kernels leave free.
          ++zx_w;
          if (zx_w == 0) project_window(item, 0);
          cudaStreamWaitEvent(s, side->zx_ready[zx_w & 1], 0);
          if (P.zx_next[item] >= 0) project_window((size_t)P.zx_next[item], zx_w + 1);
          zx_cur = zx + (size_t)(zx_w & 1) * S * B * G;
        }
      }
      ++launches;
      if (!dry && rc == MEBPTT_OK) {
        FwdRunArgs a{dops + i, n, ws, zx_cur + (size_t)(k0 - zx_lo) * B * G, sync + (size_t)launch_id * 2 * SYNC_STRIDE, status,
                     io.counters, B, H, fwd_ncg, fwd_bb, fwd_slab ? 1 : 0,
                     (uint32_t)fwd_ncg + ((fault & 1) ? 1u : 0u), (fault & 1) ? fault_poll_limit : (kSpinLimit >> 1),
                     off16(y.plane), off16(y.hsz)};
        void* args[] = {(void*)&tm_h, (void*)&tm_w, (void*)&a};
        const void* fn = (const void*)fwd_run_kernel;
        const int span = span_begin(timer, 0, n, s);
        if (!cuda_ok(launch_coop(fn, fwd_groups * fwd_ncg, 192, fwd_smem, s, args, 1), "forward run launch"))
          rc = MEBPTT_ERR_CUDA;
        span_end(timer, span, s);
      }
      ++launch_id;
    } else {
      // a backward run: consecutive operations k, k-1, ... inside one chunk of S time steps --
      // or a batch of leaves, whose forward operations are done here as well, all at once
      const bool leaf = wi.kind == WorkItem::LEAF;
      const DevOp* bops = leaf ? dops + nops + i : dops + i;
      if (!targets_waited) {
        need_x(y.t);                                  // leaves and weight gradients read x anywhere
        targets_waited = true;
      }
      const int chunk = (first.k - 1) / S;
      const int pb = chunk & 1;   // which copy of the stages this chunk uses
      const int n = wi.n;
      const int k_hi = first.k, k_lo = k_hi - n + 1;
      const int s_lo = (k_lo - 1) % S;
      need_targets(k_lo);   // the targets of steps k_lo .. t (backward steps come in descending order)
      const size_t SB = (size_t)S * B;
      __nv_bfloat16* dz_c = dz + (size_t)pb * SB * G;
      __nv_bfloat16* hprev_c = hprev + (size_t)pb * SB * H;
      __nv_bfloat16* hk_c = hk + (size_t)pb * SB * H;
      __nv_bfloat16* dy_c = dyv + (size_t)pb * SB * O;
      if (side && side_busy[pb]) {
        // these stages were last read by GEMMs on the side stream (two chunks ago): wait for them
        cudaStreamWaitEvent(s, side->done[pb], 0);
        side_busy[pb] = false;
      }
      launches += 2;   // gather_states and the backward run itself
      if (!dry && rc == MEBPTT_OK) {
        const size_t block16 = (size_t)B * H * 2 / 16;
        launch_pdl(gather_states, dim3(16, n), dim3(256), 0, s, bops, n, ws,
                   leaf ? nullptr : reinterpret_cast<uint4*>(hk_c), reinterpret_cast<uint4*>(hprev_c), S, block16);
      }
      if (leaf) {
        // z_k = W_ih x_k + b + W_hh h_{k-1} for the n leaves at once (their h_{k-1} are all
        // memorised), then h_k; the gates are redone inside the backward kernel
        const __nv_bfloat16* xk = reinterpret_cast<const __nv_bfloat16*>(io.x) + (size_t)(k_lo - 1) * B * I;
        gemm(xk, I, false, wp_ih, I, false,
             GemmOut{GemmOut::STORE_F32, zleaf + (size_t)s_lo * B * G, G, bias_p, 0}, n * B, G, I);
        // the recurrent part in the two parts the forward kernels sum it in, in their order
        const int k_first = KB0 < KBh ? 64 * KB0 : H;
        gemm(hprev_c + (size_t)s_lo * B * H, H, false, wp_hh, H, false,
             GemmOut{GemmOut::ACCUM_F32, zleaf + (size_t)s_lo * B * G, G, nullptr, 0}, n * B, G, k_first);
        if (k_first < H)
          gemm(hprev_c + (size_t)s_lo * B * H + k_first, H, false, wp_hh + k_first, H, false,
               GemmOut{GemmOut::ACCUM_F32, zleaf + (size_t)s_lo * B * G, G, nullptr, 0}, n * B, G, H - k_first);
        ++launches;
        if (!dry && rc == MEBPTT_OK)
          launch_pdl(leaf_forward, dim3(32, n), dim3(256), 0, s, bops, n, ws, zleaf, hk_c, S, B, H, io.counters);
      }
      // readout of the n steps at once, loss terms and dy, then the gradient entering h_k
      const bool fused_loss = loss_fused(B, O);
      const int parts = loss_parts_per_step(B, O);
      if (fused_loss) {
        GemmOut o{GemmOut::LOSS_DY, dy_c + (size_t)s_lo * B * O, O, io.b_out, 0};
        o.target = io.targets + (size_t)(k_lo - 1) * B * O;
        o.loss_part = loss_part + (size_t)s_lo * parts;
        o.parts = (O + 31) / 32;
        o.scale = 1.f / ((float)B * (float)O);
        gemm(hk_c + (size_t)s_lo * B * H, H, false, io.W_out, H, false, o, n * B, O, H);
      } else {
        gemm(hk_c + (size_t)s_lo * B * H, H, false, io.W_out, H, false,
             GemmOut{GemmOut::STORE_F32, yv + (size_t)s_lo * B * O, O, io.b_out, 0}, n * B, O, H);
        ++launches;
        if (!dry && rc == MEBPTT_OK)
          launch_pdl(loss_dy, dim3(LOSS_PARTS, n), dim3(256), 0, s, bops, yv, io.targets, dy_c, loss_part, S, B, O);
      }
      gemm(dy_c + (size_t)s_lo * B * O, O, false, woutT, O, false,
           GemmOut{GemmOut::STORE_F32, dha + (size_t)s_lo * B * H, H, nullptr, 0}, n * B, H, O);
      if (!dry && rc == MEBPTT_OK) {
        const bool grouped = P.bwd_grp;
        BwdRunArgs a{bops, n, ws, dha, dz_c, dh, dc, loss_part, loss_t, sync + (size_t)launch_id * 2 * SYNC_STRIDE, status,
                     io.counters, B, H, S, off16(y.plane), off16(y.hsz), leaf ? zleaf : nullptr, parts,
                     grouped ? P.bwdg_tb : P.bwd_tb, (grouped || P.bwd_slab) ? 1 : 0,
                     (uint32_t)(grouped ? P.bwdg_ncg : ncta) + ((fault & 2) ? 1u : 0u),
                     (fault & 2) ? fault_poll_limit : (kSpinLimit >> 1)};
        void* args[] = {(void*)(grouped ? &P.tm_dz_g[pb] : bwd_cs ? &tm_dz_b[pb] : &tm_dz[pb]),
                        (void*)(grouped ? &P.tm_wt_g : bwd_cs ? &tm_wt_c : &tm_wt), (void*)&a};
        const int span = span_begin(timer, 1, n, s);
        if (grouped) {
          if (!cuda_ok(launch_coop((const void*)bwd_run_group_kernel, 2 * P.bwdg_ncg, 192, P.bwdg_smem, s, args, GCS, false),
                       "backward run launch (groups of batch rows)"))
            rc = MEBPTT_ERR_CUDA;
        } else if (bwd_cs) {
          const void* fn = bwd_cs == 8 ? (const void*)bwd_run_cluster_kernel<8> : (const void*)bwd_run_cluster_kernel<4>;
          // launched in plain stream order: early residency of a clustered grid measured no gain
          if (!cuda_ok(launch_coop(fn, ncta, 192, bwdc_smem, s, args, bwd_cs, false), "backward run launch (clusters)"))
            rc = MEBPTT_ERR_CUDA;
        } else {
          const void* fn = (const void*)bwd_run_kernel<64>;
          if (!cuda_ok(launch_coop(fn, ncta, 128, bwd_smem, s, args, 1), "backward run launch")) rc = MEBPTT_ERR_CUDA;
        }
        span_end(timer, span, s);
      }
      ++launch_id;
      if (k_lo == chunk * S + 1) {
        // the chunk is complete: its weight gradients, summed over (s, b) in ascending order.
        // They depend on nothing that follows, so they go to the side stream (in order: chunk c
        // is accumulated before chunk c - 1) while the caller's stream moves on to the next chunk.
        cudaStream_t gs = s;
        if (side) {
          cudaEventRecord(side->ready[pb], s);
          cudaStreamWaitEvent(side->stream, side->ready[pb], 0);
          gs = side->stream;
        }
        const int steps = (int)((int64_t)(chunk + 1) * S <= y.t ? S : y.t - (int64_t)chunk * S);
        const int R = steps * B;
        const __nv_bfloat16* xc = reinterpret_cast<const __nv_bfloat16*>(io.x) + (size_t)chunk * S * B * I;
        gemm_on(gs, dz_c, G, true, xc, I, true, GemmOut{GemmOut::ACCUM_F32, io.dW, K, nullptr, H}, G, I, R);
        gemm_on(gs, dz_c, G, true, hprev_c, H, true, GemmOut{GemmOut::ACCUM_F32, io.dW + I, K, nullptr, H}, G, H, R);
        gemm_on(gs, dy_c, O, true, hk_c, H, true, GemmOut{GemmOut::ACCUM_F32, io.dW_out, H, nullptr, 0}, O, H, R);
        launches += 2;
        if (!dry && rc == MEBPTT_OK) {
          launch_on(gs == s, colsum_bf16, dim3((G + 63) / 64), dim3(32, 32), 0, gs, dz_c, R, G, io.db, H);
          launch_on(gs == s, colsum_bf16, dim3((O + 63) / 64), dim3(32, 32), 0, gs, dy_c, R, O, io.db_out, 0);
        }
        if (want_dx)
          gemm_on(gs, dz_c, G, false, wpT_ih, G, false,
                  GemmOut{GemmOut::STORE_F32, io.dx + (size_t)chunk * S * B * I, I, nullptr, 0}, R, I, G);
        if (side) {
          cudaEventRecord(side->done[pb], side->stream);
          side_busy[pb] = true;
        }
      }
    }
  }
  // everything the side stream did belongs to this call: join it before the last kernel
  if (side)
    for (int pb = 0; pb < 2; ++pb)
      if (side_busy[pb]) cudaStreamWaitEvent(s, side->done[pb], 0);
  ++launches;
  if (!dry && rc == MEBPTT_OK) {
    launch_pdl(finalize_tc, dim3(1), dim3(32), 0, s, loss_t, (int64_t)y.t, io.loss, io.counters, (int64_t)p->peak_units, status);
    if (!cuda_ok(cudaGetLastError(), "training step (last error)")) rc = MEBPTT_ERR_CUDA;
  }
  if (s != caller) {
    cudaEventRecord(side->join, s);
    cudaStreamWaitEvent(caller, side->join, 0);
  }
  if (dry) return launches;
  return rc;
}

}  // namespace tc
}  // namespace mebptt
