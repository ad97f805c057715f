// Step-by-step LSTM operations for float32 storage with every contraction on the tensor cores
// (MEBPTT_TF32).
//
// A float32 value v is split into two bfloat16 numbers, hi = bf16(v) and mid = bf16(v - hi), which
// together carry 16 bits of mantissa.  A product of two such values is taken as
//     a b  ~=  a_hi b_hi + a_hi b_mid + a_mid b_hi
// (the dropped term is 2^-18 relative), accumulated in float32: better than a tf32 product, at
// three bfloat16 MMAs.  The three terms are one contraction over a tripled index: the left
// operand is laid out [hi | hi | mid] along K and the right operand [hi | mid | hi], so the
// bfloat16 GEMM is used as it is.  Weights are split once per training step, activations and
// gradients where they are produced.
//
// Operations (per layer), with K = I + H, G = 4H:
//   forward    a3 = split([in ; h_prev]) ; z = a3 W3^T + b ; gates, c, h from z
//   readout    h3 = split(h) ; y = h3 Wout3^T + b_out with loss and dy (float32) in the epilogue ;
//              dy3 = split(dy) ; dha = dy3 WoutMN3
//   backward   dz3 from the stored gates ; d_in = dz3 WMN3
//   per chunk  dW += dz^T [in ; h_prev], dW_out += dy^T h from the staged halves: three GEMMs per
//              product (hi hi, hi mid, mid hi); db += sum of dz, db_out += sum of dy, as hi + mid
// All sums run in a fixed order and nothing depends on the plan: results are bit-identical across
// plans.
#include "kernels.hpp"
#include "launch.hpp"
#include "sm100.cuh"
#include "tc.hpp"

#include <cuda_bf16.h>
#include <cuda_runtime.h>

namespace mebptt {
namespace stepwise3 {

namespace {

using tc::GemmOut;
using tc::gemm_bf16;
typedef __nv_bfloat16 bf16;

__device__ __forceinline__ float sigmoidf_(float a) { return 1.0f / (1.0f + expf(-a)); }
__device__ __forceinline__ void split2(float v, bf16& hi, bf16& mid) {
  hi = __float2bfloat16_rn(v);
  mid = __float2bfloat16_rn(v - __bfloat162float(hi));
}

inline int ew_blocks(size_t n) { return (int)((n + 255) / 256 > 1184 ? 1184 : (n + 255) / 256); }

// out [R][3C] = [hi | mid | hi] of W [R][C]: the right operand of a contraction over columns.
__global__ void pack3_cols(const float* W, int R, int C, bf16* out) {
  sm100::grid_dep_wait();
  sm100::grid_dep_launch();
  const size_t n = (size_t)R * C;
  for (size_t e = blockIdx.x * (size_t)blockDim.x + threadIdx.x; e < n; e += (size_t)gridDim.x * blockDim.x) {
    const size_t r = e / C, c = e % C;
    bf16 hi, mid;
    split2(W[e], hi, mid);
    bf16* o = out + r * 3 * (size_t)C + c;
    o[0] = hi; o[C] = mid; o[2 * (size_t)C] = hi;
  }
}
// out [3R][C] = [hi ; mid ; hi] of W [R][C]: the right operand of a contraction over rows.
__global__ void pack3_rows(const float* W, int R, int C, bf16* out) {
  sm100::grid_dep_wait();
  sm100::grid_dep_launch();
  const size_t n = (size_t)R * C;
  for (size_t e = blockIdx.x * (size_t)blockDim.x + threadIdx.x; e < n; e += (size_t)gridDim.x * blockDim.x) {
    bf16 hi, mid;
    split2(W[e], hi, mid);
    out[e] = hi; out[n + e] = mid; out[2 * n + e] = hi;
  }
}
// out [B][3 (Ca + Cb)] = [hi | hi | mid] of the rows [a[b] ; b_[b]] (b_ may be NULL with Cb = 0):
// the left operand of a contraction over columns.
__global__ void split_a3(const float* a, int Ca, const float* b_, int Cb, int B, bf16* out) {
  sm100::grid_dep_wait();
  sm100::grid_dep_launch();
  const int C = Ca + Cb;
  const size_t n = (size_t)B * C;
  for (size_t e = blockIdx.x * (size_t)blockDim.x + threadIdx.x; e < n; e += (size_t)gridDim.x * blockDim.x) {
    const size_t r = e / C;
    const int c = (int)(e % C);
    const float v = c < Ca ? a[r * Ca + c] : b_[r * Cb + (c - Ca)];
    bf16 hi, mid;
    split2(v, hi, mid);
    bf16* o = out + r * 3 * (size_t)C + c;
    o[0] = hi; o[C] = hi; o[2 * (size_t)C] = mid;
  }
}

// The same split for up to 64 row blocks of [B][C] that lie apart (blockIdx.y picks the block);
// block a goes to rows a B .. of `out`.
struct RunPtrs { const float* p[64]; };
__global__ void split_blocks3(RunPtrs src, int C, int B, bf16* out) {
  sm100::grid_dep_wait();
  sm100::grid_dep_launch();
  const float* a = src.p[blockIdx.y];
  bf16* dst = out + (size_t)blockIdx.y * B * 3 * C;
  const size_t n = (size_t)B * C;
  for (size_t e = blockIdx.x * (size_t)blockDim.x + threadIdx.x; e < n; e += (size_t)gridDim.x * blockDim.x) {
    const size_t r = e / C;
    const int c = (int)(e % C);
    bf16 hi, mid;
    split2(a[e], hi, mid);
    bf16* o = dst + r * 3 * (size_t)C + c;
    o[0] = hi; o[C] = hi; o[2 * (size_t)C] = mid;
  }
}

// a3_next (optional): the left operand [B][3K] of the next step of a run, whose h columns
// (I .. I + H - 1 of each third) receive the halves of h_k here instead of from a split kernel.
// Left operands of a run of n forward operations: out[j] = [B][3 (I + H)] (blockIdx.y = j) gets the
// halves of the layer input of step j in its input columns, and out[0] those of h0 (the h of the
// state the run starts from) in its h columns; the h columns of the later steps are filled by the
// cell kernel of the step before.
__global__ void split_run_inputs(const float* in, int64_t in_step_stride, int I, const float* h0, int H, int B, bf16* out) {
  sm100::grid_dep_wait();
  sm100::grid_dep_launch();
  const int j = blockIdx.y;
  const size_t K = (size_t)I + H;
  bf16* dst = out + (size_t)j * B * 3 * K;
  const float* src = in + (size_t)j * in_step_stride;
  const size_t n = (size_t)B * (j == 0 ? K : (size_t)I);
  const size_t C = j == 0 ? K : (size_t)I;
  for (size_t e = blockIdx.x * (size_t)blockDim.x + threadIdx.x; e < n; e += (size_t)gridDim.x * blockDim.x) {
    const size_t r = e / C;
    const size_t c = e % C;
    const float v = c < (size_t)I ? src[r * I + c] : h0[r * H + (c - I)];
    bf16 hi, mid;
    split2(v, hi, mid);
    bf16* o = dst + r * 3 * K + c;
    o[0] = hi; o[K] = hi; o[2 * K] = mid;
  }
}

// z holds the contraction without the bias, or, if it was split along K, zp says where its parts
// lie (they are added here); bias [4H] is added last.
__global__ void cell_fwd(const float* z, const float* c_prev, const float* h_prev, float* h_out, float* c_out,
                         float* gates, size_t plane, float* h_in_copy, float* c_in_copy, int B, int H,
                         int64_t* counters, bf16* a3_next, int I, const float* bias, const tc::SplitParts zp) {
  sm100::grid_dep_wait();
  sm100::grid_dep_launch();
  const size_t n = (size_t)B * H;
  for (size_t e = blockIdx.x * (size_t)blockDim.x + threadIdx.x; e < n; e += (size_t)gridDim.x * blockDim.x) {
    const int b = (int)(e / H), j = (int)(e % H);
    float zi, zf, zg, zo;
    if (zp.splits) {
      zi = tc::split_parts_sum(zp, b, j);         zf = tc::split_parts_sum(zp, b, H + j);
      zg = tc::split_parts_sum(zp, b, 2 * H + j); zo = tc::split_parts_sum(zp, b, 3 * H + j);
    } else {
      const float* row = z + (size_t)b * 4 * H;
      zi = row[j]; zf = row[H + j]; zg = row[2 * H + j]; zo = row[3 * H + j];
    }
    const float gi = sigmoidf_(zi + bias[j]), gf = sigmoidf_(zf + bias[H + j]);
    const float gg = tanhf(zg + bias[2 * H + j]), go = sigmoidf_(zo + bias[3 * H + j]);
    const float cp = c_prev[e];
    const float c = fmaf(gf, cp, gi * gg);
    c_out[e] = c;
    const float hv = go * tanhf(c);
    h_out[e] = hv;
    if (a3_next) {
      const size_t K = (size_t)I + H;
      bf16 hi, mid;
      split2(hv, hi, mid);
      bf16* o = a3_next + (size_t)b * 3 * K + I + j;
      o[0] = hi; o[K] = hi; o[2 * K] = mid;
    }
    if (gates) { gates[e] = gi; gates[plane + e] = gf; gates[2 * plane + e] = gg; gates[3 * plane + e] = go; }
    if (h_in_copy) { h_in_copy[e] = h_prev[e]; c_in_copy[e] = cp; }
  }
  if (counters && blockIdx.x == 0 && threadIdx.x == 0) counters[0] += 1;
}

// Gate derivatives: dz [B][4H] float32 (for db), dz3 rows [hi | hi | mid] in the stage (left operand
// of dz W and of the chunk's dW), and the halves [hi | mid] of this step's layer input and h_{k-1}.
__global__ void gate_bwd(const float* dha, const float* dh_rec, float* dc_rec, const float* gates, size_t plane,
                         const float* c_t, const float* c_prev, float* dz, bf16* dz3, int B, int H, int64_t* counters,
                         const float* in, int I, bf16* st_in2, const float* hp, bf16* st_hp2,
                         const tc::SplitParts dh_parts) {
  sm100::grid_dep_wait();
  sm100::grid_dep_launch();
  const size_t n = (size_t)B * H;
  const size_t G = 4 * (size_t)H;
  for (size_t e = blockIdx.x * (size_t)blockDim.x + threadIdx.x; e < n; e += (size_t)gridDim.x * blockDim.x) {
    const int b = (int)(e / H), j = (int)(e % H);
    const float gi = gates[e], gf = gates[plane + e], gg = gates[2 * plane + e], go = gates[3 * plane + e];
    // the gradient from step k + 1: stored, or still in the parts of the contraction that made it
    const float dh = dha[e] + (dh_parts.splits ? tc::split_parts_sum(dh_parts, b, j) : dh_rec[e]);
    const float th = tanhf(c_t[e]);
    const float d_o = dh * th;
    const float dc = fmaf(dh * go, 1.f - th * th, dc_rec[e]);
    const float v[4] = {dc * gg * gi * (1.f - gi), dc * c_prev[e] * gf * (1.f - gf), dc * gi * (1.f - gg * gg),
                        d_o * go * (1.f - go)};
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const size_t col = (size_t)q * H + j;
      if (dz) dz[(size_t)b * G + col] = v[q];
      bf16 hi, mid;
      split2(v[q], hi, mid);
      bf16* o = dz3 + (size_t)b * 3 * G + col;
      o[0] = hi; o[G] = hi; o[2 * G] = mid;
    }
    dc_rec[e] = dc * gf;
    // h_{k-1}: same index space
    bf16 hi, mid;
    split2(hp[e], hi, mid);
    st_hp2[(size_t)b * 2 * H + j] = hi;
    st_hp2[(size_t)b * 2 * H + H + j] = mid;
  }
  const size_t ni = (size_t)B * I;
  for (size_t e = blockIdx.x * (size_t)blockDim.x + threadIdx.x; e < ni; e += (size_t)gridDim.x * blockDim.x) {
    const size_t b = e / I, c = e % I;
    bf16 hi, mid;
    split2(in[e], hi, mid);
    st_in2[b * 2 * I + c] = hi;
    st_in2[b * 2 * I + I + c] = mid;
  }
  if (counters && blockIdx.x == 0 && threadIdx.x == 0) counters[1] += 1;
}

// out[c] += sum over the rows r = 0 .. R-1 of hi + mid, for rows [hi | hi | mid] of width 3 N as
// the stages hold them: the bias gradients of a chunk (row = step within the chunk, then batch
// index).  Sixteen partial sums per column (rows r = y, y + 16, ... ascending for y = 0 .. 15),
// added in the order of y: fixed, and the same whatever the plan.  One block per 64 columns (N is
// a multiple of 8).
__global__ void __launch_bounds__(512) colsum_rows3(const bf16* v3, int R, int N, float* out) {
  __shared__ float part[16][64];
  sm100::grid_dep_wait();
  sm100::grid_dep_launch();
  const int c = blockIdx.x * 64 + 2 * threadIdx.x, y = threadIdx.y;
  float a0 = 0.f, a1 = 0.f;
  if (c < N) {
    for (int r = y; r < R; r += 16) {
      const bf16* row = v3 + (size_t)r * 3 * N + c;
      const __nv_bfloat162 hi = *reinterpret_cast<const __nv_bfloat162*>(row);
      const __nv_bfloat162 mid = *reinterpret_cast<const __nv_bfloat162*>(row + 2 * (size_t)N);
      a0 += __low2float(hi) + __low2float(mid);
      a1 += __high2float(hi) + __high2float(mid);
    }
  }
  part[y][2 * threadIdx.x] = a0;
  part[y][2 * threadIdx.x + 1] = a1;
  __syncthreads();
  const int t = y * 32 + threadIdx.x;
  if (t < 64 && blockIdx.x * 64 + t < N) {
    float acc = 0.f;
#pragma unroll
    for (int g = 0; g < 16; ++g) acc += part[g][t];
    out[blockIdx.x * 64 + t] += acc;
  }
}

// Loss terms of n steps from their partial sums, each summed in index order.
__global__ void sum_parts_steps(const float* part, int per_step, int n, float* out) {
  sm100::grid_dep_wait();
  sm100::grid_dep_launch();
  const int a = blockIdx.x * blockDim.x + threadIdx.x;
  if (a >= n) return;
  float s = 0.f;
  for (int i = 0; i < per_step; ++i) s += part[(size_t)a * per_step + i];
  out[a] = s;
}
__global__ void sum_parts(const float* part, int n, float* out) {
  sm100::grid_dep_wait();
  sm100::grid_dep_launch();
  if (threadIdx.x == 0 && blockIdx.x == 0) {
    float s = 0.f;
    for (int i = 0; i < n; ++i) s += part[i];
    *out = s;
  }
}

}  // namespace

void pack_weights(const Scratch& w, int L, int I0, int H, int O, const float* W, const size_t* w_off,
                  const float* W_out, cudaStream_t s) {
  const int G = 4 * H;
  for (int l = 0; l < L; ++l) {
    const int K = (l == 0 ? I0 : H) + H;
    const size_t n = (size_t)G * K;
    launch_pdl(pack3_cols, dim3(ew_blocks(n)), dim3(256), 0, s, W + w_off[l], G, K, w.w3 + 3 * w_off[l]);
    launch_pdl(pack3_rows, dim3(ew_blocks(n)), dim3(256), 0, s, W + w_off[l], G, K, w.wmn3 + 3 * w_off[l]);
  }
  const size_t no = (size_t)O * H;
  launch_pdl(pack3_cols, dim3(ew_blocks(no)), dim3(256), 0, s, W_out, O, H, w.wout3);
  launch_pdl(pack3_rows, dim3(ew_blocks(no)), dim3(256), 0, s, W_out, O, H, w.woutmn3);
}

int forward_step(const generic::FwdArgs& a, const Scratch& w, int l, size_t w_off, cudaStream_t s) {
  const int K = a.I + a.H, G = 4 * a.H;
  const size_t nk = (size_t)a.B * K;
  launch_pdl(split_a3, dim3(ew_blocks(nk)), dim3(256), 0, s, (const float*)a.in, a.I, (const float*)a.h_prev, a.H, a.B, w.a3);
  // split along K where that puts more SMs to work; the cell kernel adds the parts, and the bias
  tc::SplitParts zp;
  int rc = gemm_bf16(w.a3, 3 * K, false, w.w3 + 3 * w_off, 3 * K, false, GemmOut{GemmOut::STORE_F32, w.z, G, nullptr, 0},
                     a.B, G, 3 * K, w.status, s, true, &w.split, tc::gemm_split_count_deferred(a.B, G, 3 * K), &zp);
  if (rc != MEBPTT_OK) return rc;
  const size_t n = (size_t)a.B * a.H;
  launch_pdl(cell_fwd, dim3(ew_blocks(n)), dim3(256), 0, s, w.z, a.c_prev, (const float*)a.h_prev, (float*)a.h_out, a.c_out, (float*)a.gates,
                                        a.plane_elems, (float*)a.h_in_copy, a.c_in_copy, a.B, a.H, a.counters, (bf16*)nullptr, 0, a.bias, zp);
  (void)l;
  return MEBPTT_OK;
}

// n consecutive forward operations of one layer.  One launch splits the layer's inputs of all n
// steps and the h of the state the run starts from into the left operands a3_run[j] = [B][3K];
// every step is then the single-step contraction over its operand and the cell kernel, which also
// writes the halves of h_k into the operand of the next step.  The operands hold what the
// single-step function would have put there, so every sum is the same.
int forward_run_layer(const stepwise::FwdRunStep* st, int n, const float* in, int64_t in_step_stride, int I, const float* bias,
                      int B, int H, size_t plane_elems, int64_t* counters, const Scratch& w, size_t w_off,
                      float* h_stage, cudaStream_t s) {
  const int K = I + H, G = 4 * H;
  const size_t row3 = (size_t)B * 3 * K;
  launch_pdl(split_run_inputs, dim3(ew_blocks((size_t)B * K) > 128 ? 128 : ew_blocks((size_t)B * K), n), dim3(256), 0, s, in,
             in_step_stride, I, (const float*)st[0].h_prev, H, B, w.a3_run);
  const size_t nbh = (size_t)B * H;
  for (int j = 0; j < n; ++j) {
    tc::SplitParts zp;
    const int rc = gemm_bf16(w.a3_run + (size_t)j * row3, 3 * K, false, w.w3 + 3 * w_off, 3 * K, false,
                             GemmOut{GemmOut::STORE_F32, w.z, G, nullptr, 0}, B, G, 3 * K, w.status, s, true, &w.split,
                             tc::gemm_split_count_deferred(B, G, 3 * K), &zp);
    if (rc != MEBPTT_OK) return rc;
    float* h_out = (float*)st[j].h_out;
    launch_pdl(cell_fwd, dim3(ew_blocks(nbh)), dim3(256), 0, s, (const float*)w.z, st[j].c_prev, (const float*)st[j].h_prev, h_out,
               st[j].c_out, (float*)st[j].gates, plane_elems, (float*)st[j].h_in_copy, st[j].c_in_copy, B, H, counters,
               j + 1 < n ? w.a3_run + (size_t)(j + 1) * row3 : (bf16*)nullptr, I, bias, zp);
    if (h_stage) {
      // the layer above reads the h_k of the run from one block: a copy beside the tape's place
      cudaMemcpyAsync(h_stage + (size_t)j * nbh, h_out, nbh * 4, cudaMemcpyDeviceToDevice, s);
    }
  }
  return MEBPTT_OK;
}

int readout(const generic::ReadoutArgs& a, const Scratch& w, int sidx, cudaStream_t s) {
  bf16* h3 = w.st_h3 + (size_t)sidx * a.B * 3 * a.H;
  bf16* dy3 = w.st_dy3 + (size_t)sidx * a.B * 3 * a.O;
  const size_t nh = (size_t)a.B * a.H, no = (size_t)a.B * a.O;
  launch_pdl(split_a3, dim3(ew_blocks(nh)), dim3(256), 0, s, (const float*)a.h, a.H, nullptr, 0, a.B, h3);
  GemmOut o{GemmOut::LOSS_DY, nullptr, a.O, a.b_out, 0};
  o.target = a.target;
  o.dy32 = a.dy;
  o.loss_part = a.loss_part;
  o.parts = (a.O + 31) / 32;
  o.scale = 1.f / ((float)a.B * (float)a.O);
  int rc = gemm_bf16(h3, 3 * a.H, false, w.wout3, 3 * a.H, false, o, a.B, a.O, 3 * a.H, w.status, s);
  if (rc != MEBPTT_OK) return rc;
  launch_pdl(sum_parts, dim3(1), dim3(32), 0, s, a.loss_part, (a.B / 32) * o.parts, a.loss_k);
  launch_pdl(split_a3, dim3(ew_blocks(no)), dim3(256), 0, s, a.dy, a.O, nullptr, 0, a.B, dy3);
  // dha[b][j] = sum_o dy[b][o] W_out[o][j]
  return gemm_bf16(dy3, 3 * a.O, false, w.woutmn3, a.H, true, GemmOut{GemmOut::STORE_F32, a.dha, a.H, nullptr, 0}, a.B,
                   a.H, 3 * a.O, w.status, s, true, &w.split);
}

// The readout of n steps at once (a run of backward operations inside one chunk): every element
// by the sums of the single-step function, the contraction for dha split along K into the parts a
// single step would take.
int readout_run(const float* const* h_top, int n, int s_lo, const float* b_out, const float* target, float* loss_t,
                int B, int H, int O, const Scratch& w, cudaStream_t s) {
  bf16* h3 = w.st_h3 + (size_t)s_lo * B * 3 * H;
  bf16* dy3 = w.st_dy3 + (size_t)s_lo * B * 3 * O;
  const size_t nh = (size_t)B * H, no = (size_t)n * B * O;
  RunPtrs ptrs{};
  for (int a = 0; a < n; ++a) ptrs.p[a] = h_top[a];
  launch_pdl(split_blocks3, dim3(ew_blocks(nh) > 64 ? 64 : ew_blocks(nh), n), dim3(256), 0, s, ptrs, H, B, h3);
  const int parts = (O + 31) / 32, per_step = (B / 32) * parts;
  GemmOut o{GemmOut::LOSS_DY, nullptr, O, b_out, 0};
  o.target = target;
  o.dy32 = w.dy_run;
  o.loss_part = w.loss_part;
  o.parts = parts;
  o.scale = 1.f / ((float)B * (float)O);
  int rc = gemm_bf16(h3, 3 * H, false, w.wout3, 3 * H, false, o, n * B, O, 3 * H, w.status, s);
  if (rc != MEBPTT_OK) return rc;
  launch_pdl(sum_parts_steps, dim3((n + 31) / 32), dim3(32), 0, s, (const float*)w.loss_part, per_step, n, loss_t);
  launch_pdl(split_a3, dim3(ew_blocks(no)), dim3(256), 0, s, (const float*)w.dy_run, O, (const float*)nullptr, 0, n * B, dy3);
  const int splits = tc::gemm_split_count(false, true, B, H, 3 * O, w.split.partial_floats);
  return gemm_bf16(dy3, 3 * O, false, w.woutmn3, H, true, GemmOut{GemmOut::STORE_F32, w.dha_run, H, nullptr, 0}, n * B, H,
                   3 * O, w.status, s, true, &w.split_run, splits);
}

int backward_layer(const generic::BwdArgs& a, const Scratch& w, int l, size_t w_off, int sidx, cudaStream_t s) {
  const int K = a.I + a.H, G = 4 * a.H;
  const size_t n = (size_t)a.B * a.H;
  const size_t rows = (size_t)w.S * a.B;
  bf16* dz3 = w.st_dz3 + ((size_t)l * rows + (size_t)sidx * a.B) * 3 * G;
  bf16* in2 = w.st_in2 + (l == 0 ? 0 : rows * 2 * w.I0 + (size_t)(l - 1) * rows * 2 * a.H) + (size_t)sidx * a.B * 2 * a.I;
  bf16* hp2 = w.st_hp2 + ((size_t)l * rows + (size_t)sidx * a.B) * 2 * a.H;
  launch_pdl(gate_bwd, dim3(ew_blocks(n)), dim3(256), 0, s, a.dha, a.dh_rec, a.dc_rec, (const float*)a.gates, a.plane_elems, a.c_t, a.c_prev,
                                        (float*)nullptr, dz3, a.B, a.H, a.counters, (const float*)a.in, a.I, in2,
                                        (const float*)a.h_prev, hp2, w.dh_parts[l]);
  const bf16* WMN = w.wmn3 + 3 * w_off;   // [3G][K]
  if (a.d_lo) {
    int rc = gemm_bf16(dz3, 3 * G, false, WMN, K, true, GemmOut{GemmOut::STORE_F32, a.d_lo, a.I, nullptr, 0}, a.B, a.I,
                       3 * G, w.status, s, true, &w.split);
    if (rc != MEBPTT_OK) return rc;
  }
  const tc::SplitWs own{w.split_dh + (size_t)l * DH_PART_FLOATS, DH_PART_FLOATS};
  return gemm_bf16(dz3, 3 * G, false, WMN + a.I, K, true, GemmOut{GemmOut::STORE_F32, a.dh_rec, a.H, nullptr, 0}, a.B,
                   a.H, 3 * G, w.status, s, true, &own, 0, &w.dh_parts[l]);
}

namespace {
// C[m][n] += sum_r (a_hi a_mid)[r][m] (b_hi b_mid)[r][n] as hi hi + hi mid + mid hi; a3 rows are
// [hi | hi | mid] of width Ma, b2 rows [hi | mid] of width Nb.
int accum3(const bf16* a3, int Ma, const bf16* b2, int Nb, bool b_is_a3, float* C, int64_t ldc, int R, int* status,
           cudaStream_t s) {
  const int64_t lda = 3 * (int64_t)Ma, ldb = (b_is_a3 ? 3 : 2) * (int64_t)Nb;
  const bf16* a_hi = a3;
  const bf16* a_mid = a3 + 2 * (size_t)Ma;
  const bf16* b_hi = b2;
  const bf16* b_mid = b2 + (b_is_a3 ? 2 : 1) * (size_t)Nb;
  const GemmOut o{GemmOut::ACCUM_F32, C, ldc, nullptr, 0};
  int rc = gemm_bf16(a_hi, lda, true, b_hi, ldb, true, o, Ma, Nb, R, status, s);
  if (rc != MEBPTT_OK) return rc;
  rc = gemm_bf16(a_hi, lda, true, b_mid, ldb, true, o, Ma, Nb, R, status, s);
  if (rc != MEBPTT_OK) return rc;
  return gemm_bf16(a_mid, lda, true, b_hi, ldb, true, o, Ma, Nb, R, status, s);
}
}  // namespace

int flush_chunk(const Scratch& w, int steps, int L, int B, int I0, int H, int O, const size_t* w_off, float* dW,
                float* dW_out, float* db, float* db_out, cudaStream_t s) {
  const int G = 4 * H, R = steps * B;
  const size_t rows = (size_t)w.S * B;
  for (int l = 0; l < L; ++l) {
    const int I = l == 0 ? I0 : H, K = I + H;
    const bf16* dz3 = w.st_dz3 + (size_t)l * rows * 3 * G;
    launch_pdl(colsum_rows3, dim3((G + 63) / 64), dim3(32, 16), 0, s, dz3, R, G, db + (size_t)l * G);
    const bf16* in2 = w.st_in2 + (l == 0 ? 0 : rows * 2 * I0 + (size_t)(l - 1) * rows * 2 * H);
    const bf16* hp2 = w.st_hp2 + (size_t)l * rows * 2 * H;
    float* dWl = dW + w_off[l];
    int rc = accum3(dz3, G, in2, I, false, dWl, K, R, w.status, s);
    if (rc != MEBPTT_OK) return rc;
    rc = accum3(dz3, G, hp2, H, false, dWl + I, K, R, w.status, s);
    if (rc != MEBPTT_OK) return rc;
  }
  launch_pdl(colsum_rows3, dim3((O + 63) / 64), dim3(32, 16), 0, s, (const bf16*)w.st_dy3, R, O, db_out);
  return accum3(w.st_dy3, O, w.st_h3, H, true, dW_out, H, R, w.status, s);
}

}  // namespace stepwise3
}  // namespace mebptt
