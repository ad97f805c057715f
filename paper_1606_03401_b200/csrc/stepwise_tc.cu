// Step-by-step LSTM operations with every contraction on the tensor cores.
//
// The persistent kernels keep W_hh in shared memory and cover one layer, a batch of at most 64
// and H <= 1024.  Outside that range (several layers, H = 2048, B = 128) a forward or backward
// operation is carried out layer by layer as a short sequence of launches, like the CUDA-core
// path does, but with its contractions given to the tcgen05 GEMM (bfloat16 operands, float32
// accumulation in a fixed order) and the gate arithmetic in small element-wise kernels:
//   forward    z  = in W[:, :I]^T + b ;  z += h_prev W[:, I:]^T ;  gates, c, h from z
//   readout    y  = h W_out^T + b_out, loss term and dy in the GEMM's epilogue ; dha = dy W_out
//   backward   dz from the stored gates ; d_in = dz W[:, :I] ; dh = dz W[:, I:]
//   per chunk  dW += dz^T [in ; h_prev], db += sum of dz, dW_out += dy^T h and db_out += sum of dy
//              over the S steps of a chunk at once: dz, dy and the operands they meet are staged
//              per step (row block (k - 1) % S), and the chunk is flushed when its first step has
//              been backpropagated.  Chunks are tied to absolute time, so the order of every sum
//              is the same for every plan.
// dz and dy are rounded to bfloat16 before they enter a contraction or a bias gradient (as on the
// persistent path).  Every sum has a fixed order, and an operation's launches
// do not depend on the plan, so results are bit-identical across plans.
#include "kernels.hpp"
#include "launch.hpp"
#include "sm100.cuh"
#include "tc.hpp"

#include <cuda_bf16.h>
#include <cuda_runtime.h>

namespace mebptt {
namespace stepwise {

namespace {

using tc::GemmOut;
using tc::gemm_bf16;
typedef __nv_bfloat16 bf16;

__device__ __forceinline__ float sigmoidf_(float a) { return 1.0f / (1.0f + expf(-a)); }

// V consecutive elements at once (V = 4 where every array involved is 16-byte aligned, else 1).
template <int V> __device__ __forceinline__ void ld(const float* p, float (&v)[V]) {
  if constexpr (V == 4) { const float4 t = *reinterpret_cast<const float4*>(p); v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w; }
  else v[0] = *p;
}
template <int V> __device__ __forceinline__ void st(float* p, const float (&v)[V]) {
  if constexpr (V == 4) *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]);
  else *p = v[0];
}
template <int V> __device__ __forceinline__ void ld(const bf16* p, float (&v)[V]) {
  if constexpr (V == 4) {
    const uint2 t = *reinterpret_cast<const uint2*>(p);
    v[0] = __uint_as_float(t.x << 16); v[1] = __uint_as_float(t.x & 0xFFFF0000u);
    v[2] = __uint_as_float(t.y << 16); v[3] = __uint_as_float(t.y & 0xFFFF0000u);
  } else v[0] = __bfloat162float(*p);
}
template <int V> __device__ __forceinline__ void st(bf16* p, const float (&v)[V]) {   // rounds to nearest even
  if constexpr (V == 4) *reinterpret_cast<uint2*>(p) = make_uint2(sm100::pack_bf16x2(v[0], v[1]), sm100::pack_bf16x2(v[2], v[3]));
  else *p = __float2bfloat16_rn(v[0]);
}
template <int V> __device__ __forceinline__ void cp(bf16* dst, const bf16* src) {
  if constexpr (V == 4) *reinterpret_cast<uint2*>(dst) = *reinterpret_cast<const uint2*>(src);
  else *dst = *src;
}
// v[i] += the sum of the parts at (m, n + i); the V columns lie in one tile (n is a multiple of V)
template <int V> __device__ __forceinline__ void add_parts(const tc::SplitParts& sp, int m, int n, float (&v)[V]) {
  const int tile = (m >> 7) * sp.tiles_x + n / sp.bn;
  const float* p = sp.partial + (((size_t)tile * sp.splits) * 128 + (size_t)(m & 127)) * sp.bn + (n % sp.bn);
  float acc[V];
#pragma unroll
  for (int i = 0; i < V; ++i) acc[i] = 0.f;
  for (int z = 0; z < sp.splits; ++z) {
    float t[V];
    ld<V>(p + (size_t)z * 128 * sp.bn, t);
#pragma unroll
    for (int i = 0; i < V; ++i) acc[i] += t[i];
  }
#pragma unroll
  for (int i = 0; i < V; ++i) v[i] += acc[i];
}

// z [B][4H] (column q H + j: gate q of unit j, bias included) -> gates, c_k, h_k and, for an
// internal state, the copies of h_{k-1}, c_{k-1}.
// zp: where the recurrent product lies if it was split along K (its parts are then added to z here).
template <int V>
__global__ void cell_fwd(const float* z, const float* c_prev, const bf16* h_prev, bf16* h_out, float* c_out,
                         bf16* gates, size_t plane, bf16* h_in_copy, float* c_in_copy, int B, int H,
                         int64_t* counters, bf16* h_stage, const tc::SplitParts zp) {
  sm100::grid_dep_wait();
  sm100::grid_dep_launch();
  const size_t n = (size_t)B * H / V;
  for (size_t g = blockIdx.x * (size_t)blockDim.x + threadIdx.x; g < n; g += (size_t)gridDim.x * blockDim.x) {
    const size_t e = g * V;
    const int b = (int)(e / H), j = (int)(e % H);
    const float* row = z + (size_t)b * 4 * H;
    float zq[4][V];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      ld<V>(row + (size_t)q * H + j, zq[q]);
      if (zp.splits) add_parts<V>(zp, b, q * H + j, zq[q]);
    }
    float cp_[V], c[V], hv[V], gi[V], gf[V], gg[V], go[V];
    ld<V>(c_prev + e, cp_);
#pragma unroll
    for (int i = 0; i < V; ++i) {
      gi[i] = sigmoidf_(zq[0][i]); gf[i] = sigmoidf_(zq[1][i]);
      gg[i] = tanhf(zq[2][i]);     go[i] = sigmoidf_(zq[3][i]);
      c[i] = fmaf(gf[i], cp_[i], gi[i] * gg[i]);
      hv[i] = go[i] * tanhf(c[i]);
    }
    st<V>(c_out + e, c);
    st<V>(h_out + e, hv);
    if (h_stage) st<V>(h_stage + e, hv);   // a second copy, where the layer above reads its inputs of a whole run
    if (gates) {
      st<V>(gates + e, gi); st<V>(gates + plane + e, gf);
      st<V>(gates + 2 * plane + e, gg); st<V>(gates + 3 * plane + e, go);
    }
    if (h_in_copy) { cp<V>(h_in_copy + e, h_prev + e); st<V>(c_in_copy + e, cp_); }
  }
  if (counters && blockIdx.x == 0 && threadIdx.x == 0) counters[0] += 1;
}

// Gate derivatives: dh = dha + dh_rec; dz [B][4H] rounded to bfloat16 (for the contractions and the
// bias gradient), and in float32 as well if dz is given; dc_rec = dc * f.
// Also copies this step's layer input and h_{k-1} to their stages (n_in16, n_hp16: 16-byte words).
template <int V>
__global__ void gate_bwd(const float* dha, const float* dh_rec, float* dc_rec, const bf16* gates, size_t plane,
                         const float* c_t, const float* c_prev, float* dz, bf16* dz16, int B, int H,
                         int64_t* counters, const uint4* in, uint4* st_in, size_t n_in16, const uint4* hp,
                         uint4* st_hp, size_t n_hp16, const tc::SplitParts dh_parts) {
  sm100::grid_dep_wait();
  sm100::grid_dep_launch();
  const size_t n = (size_t)B * H / V;
  for (size_t e = blockIdx.x * (size_t)blockDim.x + threadIdx.x; e < n_in16; e += (size_t)gridDim.x * blockDim.x)
    st_in[e] = in[e];
  for (size_t e = blockIdx.x * (size_t)blockDim.x + threadIdx.x; e < n_hp16; e += (size_t)gridDim.x * blockDim.x)
    st_hp[e] = hp[e];
  for (size_t g = blockIdx.x * (size_t)blockDim.x + threadIdx.x; g < n; g += (size_t)gridDim.x * blockDim.x) {
    const size_t e = g * V;
    const int b = (int)(e / H), j = (int)(e % H);
    float gi[V], gf[V], gg[V], go[V], dh[V], rec[V], ct[V], cpv[V], dcr[V];
    ld<V>(gates + e, gi); ld<V>(gates + plane + e, gf); ld<V>(gates + 2 * plane + e, gg); ld<V>(gates + 3 * plane + e, go);
    ld<V>(dha + e, dh);
    // the gradient from step k + 1: stored, or still in the parts of the contraction that made it
    if (dh_parts.splits) {
#pragma unroll
      for (int i = 0; i < V; ++i) rec[i] = 0.f;
      add_parts<V>(dh_parts, b, j, rec);
    } else {
      ld<V>(dh_rec + e, rec);
    }
    ld<V>(c_t + e, ct); ld<V>(c_prev + e, cpv); ld<V>(dc_rec + e, dcr);
    float v[4][V], dcn[V];
#pragma unroll
    for (int i = 0; i < V; ++i) {
      const float d = dh[i] + rec[i];
      const float th = tanhf(ct[i]);
      const float d_o = d * th;
      const float dc = fmaf(d * go[i], 1.f - th * th, dcr[i]);
      v[0][i] = dc * gg[i] * gi[i] * (1.f - gi[i]);
      v[1][i] = dc * cpv[i] * gf[i] * (1.f - gf[i]);
      v[2][i] = dc * gi[i] * (1.f - gg[i] * gg[i]);
      v[3][i] = d_o * go[i] * (1.f - go[i]);
      dcn[i] = dc * gf[i];
    }
    const size_t r = (size_t)b * 4 * H + j;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      if (dz) st<V>(dz + r + (size_t)q * H, v[q]);
      st<V>(dz16 + r + (size_t)q * H, v[q]);
    }
    st<V>(dc_rec + e, dcn);
  }
  if (counters && blockIdx.x == 0 && threadIdx.x == 0) counters[1] += 1;
}

// every pointer a multiple of 16 bytes?
template <class... P>
inline bool aligned16(P... p) { return ((... | reinterpret_cast<uintptr_t>(p)) & 15) == 0; }

inline int ew_blocks(size_t n) { return (int)((n + 255) / 256 > 1184 ? 1184 : (n + 255) / 256); }

// The two element-wise kernels, four elements per thread where the addresses allow (same results).
void run_cell_fwd(cudaStream_t s, const float* z, const float* c_prev, const bf16* h_prev, bf16* h_out, float* c_out,
                  bf16* gates, size_t plane, bf16* h_in_copy, float* c_in_copy, int B, int H, int64_t* counters,
                  bf16* h_stage, const tc::SplitParts& zp) {
  const size_t n = (size_t)B * H;
  const bool vec = H % 4 == 0 && plane % 8 == 0 &&
                   aligned16(z, c_prev, h_prev, h_out, c_out, gates, h_in_copy, c_in_copy, h_stage, zp.partial);
  if (vec)
    launch_pdl(cell_fwd<4>, dim3(ew_blocks(n / 4)), dim3(256), 0, s, z, c_prev, h_prev, h_out, c_out, gates, plane, h_in_copy,
               c_in_copy, B, H, counters, h_stage, zp);
  else
    launch_pdl(cell_fwd<1>, dim3(ew_blocks(n)), dim3(256), 0, s, z, c_prev, h_prev, h_out, c_out, gates, plane, h_in_copy,
               c_in_copy, B, H, counters, h_stage, zp);
}
void run_gate_bwd(cudaStream_t s, const float* dha, const float* dh_rec, float* dc_rec, const bf16* gates, size_t plane,
                  const float* c_t, const float* c_prev, bf16* dz16, int B, int H, int64_t* counters, const uint4* in,
                  uint4* st_in, size_t n_in16, const uint4* hp, uint4* st_hp, size_t n_hp16, const tc::SplitParts& parts) {
  const size_t n = (size_t)B * H;
  const bool vec = H % 4 == 0 && plane % 8 == 0 && aligned16(dha, dh_rec, dc_rec, gates, c_t, c_prev, dz16, parts.partial);
  if (vec)
    launch_pdl(gate_bwd<4>, dim3(ew_blocks(n / 4)), dim3(256), 0, s, dha, dh_rec, dc_rec, gates, plane, c_t, c_prev,
               (float*)nullptr, dz16, B, H, counters, in, st_in, n_in16, hp, st_hp, n_hp16, parts);
  else
    launch_pdl(gate_bwd<1>, dim3(ew_blocks(n)), dim3(256), 0, s, dha, dh_rec, dc_rec, gates, plane, c_t, c_prev,
               (float*)nullptr, dz16, B, H, counters, in, st_in, n_in16, hp, st_hp, n_hp16, parts);
}

// out[c] += sum over the rows r = 0 .. R-1 of v[r][c]: the bias gradients of a chunk from its
// staged rows (row = step within the chunk, then batch index).  Sixteen partial sums per column
// (rows r = y, y + 16, ... ascending for y = 0 .. 15), added in the order of y: fixed, and the
// same whatever the plan.  One block per 64 columns (N is a multiple of 8).
__global__ void __launch_bounds__(512) colsum_rows(const bf16* v, int R, int N, float* out) {
  __shared__ float part[16][64];
  sm100::grid_dep_wait();
  sm100::grid_dep_launch();
  const int c = blockIdx.x * 64 + 2 * threadIdx.x, y = threadIdx.y;
  float a0 = 0.f, a1 = 0.f;
  if (c < N) {
    int r = y;
    for (; r + 48 < R; r += 64) {
      __nv_bfloat162 x[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) x[u] = *reinterpret_cast<const __nv_bfloat162*>(v + (size_t)(r + 16 * u) * N + c);
#pragma unroll
      for (int u = 0; u < 4; ++u) { a0 += __low2float(x[u]); a1 += __high2float(x[u]); }
    }
    for (; r < R; r += 16) {
      const __nv_bfloat162 x = *reinterpret_cast<const __nv_bfloat162*>(v + (size_t)r * N + c);
      a0 += __low2float(x); a1 += __high2float(x);
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

// Loss term of one step from its partial sums (block 0, one thread); every block helps copy the
// top layer's h_k to its stage.
__global__ void sum_parts_stage_h(const float* part, int n, float* out, const uint4* h, uint4* st_h, size_t n_h16) {
  sm100::grid_dep_wait();
  sm100::grid_dep_launch();
  for (size_t e = blockIdx.x * (size_t)blockDim.x + threadIdx.x; e < n_h16; e += (size_t)gridDim.x * blockDim.x)
    st_h[e] = h[e];
  if (threadIdx.x == 0 && blockIdx.x == 0) {
    float s = 0.f;
    for (int i = 0; i < n; ++i) s += part[i];
    *out = s;
  }
}

// Up to 64 device pointers passed by value (a run has at most 64 steps).
struct RunPtrs { const void* p[64]; };

// Row block a of `dst` (n16 16-byte words each) <- src.p[a]; blockIdx.y = a.
__global__ void stage_blocks(RunPtrs src, uint4* dst, size_t n16) {
  sm100::grid_dep_wait();
  sm100::grid_dep_launch();
  const uint4* from = reinterpret_cast<const uint4*>(src.p[blockIdx.y]);
  uint4* to = dst + (size_t)blockIdx.y * n16;
  for (size_t e = blockIdx.x * (size_t)blockDim.x + threadIdx.x; e < n16; e += (size_t)gridDim.x * blockDim.x) to[e] = from[e];
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


}  // namespace

int forward_step(const generic::FwdArgs& a, const Scratch& w, cudaStream_t s) {
  const int K = a.I + a.H, G = 4 * a.H;
  const bf16* W = (const bf16*)a.W;
  int rc = gemm_bf16(a.in, a.I, false, W, K, false, GemmOut{GemmOut::STORE_F32, w.z, G, a.bias, 0}, a.B, G, a.I,
                     w.status, s, true, &w.split);
  if (rc != MEBPTT_OK) return rc;
  // the recurrent part: split along K where that puts more SMs to work, its parts added by the cell kernel
  tc::SplitParts zp;
  rc = gemm_bf16(a.h_prev, a.H, false, W + a.I, K, false, GemmOut{GemmOut::ACCUM_F32, w.z, G, nullptr, 0}, a.B, G,
                 a.H, w.status, s, true, &w.split, tc::gemm_split_count_deferred(a.B, G, a.H), &zp);
  if (rc != MEBPTT_OK) return rc;
  run_cell_fwd(s, w.z, a.c_prev, (const bf16*)a.h_prev, (bf16*)a.h_out, a.c_out, (bf16*)a.gates, a.plane_elems,
               (bf16*)a.h_in_copy, a.c_in_copy, a.B, a.H, a.counters, (bf16*)nullptr, zp);
  return MEBPTT_OK;
}

int readout(const generic::ReadoutArgs& a, const Scratch& w, int sidx, cudaStream_t s) {
  const bf16* W_out = (const bf16*)a.W_out;
  bf16* dy16 = w.st_dy + (size_t)sidx * a.B * a.O;
  GemmOut o{GemmOut::LOSS_DY, dy16, a.O, a.b_out, 0};
  o.target = a.target;
  o.loss_part = a.loss_part;
  o.parts = (a.O + 31) / 32;
  o.scale = 1.f / ((float)a.B * (float)a.O);
  int rc = gemm_bf16(a.h, a.H, false, W_out, a.H, false, o, a.B, a.O, a.H, w.status, s, true, &w.split);
  if (rc != MEBPTT_OK) return rc;
  const size_t n_h16 = (size_t)a.B * a.H * 2 / 16;
  launch_pdl(sum_parts_stage_h, dim3(ew_blocks(n_h16 * 8)), dim3(256), 0, s, a.loss_part, (a.B / 32) * o.parts, a.loss_k, (const uint4*)a.h,
                                                          (uint4*)(w.st_h + (size_t)sidx * a.B * a.H), n_h16);
  // dha[b][j] = sum_o dy[b][o] W_out[o][j]: W_out read as the [k][n] operand
  rc = gemm_bf16(dy16, a.O, false, W_out, a.H, true, GemmOut{GemmOut::STORE_F32, a.dha, a.H, nullptr, 0}, a.B, a.H,
                 a.O, w.status, s, true, &w.split);
  return rc;   // db_out is summed from the staged dy when the chunk is flushed
}

int backward_layer(const generic::BwdArgs& a, const Scratch& w, int l, int sidx, cudaStream_t s) {
  const int K = a.I + a.H, G = 4 * a.H;
  const bf16* W = (const bf16*)a.W;
  const size_t rows = (size_t)w.S * a.B;   // rows of one layer's stages
  bf16* dz16 = w.st_dz + ((size_t)l * rows + (size_t)sidx * a.B) * G;
  bf16* st_in = w.st_in + (l == 0 ? 0 : rows * w.I0 + (size_t)(l - 1) * rows * a.H) + (size_t)sidx * a.B * a.I;
  bf16* st_hp = w.st_hp + ((size_t)l * rows + (size_t)sidx * a.B) * a.H;
  run_gate_bwd(s, a.dha, a.dh_rec, a.dc_rec, (const bf16*)a.gates, a.plane_elems, a.c_t, a.c_prev, dz16, a.B, a.H, a.counters,
               (const uint4*)a.in, (uint4*)st_in, (size_t)a.B * a.I * 2 / 16, (const uint4*)a.h_prev, (uint4*)st_hp,
               (size_t)a.B * a.H * 2 / 16, w.dh_parts[l]);
  // d_in = dz W: columns < I feed dx or the layer below, the rest is the new dh_rec
  if (a.d_lo) {
    int rc = gemm_bf16(dz16, G, false, W, K, true, GemmOut{GemmOut::STORE_F32, a.d_lo, a.I, nullptr, 0}, a.B, a.I, G,
                       w.status, s, true, &w.split);
    if (rc != MEBPTT_OK) return rc;
  }
  const tc::SplitWs own{w.split_dh + (size_t)l * DH_PART_FLOATS, DH_PART_FLOATS};
  return gemm_bf16(dz16, G, false, W + a.I, K, true, GemmOut{GemmOut::STORE_F32, a.dh_rec, a.H, nullptr, 0}, a.B, a.H,
                   G, w.status, s, true, &own, 0, &w.dh_parts[l]);
}

// Weight gradients of a finished chunk: `steps` row blocks of B rows, from block 0 on.
int flush_chunk(const Scratch& w, int steps, int L, int B, int I0, int H, int O, const size_t* w_off, float* dW,
                float* dW_out, float* db, float* db_out, cudaStream_t s) {
  const int G = 4 * H, R = steps * B;
  const size_t rows = (size_t)w.S * B;
  for (int l = 0; l < L; ++l) {
    const int I = l == 0 ? I0 : H, K = I + H;
    const bf16* dz = w.st_dz + (size_t)l * rows * G;
    // db[g] += sum over (step, b) of the staged dz (as the contractions below see it)
    launch_pdl(colsum_rows, dim3((G + 63) / 64), dim3(32, 16), 0, s, dz, R, G, db + (size_t)l * G);
    const bf16* in = w.st_in + (l == 0 ? 0 : rows * I0 + (size_t)(l - 1) * rows * H);
    const bf16* hp = w.st_hp + (size_t)l * rows * H;
    float* dWl = dW + w_off[l];
    // dW[g][c] += sum over (step, b) of dz[.][g] [in ; h_prev][.][c]: both operands stored [k][.]
    int rc = gemm_bf16(dz, G, true, in, I, true, GemmOut{GemmOut::ACCUM_F32, dWl, K, nullptr, 0}, G, I, R, w.status, s);
    if (rc != MEBPTT_OK) return rc;
    rc = gemm_bf16(dz, G, true, hp, H, true, GemmOut{GemmOut::ACCUM_F32, dWl + I, K, nullptr, 0}, G, H, R, w.status, s);
    if (rc != MEBPTT_OK) return rc;
  }
  launch_pdl(colsum_rows, dim3((O + 63) / 64), dim3(32, 16), 0, s, (const bf16*)w.st_dy, R, O, db_out);
  return gemm_bf16(w.st_dy, O, true, w.st_h, H, true, GemmOut{GemmOut::ACCUM_F32, dW_out, H, nullptr, 0}, O, H, R,
                   w.status, s);
}

// ---- runs of consecutive operations, one layer at a time -----------------------------------------
// What depends on the previous step is only the product with the recurrent weights; the product
// with the layer's input, the readout and the gradient handed to the layer below are taken for
// all steps of the run at once.  Every element is computed by the same sums in the same order as
// in the single-step functions above (a contraction that those split along K is split into the
// same parts here), so a plan's results do not depend on how its tape falls into runs.

int forward_run_layer(const FwdRunStep* st, int n, const void* in, int I, const void* Wl, const float* bias,
                      bool stage_h, int B, int H, size_t plane_elems, int64_t* counters, const Scratch& w,
                      cudaStream_t s) {
  const int K = I + H, G = 4 * H;
  const bf16* W = (const bf16*)Wl;
  int rc = gemm_bf16(in, I, false, W, K, false, GemmOut{GemmOut::STORE_F32, w.zrun, G, bias, 0}, n * B, G, I, w.status, s);
  if (rc != MEBPTT_OK) return rc;
  const size_t bh = (size_t)B * H;
  for (int j = 0; j < n; ++j) {
    float* z = w.zrun + (size_t)j * B * G;
    tc::SplitParts zp;
    rc = gemm_bf16(st[j].h_prev, H, false, W + I, K, false, GemmOut{GemmOut::ACCUM_F32, z, G, nullptr, 0}, B, G, H,
                   w.status, s, true, &w.split, tc::gemm_split_count_deferred(B, G, H), &zp);
    if (rc != MEBPTT_OK) return rc;
    run_cell_fwd(s, z, st[j].c_prev, (const bf16*)st[j].h_prev, (bf16*)st[j].h_out, st[j].c_out, (bf16*)st[j].gates,
                 plane_elems, (bf16*)st[j].h_in_copy, st[j].c_in_copy, B, H, counters,
                 stage_h ? w.hrun + (size_t)j * bh : (bf16*)nullptr, zp);
  }
  return MEBPTT_OK;
}

int readout_run(const void* const* h_top, int n, int s_lo, const void* W_out_, const float* b_out, const float* target,
                float* loss_t, int B, int H, int O, const Scratch& w, cudaStream_t s) {
  const bf16* W_out = (const bf16*)W_out_;
  const size_t n_h16 = (size_t)B * H * 2 / 16;
  RunPtrs ptrs{};
  for (int a = 0; a < n; ++a) ptrs.p[a] = h_top[a];
  bf16* st_h = w.st_h + (size_t)s_lo * B * H;
  bf16* dy16 = w.st_dy + (size_t)s_lo * B * O;
  launch_pdl(stage_blocks, dim3(ew_blocks(n_h16 * 8) > 64 ? 64 : ew_blocks(n_h16 * 8), n), dim3(256), 0, s, ptrs,
             (uint4*)st_h, n_h16);
  const int parts = (O + 31) / 32, per_step = (B / 32) * parts;
  GemmOut o{GemmOut::LOSS_DY, dy16, O, b_out, 0};
  o.target = target;
  o.loss_part = w.loss_part;
  o.parts = parts;
  o.scale = 1.f / ((float)B * (float)O);
  int rc = gemm_bf16(st_h, H, false, W_out, H, false, o, n * B, O, H, w.status, s);
  if (rc != MEBPTT_OK) return rc;
  launch_pdl(sum_parts_steps, dim3((n + 31) / 32), dim3(32), 0, s, (const float*)w.loss_part, per_step, n, loss_t);
  // the gradient entering the top layer at every step of the run, split along K like a single step's
  const int splits = tc::gemm_split_count(false, true, B, H, O, w.split.partial_floats);
  rc = gemm_bf16(dy16, O, false, W_out, H, true, GemmOut{GemmOut::STORE_F32, w.dha_run, H, nullptr, 0}, n * B, H, O,
                 w.status, s, true, &w.split_run, splits);
  return rc;
}

int backward_run_layer(const BwdRunStep* st, int n, int s_lo, int l, int I, const void* Wl, float* dh_rec, float* dc_rec,
                       float* d_lo, int B, int H, size_t plane_elems, int64_t* counters,
                       const Scratch& w, cudaStream_t s) {
  const int K = I + H, G = 4 * H;
  const size_t bh = (size_t)B * H;
  const bf16* W = (const bf16*)Wl;
  const size_t rows = (size_t)w.S * B;
  bf16* dz_l = w.st_dz + (size_t)l * rows * G;
  bf16* in_l = w.st_in + (l == 0 ? 0 : rows * w.I0 + (size_t)(l - 1) * rows * H);
  bf16* hp_l = w.st_hp + (size_t)l * rows * H;
  for (int a = n - 1; a >= 0; --a) {   // time descending
    const size_t row0 = (size_t)(s_lo + a) * B;
    bf16* dz16 = dz_l + row0 * G;
    run_gate_bwd(s, w.dha_run + (size_t)a * bh, dh_rec, dc_rec, (const bf16*)st[a].gates, plane_elems, st[a].c_t,
                 st[a].c_prev, dz16, B, H, counters, (const uint4*)st[a].in, (uint4*)(in_l + row0 * I),
                 (size_t)B * I * 2 / 16, (const uint4*)st[a].h_prev, (uint4*)(hp_l + row0 * H), (size_t)B * H * 2 / 16,
                 w.dh_parts[l]);
    const tc::SplitWs own{w.split_dh + (size_t)l * DH_PART_FLOATS, DH_PART_FLOATS};
    const int rc = gemm_bf16(dz16, G, false, W + I, K, true, GemmOut{GemmOut::STORE_F32, dh_rec, H, nullptr, 0}, B, H, G,
                             w.status, s, true, &own, 0, &w.dh_parts[l]);
    if (rc != MEBPTT_OK) return rc;
  }
  if (!d_lo) return MEBPTT_OK;
  // the gradient w.r.t. the layer's inputs (dx, or what enters the layer below) for the whole run
  const int splits = tc::gemm_split_count(false, true, B, I, G, w.split.partial_floats);
  return gemm_bf16(dz_l + (size_t)s_lo * B * G, G, false, W, K, true, GemmOut{GemmOut::STORE_F32, d_lo, I, nullptr, 0},
                   n * B, I, G, w.status, s, true, &w.split_run, splits);
}

}  // namespace stepwise
}  // namespace mebptt
