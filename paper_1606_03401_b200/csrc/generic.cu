// Shape-agnostic kernels of the recurrent cores (LSTM, and the GRU further down): float32 FMA
// arithmetic on CUDA cores.
//
// This is the path of MEBPTT_FP32 (exact float32 products, which tensor cores do not offer) and
// of every shape the tensor-core kernels do not cover.  Operands are float32 or bfloat16 in
// memory and are widened to float32; all sums are float32 and run in a fixed order (the k loop
// of one thread), so results do not depend on the plan, on the launch order of blocks or on
// the state a forward operation is asked to write.
//
// All contractions go through one tiled kernel, gemm_tiled: a 64 x 64 output tile per block of
// 256 threads, a 4 x 4 micro-tile per thread, K consumed in slices of 16 through shared
// memory.  Operand access and the epilogue are functors, which lets the same kernel serve
//   forward   z[b][4j+q]   = sum_k [in ; h_prev][b][k] W[qH+j][k]      (gates of one unit adjacent)
//   readout   y[b][o]      = sum_j h[b][j] W_out[o][j]
//   dha       dha[b][j]    = sum_o dy[b][o] W_out[o][j]
//   d_in      d_in[b][c]   = sum_g dz[b][g] W[g][c]
//   dW        dW[g][c]    += sum_b dz[b][g] [in ; h_prev][b][c]
//   dW_out    dW_out[o][j]+= sum_b dy[b][o] h[b][j]
#include "kernels.hpp"

#include <cuda_bf16.h>
#include <cuda_runtime.h>

namespace mebptt {
namespace generic {

namespace {

constexpr int TM = 64, TN = 64, TK = 16;

__device__ __forceinline__ float ldf(const float* p, size_t i) { return p[i]; }
__device__ __forceinline__ float ldf(const __nv_bfloat16* p, size_t i) { return __bfloat162float(p[i]); }
__device__ __forceinline__ void stf(float* p, size_t i, float v) { p[i] = v; }
__device__ __forceinline__ void stf(__nv_bfloat16* p, size_t i, float v) { p[i] = __float2bfloat16_rn(v); }

__device__ __forceinline__ float sigmoidf_(float a) { return 1.0f / (1.0f + expf(-a)); }

// AK / BK: true when the operand is contiguous along k (threads then walk k fastest).
template <bool AK, bool BK, bool REDUCE, class FA, class FB, class Epi>
__global__ void __launch_bounds__(256) gemm_tiled(int M, int N, int K, FA fa, FB fb, Epi epi) {
  __shared__ float As[TK][TM + 4];
  __shared__ float Bs[TK][TN + 4];
  __shared__ float red[256];
  const int tid = threadIdx.x;
  const int tx = tid % 16, ty = tid / 16;
  const int m0 = blockIdx.y * TM, n0 = blockIdx.x * TN;
  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

  for (int k0 = 0; k0 < K; k0 += TK) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int idx = tid + i * 256;
      int m, k;
      if (AK) { m = idx / TK; k = idx % TK; } else { k = idx / TM; m = idx % TM; }
      const int gm = m0 + m, gk = k0 + k;
      As[k][m] = (gm < M && gk < K) ? fa(gm, gk) : 0.f;
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int idx = tid + i * 256;
      int n, k;
      if (BK) { n = idx / TK; k = idx % TK; } else { k = idx / TN; n = idx % TN; }
      const int gn = n0 + n, gk = k0 + k;
      Bs[k][n] = (gn < N && gk < K) ? fb(gk, gn) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < TK; ++kk) {
      float a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = As[kk][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) b[j] = Bs[kk][tx * 4 + j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
  const float part = epi(acc, m0 + ty * 4, n0 + tx * 4, M, N);
  if (REDUCE) {
    // fixed-order tree over the block, then one value per block
    red[tid] = part;
    __syncthreads();
    for (int s = 128; s > 0; s >>= 1) {
      if (tid < s) red[tid] += red[tid + s];
      __syncthreads();
    }
    if (tid == 0) epi.block_result(red[0], blockIdx.y * gridDim.x + blockIdx.x);
  }
}

// ------------------------------------------------------------------ forward
template <class T>
struct FwdA {  // [in ; h_prev][b][k]
  const T* in; const T* h_prev; int I, H;
  __device__ float operator()(int b, int k) const {
    return k < I ? ldf(in, (size_t)b * I + k) : ldf(h_prev, (size_t)b * H + (k - I));
  }
};
template <class T>
struct FwdB {  // column n = 4 j + q  <->  weight row q H + j
  const T* W; int H, K;
  __device__ float operator()(int k, int n) const {
    const int j = n >> 2, q = n & 3;
    return ldf(W, (size_t)(q * H + j) * K + k);
  }
};
template <class T>
struct FwdEpi {
  const float* bias; const float* c_prev; const T* h_prev;
  T* h_out; float* c_out; T* gates; T* h_in_copy; float* c_in_copy;
  int B, H; size_t plane;  // plane: elements between gate planes
  int64_t* counters;
  __device__ float operator()(float (&acc)[4][4], int b0, int n0, int M, int N) const {
    const int j = n0 >> 2;
    if (j < H) {
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        const int b = b0 + r;
        if (b >= B) break;
        const size_t e = (size_t)b * H + j;
        const float gi = sigmoidf_(acc[r][0] + bias[0 * H + j]);
        const float gf = sigmoidf_(acc[r][1] + bias[1 * H + j]);
        const float gg = tanhf(acc[r][2] + bias[2 * H + j]);
        const float go = sigmoidf_(acc[r][3] + bias[3 * H + j]);
        const float cp = c_prev[e];
        const float c = fmaf(gf, cp, gi * gg);
        const float h = go * tanhf(c);
        c_out[e] = c;
        stf(h_out, e, h);
        if (gates) {
          stf(gates, 0 * plane + e, gi);
          stf(gates, 1 * plane + e, gf);
          stf(gates, 2 * plane + e, gg);
          stf(gates, 3 * plane + e, go);
        }
        if (h_in_copy) { h_in_copy[e] = h_prev[e]; c_in_copy[e] = cp; }
      }
    }
    if (counters && blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) counters[0] += 1;
    return 0.f;
  }
  __device__ void block_result(float, int) const {}
};

// ------------------------------------------------------------------ readout, loss, dy
template <class T>
struct RoA { const T* h; int H; __device__ float operator()(int b, int k) const { return ldf(h, (size_t)b * H + k); } };
template <class T>
struct RoB { const T* W_out; int H; __device__ float operator()(int k, int o) const { return ldf(W_out, (size_t)o * H + k); } };
struct RoEpi {
  const float* b_out; const float* target; float* dy; float* loss_part; int B, O; float inv;
  __device__ float operator()(float (&acc)[4][4], int b0, int o0, int M, int N) const {
    float s = 0.f;
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const int b = b0 + r, o = o0 + c;
        if (b < B && o < O) {
          const float d = acc[r][c] + b_out[o] - target[(size_t)b * O + o];
          dy[(size_t)b * O + o] = 2.f * d * inv;
          s = fmaf(d, d, s);
        }
      }
    return s;
  }
  __device__ void block_result(float v, int blk) const { loss_part[blk] = v; }
};

// dha[b][j] = sum_o dy[b][o] W_out[o][j]
struct DyA { const float* dy; int O; __device__ float operator()(int b, int o) const { return dy[(size_t)b * O + o]; } };
template <class T>
struct WoutB { const T* W_out; int H; __device__ float operator()(int o, int j) const { return ldf(W_out, (size_t)o * H + j); } };
struct StoreEpi {
  float* out; int ld;
  __device__ float operator()(float (&acc)[4][4], int m0, int n0, int M, int N) const {
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
      for (int c = 0; c < 4; ++c)
        if (m0 + r < M && n0 + c < N) out[(size_t)(m0 + r) * ld + n0 + c] = acc[r][c];
    return 0.f;
  }
  __device__ void block_result(float, int) const {}
};
struct AccumEpi {
  float* out; int ld;
  __device__ float operator()(float (&acc)[4][4], int m0, int n0, int M, int N) const {
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
      for (int c = 0; c < 4; ++c)
        if (m0 + r < M && n0 + c < N) out[(size_t)(m0 + r) * ld + n0 + c] += acc[r][c];
    return 0.f;
  }
  __device__ void block_result(float, int) const {}
};

// dW_out[o][j] += sum_b dy[b][o] h[b][j]
struct DyTA { const float* dy; int O; __device__ float operator()(int o, int b) const { return dy[(size_t)b * O + o]; } };
template <class T>
struct HB { const T* h; int H; __device__ float operator()(int b, int j) const { return ldf(h, (size_t)b * H + j); } };

// d_in[b][c] = sum_g dz[b][g] W[g][c]; columns < I go to `lo` (dx or the layer below), the rest to dh
struct DzA { const float* dz; int G; __device__ float operator()(int b, int g) const { return dz[(size_t)b * G + g]; } };
template <class T>
struct WB { const T* W; int K; __device__ float operator()(int g, int c) const { return ldf(W, (size_t)g * K + c); } };
struct DinEpi {
  float* lo; int I; float* dh; int H;
  __device__ float operator()(float (&acc)[4][4], int b0, int c0, int M, int N) const {
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const int b = b0 + r, col = c0 + c;
        if (b < M && col < N) {
          if (col < I) { if (lo) lo[(size_t)b * I + col] = acc[r][c]; }
          else dh[(size_t)b * H + (col - I)] = acc[r][c];
        }
      }
    return 0.f;
  }
  __device__ void block_result(float, int) const {}
};

// dW[g][c] += sum_b dz[b][g] [in ; h_prev][b][c]
struct DzTA { const float* dz; int G; __device__ float operator()(int g, int b) const { return dz[(size_t)b * G + g]; } };
template <class T>
struct InB {
  const T* in; const T* h_prev; int I, H;
  __device__ float operator()(int b, int c) const {
    return c < I ? ldf(in, (size_t)b * I + c) : ldf(h_prev, (size_t)b * H + (c - I));
  }
};

// ------------------------------------------------------------------ element-wise kernels
// Gate derivatives of one layer at one step.  dh = dha + dh_rec; writes dz [B][4H] (gate-major
// columns q H + j) and dc_rec = dc * f.
template <class T>
__global__ void gate_bwd(const float* dha, const float* dh_rec, float* dc_rec, const T* gates, size_t plane,
                         const float* c_t, const float* c_prev, float* dz, int B, int H, int64_t* counters) {
  const size_t n = (size_t)B * H;
  for (size_t e = blockIdx.x * (size_t)blockDim.x + threadIdx.x; e < n; e += (size_t)gridDim.x * blockDim.x) {
    const int b = (int)(e / H), j = (int)(e % H);
    const float gi = ldf(gates, 0 * plane + e), gf = ldf(gates, 1 * plane + e);
    const float gg = ldf(gates, 2 * plane + e), go = ldf(gates, 3 * plane + e);
    const float dh = dha[e] + dh_rec[e];
    const float th = tanhf(c_t[e]);
    const float d_o = dh * th;
    const float dc = fmaf(dh * go, 1.f - th * th, dc_rec[e]);
    const float di = dc * gg, df = dc * c_prev[e], dg = dc * gi;
    float* row = dz + (size_t)b * 4 * H;
    row[0 * H + j] = di * gi * (1.f - gi);
    row[1 * H + j] = df * gf * (1.f - gf);
    row[2 * H + j] = dg * (1.f - gg * gg);
    row[3 * H + j] = d_o * go * (1.f - go);
    dc_rec[e] = dc * gf;
  }
  if (counters && blockIdx.x == 0 && threadIdx.x == 0) counters[1] += 1;
}

// out[n] += sum_b v[b][n], b ascending
__global__ void colsum_accum(const float* v, int B, int N, float* out) {
  const int n = blockIdx.x * blockDim.x + threadIdx.x;
  if (n >= N) return;
  float s = 0.f;
  for (int b = 0; b < B; ++b) s += v[(size_t)b * N + n];
  out[n] += s;
}

__global__ void sum_partials(const float* part, int n, float scale, float* out) {
  if (threadIdx.x == 0 && blockIdx.x == 0) {
    float s = 0.f;
    for (int i = 0; i < n; ++i) s += part[i];
    *out = s * scale;
  }
}

// loss = sum_t loss_t in ascending t by one warp (lane-strided partials, then a fixed tree)
__global__ void finalize(const float* loss_t, int64_t t, float* loss, int64_t* counters, int64_t peak_units,
                         const int* status) {
  float s = 0.f;
  for (int64_t i = threadIdx.x; i < t; i += 32) s += loss_t[i];
  for (int o = 16; o > 0; o >>= 1) s += __shfl_down_sync(0xffffffffu, s, o);
  if (threadIdx.x == 0) {
    *loss = s;
    counters[2] = peak_units;
    counters[3] = *status;
  }
}

inline dim3 tiles(int M, int N) { return dim3((N + TN - 1) / TN, (M + TM - 1) / TM); }

// ------------------------------------------------------------------ the GRU core
// r = sigmoid(W_r [x ; h] + b_r), z = sigmoid(W_z [x ; h] + b_z), q = W_hn h,
// n = tanh(W_xn x + b_n + r q), h' = (1 - z) n + z h.  The forward contraction keeps the layout of
// the LSTM one -- four adjacent columns per hidden unit -- with the columns r, z, the input part of
// n and its recurrent part q; the four planes of an internal state hold r, z, n, q.  The hidden
// state is h alone (the cell-state part of a slot stays unused).
template <class T>
struct GruFwdB {  // column 4 j + c: c = 0, 1 -> weight rows c H + j; c = 2 -> row 2H + j over the input columns, c = 3 over the recurrent ones
  const T* W; int H, K, I;
  __device__ float operator()(int k, int n) const {
    const int j = n >> 2, c = n & 3;
    if (c < 2) return ldf(W, (size_t)(c * H + j) * K + k);
    return ((c == 2) == (k < I)) ? ldf(W, (size_t)(2 * H + j) * K + k) : 0.f;
  }
};
template <class T>
struct GruFwdEpi {
  const float* bias; const T* h_prev; T* h_out; T* gates; T* h_in_copy;
  int B, H; size_t plane;
  int64_t* counters;
  __device__ float operator()(float (&acc)[4][4], int b0, int n0, int M, int N) const {
    const int j = n0 >> 2;
    if (j < H) {
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        const int b = b0 + r;
        if (b >= B) break;
        const size_t e = (size_t)b * H + j;
        const float gr = sigmoidf_(acc[r][0] + bias[0 * H + j]);
        const float gz = sigmoidf_(acc[r][1] + bias[1 * H + j]);
        const float q = acc[r][3];
        const float gn = tanhf(fmaf(gr, q, acc[r][2] + bias[2 * H + j]));
        const float hp = ldf(h_prev, e);
        stf(h_out, e, fmaf(gz, hp - gn, gn));   // (1 - z) n + z h
        if (gates) {
          stf(gates, 0 * plane + e, gr);
          stf(gates, 1 * plane + e, gz);
          stf(gates, 2 * plane + e, gn);
          stf(gates, 3 * plane + e, q);
        }
        if (h_in_copy) h_in_copy[e] = h_prev[e];
      }
    }
    if (counters && blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) counters[0] += 1;
    return 0.f;
  }
  __device__ void block_result(float, int) const {}
};
// Gate derivatives.  dz4 [B][4H], column blocks: d r_pre, d z_pre, d n_pre, d q; dhz = dh z is the
// part of the gradient that reaches h_{k-1} past the gates.
template <class T>
__global__ void gru_gate_bwd(const float* dha, const float* dh_rec, float* dhz, const T* gates, size_t plane,
                             const T* h_prev, float* dz4, int B, int H, int64_t* counters) {
  const size_t n = (size_t)B * H;
  for (size_t e = blockIdx.x * (size_t)blockDim.x + threadIdx.x; e < n; e += (size_t)gridDim.x * blockDim.x) {
    const int b = (int)(e / H), j = (int)(e % H);
    const float gr = ldf(gates, 0 * plane + e), gz = ldf(gates, 1 * plane + e);
    const float gn = ldf(gates, 2 * plane + e), q = ldf(gates, 3 * plane + e);
    const float dh = dha[e] + dh_rec[e];
    const float dn_pre = dh * (1.f - gz) * (1.f - gn * gn);
    const float dz_pre = dh * (ldf(h_prev, e) - gn) * gz * (1.f - gz);
    float* row = dz4 + (size_t)b * 4 * H;
    row[0 * H + j] = dn_pre * q * gr * (1.f - gr);
    row[1 * H + j] = dz_pre;
    row[2 * H + j] = dn_pre;
    row[3 * H + j] = dn_pre * gr;
    dhz[e] = dh * gz;
  }
  if (counters && blockIdx.x == 0 && threadIdx.x == 0) counters[1] += 1;
}
// the [4H][K] matrix dz4 is contracted against: rows c H + j of W for c = 0, 1; row 2H + j over the
// input columns for c = 2 and over the recurrent columns for c = 3.  col0: first column asked for.
template <class T>
struct GruWB {
  const T* W; int H, K, I, col0;
  __device__ float operator()(int g, int c) const {
    const int blk = g / H, j = g - blk * H, col = c + col0;
    if (blk < 2) return ldf(W, (size_t)(blk * H + j) * K + col);
    return ((blk == 2) == (col < I)) ? ldf(W, (size_t)(2 * H + j) * K + col) : 0.f;
  }
};
// like DinEpi, plus the part of dh that bypasses the gates
struct GruDinEpi {
  float* lo; int I; float* dh; int H; const float* dhz;
  __device__ float operator()(float (&acc)[4][4], int b0, int c0, int M, int N) const {
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const int b = b0 + r, col = c0 + c;
        if (b < M && col < N) {
          if (col < I) { if (lo) lo[(size_t)b * I + col] = acc[r][c]; }
          else dh[(size_t)b * H + (col - I)] = acc[r][c] + dhz[(size_t)b * H + (col - I)];
        }
      }
    return 0.f;
  }
  __device__ void block_result(float, int) const {}
};
// out[n] += sum_b v[b][n] over the first N columns of rows that are `ld` apart, b ascending
__global__ void colsum_accum_ld(const float* v, int B, int N, int ld, float* out) {
  const int n = blockIdx.x * blockDim.x + threadIdx.x;
  if (n >= N) return;
  float s = 0.f;
  for (int b = 0; b < B; ++b) s += v[(size_t)b * ld + n];
  out[n] += s;
}

template <class T>
void gru_forward_step_t(const FwdArgs& a, cudaStream_t s) {
  const int K = a.I + a.H;
  FwdA<T> fa{(const T*)a.in, (const T*)a.h_prev, a.I, a.H};
  GruFwdB<T> fb{(const T*)a.W, a.H, K, a.I};
  GruFwdEpi<T> epi{a.bias, (const T*)a.h_prev, (T*)a.h_out, (T*)a.gates, (T*)a.h_in_copy, a.B, a.H, a.plane_elems,
                   a.counters};
  gemm_tiled<true, true, false><<<tiles(a.B, 4 * a.H), 256, 0, s>>>(a.B, 4 * a.H, K, fa, fb, epi);
}

template <class T>
void gru_backward_layer_t(const BwdArgs& a, cudaStream_t s) {
  const int K = a.I + a.H, H = a.H, G4 = 4 * a.H;
  const size_t n = (size_t)a.B * a.H;
  const int blocks = (int)((n + 255) / 256 > 1184 ? 1184 : (n + 255) / 256);
  float* dhz = a.dc_rec;   // a GRU carries no cell-state gradient: the buffer holds dh z for this step
  gru_gate_bwd<T><<<blocks, 256, 0, s>>>(a.dha, a.dh_rec, dhz, (const T*)a.gates, a.plane_elems, (const T*)a.h_prev,
                                          a.dz, a.B, a.H, a.counters);
  // dW: the rows of r and z against [in ; h_prev]; the rows of n against in (d n_pre) and h_prev (d q)
  gemm_tiled<false, false, false><<<tiles(2 * H, K), 256, 0, s>>>(2 * H, K, a.B, DzTA{a.dz, G4},
                                                                   InB<T>{(const T*)a.in, (const T*)a.h_prev, a.I, a.H},
                                                                   AccumEpi{a.dW, K});
  gemm_tiled<false, false, false><<<tiles(H, a.I), 256, 0, s>>>(H, a.I, a.B, DzTA{a.dz + 2 * H, G4},
                                                                 HB<T>{(const T*)a.in, a.I},
                                                                 AccumEpi{a.dW + (size_t)2 * H * K, K});
  gemm_tiled<false, false, false><<<tiles(H, H), 256, 0, s>>>(H, H, a.B, DzTA{a.dz + 3 * H, G4},
                                                               HB<T>{(const T*)a.h_prev, a.H},
                                                               AccumEpi{a.dW + (size_t)2 * H * K + a.I, K});
  colsum_accum_ld<<<(3 * H + 127) / 128, 128, 0, s>>>(a.dz, a.B, 3 * H, G4, a.db);
  // d_in = dz4 against the expanded weights, plus dh z on the recurrent columns
  if (a.d_lo) {
    gemm_tiled<true, false, false><<<tiles(a.B, K), 256, 0, s>>>(a.B, K, G4, DzA{a.dz, G4},
                                                                  GruWB<T>{(const T*)a.W, H, K, a.I, 0},
                                                                  GruDinEpi{a.d_lo, a.I, a.dh_rec, a.H, dhz});
  } else {
    gemm_tiled<true, false, false><<<tiles(a.B, H), 256, 0, s>>>(a.B, H, G4, DzA{a.dz, G4},
                                                                  GruWB<T>{(const T*)a.W, H, K, a.I, a.I},
                                                                  GruDinEpi{nullptr, 0, a.dh_rec, a.H, dhz});
  }
}

template <class T>
void forward_step_t(const FwdArgs& a, cudaStream_t s) {
  const int K = a.I + a.H;
  FwdA<T> fa{(const T*)a.in, (const T*)a.h_prev, a.I, a.H};
  FwdB<T> fb{(const T*)a.W, a.H, K};
  FwdEpi<T> epi{a.bias, a.c_prev, (const T*)a.h_prev, (T*)a.h_out, a.c_out, (T*)a.gates,
                (T*)a.h_in_copy, a.c_in_copy, a.B, a.H, a.plane_elems, a.counters};
  gemm_tiled<true, true, false><<<tiles(a.B, 4 * a.H), 256, 0, s>>>(a.B, 4 * a.H, K, fa, fb, epi);
}

template <class T>
void readout_t(const ReadoutArgs& a, cudaStream_t s) {
  RoA<T> fa{(const T*)a.h, a.H};
  RoB<T> fb{(const T*)a.W_out, a.H};
  RoEpi epi{a.b_out, a.target, a.dy, a.loss_part, a.B, a.O, 1.f / ((float)a.B * (float)a.O)};
  gemm_tiled<true, true, true><<<tiles(a.B, a.O), 256, 0, s>>>(a.B, a.O, a.H, fa, fb, epi);
  sum_partials<<<1, 32, 0, s>>>(a.loss_part, a.n_loss_part, 1.f / ((float)a.B * (float)a.O), a.loss_k);
  // dha = dy W_out
  gemm_tiled<true, false, false><<<tiles(a.B, a.H), 256, 0, s>>>(a.B, a.H, a.O, DyA{a.dy, a.O},
                                                                  WoutB<T>{(const T*)a.W_out, a.H},
                                                                  StoreEpi{a.dha, a.H});
  // dW_out += dy^T h ; db_out += sum_b dy
  gemm_tiled<false, false, false><<<tiles(a.O, a.H), 256, 0, s>>>(a.O, a.H, a.B, DyTA{a.dy, a.O},
                                                                   HB<T>{(const T*)a.h, a.H},
                                                                   AccumEpi{a.dW_out, a.H});
  colsum_accum<<<(a.O + 127) / 128, 128, 0, s>>>(a.dy, a.B, a.O, a.db_out);
}

template <class T>
void backward_layer_t(const BwdArgs& a, cudaStream_t s) {
  const int K = a.I + a.H, G = 4 * a.H;
  const size_t n = (size_t)a.B * a.H;
  const int blocks = (int)((n + 255) / 256 > 1184 ? 1184 : (n + 255) / 256);
  gate_bwd<T><<<blocks, 256, 0, s>>>(a.dha, a.dh_rec, a.dc_rec, (const T*)a.gates, a.plane_elems, a.c_t,
                                      a.c_prev, a.dz, a.B, a.H, a.counters);
  // dW += dz^T [in ; h_prev] ; db += sum_b dz     (uses h_prev before dh_rec is replaced)
  gemm_tiled<false, false, false><<<tiles(G, K), 256, 0, s>>>(G, K, a.B, DzTA{a.dz, G},
                                                               InB<T>{(const T*)a.in, (const T*)a.h_prev, a.I, a.H},
                                                               AccumEpi{a.dW, K});
  colsum_accum<<<(G + 127) / 128, 128, 0, s>>>(a.dz, a.B, G, a.db);
  // d_in = dz W : columns < I feed dx or the layer below, the rest is the new dh_rec
  if (a.d_lo) {
    gemm_tiled<true, false, false><<<tiles(a.B, K), 256, 0, s>>>(a.B, K, G, DzA{a.dz, G}, WB<T>{(const T*)a.W, K},
                                                                  DinEpi{a.d_lo, a.I, a.dh_rec, a.H});
  } else {
    // only the recurrent columns are needed: contract against W[:, I:]
    gemm_tiled<true, false, false><<<tiles(a.B, a.H), 256, 0, s>>>(a.B, a.H, G, DzA{a.dz, G},
                                                                    WB<T>{(const T*)a.W + a.I, K},
                                                                    DinEpi{nullptr, 0, a.dh_rec, a.H});
  }
}

}  // namespace

void forward_step(int dtype, const FwdArgs& a, cudaStream_t s) {
  if (dtype == MEBPTT_BF16) forward_step_t<__nv_bfloat16>(a, s);
  else forward_step_t<float>(a, s);
}
void readout(int dtype, const ReadoutArgs& a, cudaStream_t s) {
  if (dtype == MEBPTT_BF16) readout_t<__nv_bfloat16>(a, s);
  else readout_t<float>(a, s);
}
void backward_layer(int dtype, const BwdArgs& a, cudaStream_t s) {
  if (dtype == MEBPTT_BF16) backward_layer_t<__nv_bfloat16>(a, s);
  else backward_layer_t<float>(a, s);
}
void gru_forward_step(int dtype, const FwdArgs& a, cudaStream_t s) {
  if (dtype == MEBPTT_BF16) gru_forward_step_t<__nv_bfloat16>(a, s);
  else gru_forward_step_t<float>(a, s);
}
void gru_backward_layer(int dtype, const BwdArgs& a, cudaStream_t s) {
  if (dtype == MEBPTT_BF16) gru_backward_layer_t<__nv_bfloat16>(a, s);
  else gru_backward_layer_t<float>(a, s);
}
void finalize_step(const float* loss_t, int64_t t, float* loss, int64_t* counters, int64_t peak_units,
                   const int* status, cudaStream_t s) {
  finalize<<<1, 32, 0, s>>>(loss_t, t, loss, counters, peak_units, status);
}
}  // namespace generic
}  // namespace mebptt
