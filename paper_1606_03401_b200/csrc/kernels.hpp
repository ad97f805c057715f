// Host-callable launchers of the device kernels (declarations shared by the executor).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstddef>
#include <cstdint>

#include "mebptt.h"
#include "tc.hpp"

namespace mebptt {
namespace generic {

// One forward operation of one layer: state k-1 -> state k.
struct FwdArgs {
  const void* in;        // [B][I] operand type: x_k or the h_k of the layer below
  const void* h_prev;    // [B][H] operand type
  const float* c_prev;   // [B][H]
  const void* W;         // [4H][I + H] operand type
  const float* bias;     // [4H]
  void* h_out;           // [B][H] operand type
  float* c_out;          // [B][H]
  void* gates;           // four planes [B][H] operand type, or NULL (hidden-state format)
  void* h_in_copy;       // copy of h_prev for the internal state, or NULL
  float* c_in_copy;      // copy of c_prev (non-NULL iff h_in_copy is)
  size_t plane_elems;    // elements between gate planes
  int B, I, H;
  int64_t* counters;     // NULL for all but the first layer
};

// Readout, loss term and output gradient of step k, plus their parameter gradients.
struct ReadoutArgs {
  const void* h;         // [B][H] top layer h_k
  const void* W_out;     // [O][H]
  const float* b_out;    // [O]
  const float* target;   // [B][O]
  float* dy;             // [B][O] scratch
  float* loss_part;      // scratch, n_loss_part values
  int n_loss_part;
  float* loss_k;         // loss term of this step
  float* dha;            // [B][H]: dy W_out, the gradient entering the top layer
  float* dW_out;         // [O][H] accumulated
  float* db_out;         // [O] accumulated
  int B, H, O;
};

// One backward operation of one layer.
struct BwdArgs {
  const float* dha;      // [B][H] gradient from above (readout or the layer above)
  float* dh_rec;         // [B][H] in: gradient from step k+1; out: gradient for step k-1
  float* dc_rec;         // [B][H] likewise for c
  const void* gates;     // four planes
  size_t plane_elems;
  const float* c_t;      // [B][H]
  const float* c_prev;   // [B][H]
  const void* in;        // [B][I] input of this layer at step k
  const void* h_prev;    // [B][H]
  const void* W;         // [4H][I + H]
  float* dz;             // [B][4H] scratch
  float* dW;             // [4H][I + H] accumulated
  float* db;             // [4H] accumulated
  float* d_lo;           // [B][I]: gradient w.r.t. `in` (dx_k or the dha of the layer below), or NULL
  int B, I, H;
  int64_t* counters;     // NULL for all but the top layer
};

void forward_step(int dtype, const FwdArgs& a, cudaStream_t s);
void readout(int dtype, const ReadoutArgs& a, cudaStream_t s);
void backward_layer(int dtype, const BwdArgs& a, cudaStream_t s);
// The same two operations for the GRU core (W is [3H][I + H], gate blocks r, z, n; bias [3H]; the four
// planes of an internal state hold r, z, n and q = W_hn h; c_prev / c_out / c_t are not used and dc_rec
// serves as scratch).
void gru_forward_step(int dtype, const FwdArgs& a, cudaStream_t s);
void gru_backward_layer(int dtype, const BwdArgs& a, cudaStream_t s);
// status: device word whose value goes to counters[3]
void finalize_step(const float* loss_t, int64_t t, float* loss, int64_t* counters, int64_t peak_units,
                   const int* status, cudaStream_t s);
void copy_bytes(void* dst, const void* src, size_t bytes, cudaStream_t s);

}  // namespace generic

// The same three operations with their contractions on the tensor cores (bfloat16 storage,
// dimensions that are multiples of 8, B a multiple of 32).  Each returns a status.
// Floats of split-K scratch for one step's dh = dz W_hh of one layer: a wave of 128 x 128 tiles.
constexpr size_t DH_PART_FLOATS = (size_t)148 * 128 * 128;

namespace stepwise {
struct Scratch {
  float* z;                 // [B][4H] pre-activations of the forward operation in flight
  int* status;              // device word that receives MEBPTT_ERR_TIMEOUT from a bounded wait
  tc::SplitWs split;        // scratch of the contractions that are split along K
  // stages of one chunk of S time steps, row block (k - 1) % S of B rows per step
  int S, I0;                // I0: input width of the first layer
  __nv_bfloat16* st_dz;     // [L][S B][4H]
  __nv_bfloat16* st_in;     // layer 0: [S B][I0]; layers l > 0: [S B][H] each, after it
  __nv_bfloat16* st_hp;     // [L][S B][H]  h_{k-1}
  __nv_bfloat16* st_dy;     // [S B][O]
  __nv_bfloat16* st_h;      // [S B][H]  top layer h_k
  // a run of up to S operations, one layer at a time
  float* zrun;              // [S B][4H] pre-activations of the run's steps
  __nv_bfloat16* hrun;      // [S B][H]  the layer's h_k, read by the layer above
  float* dha_run;           // [S B][H]  gradient entering the layer at each step (row block: step - first step)
  float* loss_part;         // partial sums of the loss terms, per step
  // the recurrent gradient dh = dz W_hh of a layer is consumed only by the layer's next gate
  // kernel: where that contraction is split along K, the gate kernel adds the parts itself
  float* split_dh;          // [L][DH_PART_FLOATS] split-K scratch of that product, one per layer
  tc::SplitParts* dh_parts; // host, [L]: where each layer's latest dh lies (updated by every backward operation)
  tc::SplitWs split_run;    // split-K scratch for a product over all rows of a run
};
int forward_step(const generic::FwdArgs& a, const Scratch& w, cudaStream_t s);
// sidx: row block of this step in the stages; l: layer
int readout(const generic::ReadoutArgs& a, const Scratch& w, int sidx, cudaStream_t s);
int backward_layer(const generic::BwdArgs& a, const Scratch& w, int l, int sidx, cudaStream_t s);
// dW (w_off[l]: element offset of layer l), db ([L][4H]), dW_out and db_out from the first `steps` row blocks of the stages
int flush_chunk(const Scratch& w, int steps, int L, int B, int I0, int H, int O, const size_t* w_off, float* dW,
                float* dW_out, float* db, float* db_out, cudaStream_t s);

// One step of a run, as one layer sees it.
struct FwdRunStep {
  const void* h_prev; const float* c_prev;     // state k-1 of the layer
  void* h_out; float* c_out;                   // where state k goes
  void* gates; void* h_in_copy; float* c_in_copy;   // as in FwdArgs
};
struct BwdRunStep {
  const void* gates; const float* c_t; const float* c_prev; const void* in; const void* h_prev;   // as in BwdArgs
};
// n consecutive forward operations of one layer.  in: the layer's inputs of all n steps, [n B][I]
// (x, or w.hrun as the layer below left it); stage_h: leave the layer's h_k in w.hrun.
int forward_run_layer(const FwdRunStep* st, int n, const void* in, int I, const void* W, const float* bias, bool stage_h,
                      int B, int H, size_t plane_elems, int64_t* counters, const Scratch& w, cudaStream_t s);
// Readout, loss terms, dy and the gradient entering the top layer (-> w.dha_run) for the n steps
// whose stages are the row blocks s_lo .. s_lo + n - 1; h_top[a]: the top layer's h of step s_lo + a;
// target, loss_t: those of the first of the steps.
int readout_run(const void* const* h_top, int n, int s_lo, const void* W_out, const float* b_out, const float* target,
                float* loss_t, int B, int H, int O, const Scratch& w, cudaStream_t s);
// The n backward operations of layer l, time descending (st[a]: step s_lo + a), reading w.dha_run;
// d_lo (nullable): [n B][I] gradient w.r.t. the layer's inputs, written once for the whole run.
int backward_run_layer(const BwdRunStep* st, int n, int s_lo, int l, int I, const void* W, float* dh_rec, float* dc_rec,
                       float* d_lo, int B, int H, size_t plane_elems, int64_t* counters,
                       const Scratch& w, cudaStream_t s);
}  // namespace stepwise

// The same for float32 storage (MEBPTT_TF32): operands split into two bfloat16 halves, three
// bfloat16 products per float32 product.
namespace stepwise3 {
struct Scratch {
  float* z;                  // [B][4H]
  int* status;
  tc::SplitWs split;
  int S, I0;
  __nv_bfloat16* a3;         // [B][3 (I + H)]: the forward operation's left operand
  __nv_bfloat16* w3;         // per layer at 3 * (element offset of the layer): [4H][3K], [hi | mid | hi]
  __nv_bfloat16* wmn3;       // likewise [3 * 4H][K], [hi ; mid ; hi]
  __nv_bfloat16* wout3;      // [O][3H]
  __nv_bfloat16* woutmn3;    // [3 O][H]
  // stages of one chunk of S steps, row block (k - 1) % S of B rows per step
  __nv_bfloat16* st_dz3;     // [L][S B][3 * 4H]  [hi | hi | mid]
  __nv_bfloat16* st_in2;     // layer 0: [S B][2 I0]; layers l > 0: [S B][2H] each, after it; [hi | mid]
  __nv_bfloat16* st_hp2;     // [L][S B][2H]
  __nv_bfloat16* st_dy3;     // [S B][3 O]
  __nv_bfloat16* st_h3;      // [S B][3 H]  top layer h_k
  // the readout of a run of up to S backward operations at once
  float* dy_run;             // [S B][O]
  float* dha_run;            // [S B][H]  gradient entering the top layer at each step of the run
  float* loss_part;          // partial sums of the loss terms, per step
  float* split_dh;           // as on the bfloat16 path: per-layer split-K scratch of dh = dz W_hh,
  tc::SplitParts* dh_parts;  // and where each layer's latest dh lies (host, [L])
  tc::SplitWs split_run;     // split-K scratch for a product over all rows of a run
  __nv_bfloat16* a3_run;     // [S][B][3 (I + H)]: left operands of a run of forward operations
  float* h_run;              // [S][B][H]: a layer's h_k of a run, the inputs of the layer above
};
// W: all layers' weights (float32), w_off[l] the element offset of layer l
void pack_weights(const Scratch& w, int L, int I0, int H, int O, const float* W, const size_t* w_off,
                  const float* W_out, cudaStream_t s);
int forward_step(const generic::FwdArgs& a, const Scratch& w, int l, size_t w_off, cudaStream_t s);
int readout(const generic::ReadoutArgs& a, const Scratch& w, int sidx, cudaStream_t s);
int backward_layer(const generic::BwdArgs& a, const Scratch& w, int l, size_t w_off, int sidx, cudaStream_t s);
// Readout, loss terms, dy and the gradient entering the top layer (-> w.dha_run, row block a for
// step s_lo + a) of n steps at once; h_top[a]: the top layer's h of step s_lo + a; target, loss_t:
// those of the first of the steps.
int readout_run(const float* const* h_top, int n, int s_lo, const float* b_out, const float* target, float* loss_t,
                int B, int H, int O, const Scratch& w, cudaStream_t s);
int flush_chunk(const Scratch& w, int steps, int L, int B, int I0, int H, int O, const size_t* w_off, float* dW,
                float* dW_out, float* db, float* db_out, cudaStream_t s);
// n consecutive forward operations of one layer (st as on the bfloat16 path).  in: the layer's input
// of the first step, the others in_step_stride floats apart; h_stage (nullable): [n][B][H] copy of
// the layer's h_k for the layer above.
int forward_run_layer(const stepwise::FwdRunStep* st, int n, const float* in, int64_t in_step_stride, int I,
                      const float* bias, int B, int H, size_t plane_elems, int64_t* counters, const Scratch& w,
                      size_t w_off, float* h_stage, cudaStream_t s);
}  // namespace stepwise3
}  // namespace mebptt
