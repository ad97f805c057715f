// Device memory layout of hidden states, internal states and the workspace.
//
// A hidden state (Definition 2) of the stack is, per layer, h (operand type) followed by c
// (float32).  An internal state (Definition 3) is the output hidden state, the four gate
// planes i, f, g, o of every layer (operand type, each [B][H]) and a copy of the input hidden
// state.  The output hidden state comes first, so that a forward operation can read "the hidden
// state at a location" without knowing which of the two formats the location holds.
//
// Every block starts at a multiple of `granule` = lcm(256, H * element size) bytes from the
// workspace base: the tensor-core path addresses h blocks through one TMA tensor map that views
// the whole workspace as rows of H elements, so a block's offset must be a whole number of rows.
#pragma once

#include <cstddef>
#include <cstdint>
#include <vector>

#include "mebptt.h"
#include "plan.hpp"

namespace mebptt {

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
inline size_t gcd_sz(size_t a, size_t b) { while (b) { size_t r = a % b; a = b; b = r; } return a; }

struct Layout {
  int L = 0, I = 0, H = 0, O = 0, B = 0;
  int dtype = 0;
  int64_t t = 0;
  bool tensor_path = false;
  bool stepwise_tc = false;   // step-by-step operations with their contractions on the tensor cores
  bool stepwise_x3 = false;   // likewise for float32 storage, operands split into bfloat16 halves
  bool gru = false;           // the core is a GRU (CUDA-core kernels)
  int NG = 4;                 // row blocks of H rows in a layer's weight matrix and bias: 4 (LSTM) or 3 (GRU)
  size_t esz = 0;        // bytes of one operand element
  size_t granule = 0;
  size_t hsz = 0;        // one layer's h
  size_t csz = 0;        // one layer's c
  size_t gsz = 0;        // one layer's four gate planes
  size_t plane = 0;      // one gate plane
  size_t unit = 0;       // one hidden state of the stack
  size_t loc_bytes = 0;  // what one unit of a tape location (and of the plan's budget m) is in bytes: unit / sigma
  size_t rec = 0;        // one internal state
  // record-relative offsets
  size_t rec_gates = 0;  // gates of layer 0
  size_t rec_in = 0;     // input hidden state
  // workspace offsets: states
  size_t off_arena = 0, off_core = 0, off_ping = 0, off_pong = 0, off_init = 0;
  // carried gradients and per-step scratch of the CUDA-core path
  size_t off_dh = 0, off_dc = 0, off_dha = 0, off_dz = 0, off_dy = 0;
  size_t off_loss_part = 0, off_loss_t = 0;
  // tensor-core path: packed weights, staging of S consecutive time steps, control
  int S = 0;             // time steps per staged chunk
  size_t off_wp_ih = 0, off_wp_hh = 0, off_wpT_hh = 0, off_wpT_ih = 0, off_bias_p = 0, off_woutT = 0;
  size_t off_a3 = 0, off_w3 = 0, off_wmn3 = 0, off_wout3 = 0, off_woutmn3 = 0;
  size_t off_z = 0, off_split = 0, off_st_dz = 0, off_st_in = 0, off_st_hp = 0, off_st_dy = 0, off_st_h = 0;
  size_t off_zx = 0, off_zleaf = 0, off_hprev = 0, off_hk = 0, off_y = 0;
  size_t off_sync = 0, off_tape = 0, off_status = 0, off_split_dh = 0;
  size_t off_a3_run = 0, off_zrun = 0, off_hrun = 0, off_dha_run = 0, off_dy_run = 0, split_floats = 0;
  size_t n_sync = 0, tape_bytes = 0;
  size_t total = 0;
  int64_t arena_units = 0;
  int n_loss_part = 0;

  size_t w_layer_elems(int l) const { return (size_t)NG * H * ((l == 0 ? I : H) + H); }
  size_t w_layer_offset(int l) const {  // elements before layer l
    size_t o = 0;
    for (int i = 0; i < l; ++i) o += w_layer_elems(i);
    return o;
  }
  size_t w_total_elems() const { return w_layer_offset(L); }
  // within a hidden block
  size_t h_off(int l) const { return (size_t)l * (hsz + csz); }
  size_t c_off(int l) const { return (size_t)l * (hsz + csz) + hsz; }
};

inline bool valid_desc(const mebptt_lstm_desc* d) {
  if (!d) return false;
  if (d->layers < 1 || d->layers > 16) return false;
  if (d->input < 1 || d->hidden < 1 || d->readout < 1 || d->batch < 1 || d->t < 1) return false;
  if (d->input > (1 << 16) || d->hidden > (1 << 16) || d->readout > (1 << 16) || d->batch > (1 << 16)) return false;
  if (d->dtype != MEBPTT_FP32 && d->dtype != MEBPTT_TF32 && d->dtype != MEBPTT_BF16) return false;
  if (d->want_dx != 0 && d->want_dx != 1) return false;
  if (d->flags & ~(MEBPTT_FLAG_NO_TENSOR_CORES | MEBPTT_FLAG_TIME_RUNS | MEBPTT_FLAG_GRU)) return false;
  return true;
}

// Shapes the tensor-core kernels cover: one layer, bfloat16 operands, a batch that fits one MMA
// tile, sizes that keep every TMA stride a multiple of 16 bytes, and a recurrent weight slice per
// CTA (8 hidden units x 4 gates x H) that fits in shared memory with one CTA per SM.
inline bool tensor_path_supported(const mebptt_lstm_desc* d) {
  return !(d->flags & (MEBPTT_FLAG_NO_TENSOR_CORES | MEBPTT_FLAG_GRU)) && d->dtype == MEBPTT_BF16 && d->layers == 1 && d->batch <= 64 && d->hidden % 8 == 0 &&
         d->input % 8 == 0 && d->readout % 8 == 0 && d->hidden >= 64 &&
         d->hidden <= 1024;
}

// Partial sums of the squared error per time step on the tensor-core path.  Where 32-row groups
// of the readout tile stay inside one step (B % 32 == 0) the readout GEMM's epilogue forms them:
// one per (32 batch rows, 32 readout columns).  Otherwise a separate kernel forms 64 per step.
inline bool loss_fused(int B, int O) { return B % 32 == 0 && (B / 32) * ((O + 31) / 32) <= 256; }
inline int loss_parts_per_step(int B, int O) { return loss_fused(B, O) ? (B / 32) * ((O + 31) / 32) : 64; }

// Shapes outside the persistent kernels' range whose step-by-step operations can still give
// their contractions to the tensor-core GEMM: bfloat16 storage, TMA-friendly strides, and whole
// 32-row groups per step for the loss epilogue.
inline bool stepwise_tc_supported(const mebptt_lstm_desc* d) {
  return !(d->flags & (MEBPTT_FLAG_NO_TENSOR_CORES | MEBPTT_FLAG_GRU)) && !tensor_path_supported(d) && d->dtype == MEBPTT_BF16 &&
         d->batch % 32 == 0 && d->input % 8 == 0 && d->hidden % 8 == 0 && d->readout % 8 == 0 && d->hidden >= 64 &&
         (d->batch / 32) * ((d->readout + 31) / 32) <= 4096;
}

// Float32 storage with tensor-core contractions (MEBPTT_TF32): the same step-by-step scheme over
// operands split into bfloat16 halves.
inline bool stepwise_x3_supported(const mebptt_lstm_desc* d) {
  return !(d->flags & (MEBPTT_FLAG_NO_TENSOR_CORES | MEBPTT_FLAG_GRU)) && d->dtype == MEBPTT_TF32 && d->batch % 32 == 0 &&
         d->input % 8 == 0 && d->hidden % 8 == 0 && d->readout % 8 == 0 && d->hidden >= 64 &&
         (d->batch / 32) * ((d->readout + 31) / 32) <= 4096;
}

inline void state_layout(const mebptt_lstm_desc* d, Layout& y) {
  y.L = d->layers; y.I = d->input; y.H = d->hidden; y.O = d->readout; y.B = d->batch;
  y.dtype = d->dtype; y.t = d->t;
  y.gru = (d->flags & MEBPTT_FLAG_GRU) != 0;
  y.NG = y.gru ? 3 : 4;
  y.tensor_path = tensor_path_supported(d);
  y.stepwise_tc = stepwise_tc_supported(d);
  y.stepwise_x3 = stepwise_x3_supported(d);
  y.esz = (d->dtype == MEBPTT_BF16) ? 2 : 4;
  const size_t row = (size_t)y.H * y.esz;
  y.granule = 256 / gcd_sz(256, row) * row;  // lcm(256, row bytes)
  const size_t bh = (size_t)y.B * y.H;
  y.hsz = align_up(bh * y.esz, y.granule);
  y.csz = align_up(bh * 4, y.granule);
  y.plane = align_up(bh * y.esz, y.granule);
  y.gsz = 4 * y.plane;
  y.unit = (size_t)y.L * (y.hsz + y.csz);
  y.rec_gates = y.unit;
  y.rec_in = y.unit + (size_t)y.L * y.gsz;
  y.rec = y.rec_in + y.unit;
}

// Steps per chunk on the step-by-step paths: 2048 rows of the batched GEMMs, at most 32 steps (at
// batch 32, 64 steps were measured: config 4 at full memory 134 -> 128 ms per step for 134 MB more
// working memory, not taken).  At config 5 (B = 128): 1024 rows
// 31.1 ms per step at t = 256 and 229 MB of working memory, 2048 rows 28.0 ms and 407 MB.
inline int stepwise_chunk_steps(int B) {
  const int s = 2048 / B > 0 ? 2048 / B : 1;
  return s > 32 ? 32 : s;
}

// The tensor-core executor cuts the tape into work items:
//   FWD   a run of consecutive forward operations, each starting from the state the previous one
//         wrote, at most S of them (one persistent launch);
//   BWD   a run of consecutive backward operations inside one chunk of S time steps;
//   LEAF  n >= 2 consecutive leaves of the recursion -- FWD(k -> working core), BWD(k),
//         FWD(k-1 -> working core), BWD(k-1), ... -- whose forward operations each start from a
//         memorised state, inside one chunk.  Their forward operations do not depend on one another,
//         so they are computed together by batched GEMMs instead of step by step.
struct WorkItem {
  enum Kind { FWD, BWD, LEAF } kind;
  size_t i;   // first tape entry
  int n;      // operations (FWD, BWD) or leaves (LEAF: 2 n tape entries)
};
inline bool is_leaf_at(const Plan* p, size_t i) {
  const size_t n = p->tape.size();
  if (i + 1 >= n) return false;
  const mebptt_op& f = p->tape[i];
  const mebptt_op& b = p->tape[i + 1];
  if (f.kind != MEBPTT_OP_FWD || b.kind != MEBPTT_OP_BWD) return false;
  if (f.dst != MEBPTT_LOC_CORE || b.src != MEBPTT_LOC_CORE || f.k != b.k) return false;
  if (f.src == MEBPTT_LOC_CORE) return false;
  // a leaf proper: not the last step of a longer sweep
  if (i > 0 && p->tape[i - 1].kind == MEBPTT_OP_FWD && p->tape[i - 1].dst == f.src && p->tape[i - 1].k == f.k - 1)
    return false;
  return true;
}
inline std::vector<WorkItem> work_items(const Plan* p, int S) {
  std::vector<WorkItem> items;
  const size_t n = p->tape.size();
  size_t i = 0;
  while (i < n) {
    if (is_leaf_at(p, i)) {
      const int chunk = (p->tape[i].k - 1) / S;
      int leaves = 1;
      while (is_leaf_at(p, i + 2 * (size_t)leaves) && p->tape[i + 2 * (size_t)leaves].k == p->tape[i].k - leaves &&
             (p->tape[i + 2 * (size_t)leaves].k - 1) / S == chunk)
        ++leaves;
      if (leaves >= 2) {
        items.push_back(WorkItem{WorkItem::LEAF, i, leaves});
        i += 2 * (size_t)leaves;
        continue;
      }
    }
    size_t j = i + 1;
    if (p->tape[i].kind == MEBPTT_OP_FWD) {
      while (j < n && j - i < (size_t)S && p->tape[j].kind == MEBPTT_OP_FWD && p->tape[j].k == p->tape[j - 1].k + 1 &&
             p->tape[j].src == p->tape[j - 1].dst)
        ++j;
      items.push_back(WorkItem{WorkItem::FWD, i, (int)(j - i)});
    } else {
      const int chunk = (p->tape[i].k - 1) / S;
      while (j < n && p->tape[j].kind == MEBPTT_OP_BWD && (p->tape[j].k - 1) / S == chunk) ++j;
      items.push_back(WorkItem{WorkItem::BWD, i, (int)(j - i)});
    }
    i = j;
  }
  return items;
}

inline void workspace_layout(const mebptt_lstm_desc* d, const Plan* p, Layout& y) {
  state_layout(d, y);
  y.arena_units = p->arena_units;
  y.loc_bytes = y.unit / (size_t)(p->sigma > 0 ? p->sigma : 1);
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t r = o; o = align_up(o + bytes, y.granule); return r; };
  y.off_arena = take((size_t)y.arena_units * y.loc_bytes);
  y.off_core = take(y.rec);
  y.off_ping = take(y.unit);
  y.off_pong = take(y.unit);
  const size_t bh4 = (size_t)y.B * y.H * 4;
  y.off_dh = take((size_t)y.L * bh4);
  y.off_dc = take((size_t)y.L * bh4);
  y.off_loss_t = take((size_t)y.t * 4);
  if (!y.tensor_path) {
    y.off_dha = take(bh4);
    y.off_dz = take((size_t)y.B * 4 * y.H * 4);
    y.off_dy = take((size_t)y.B * y.O * 4);
    y.n_loss_part = ((y.B + 63) / 64) * ((y.O + 63) / 64);
    if (y.stepwise_tc) {
      y.n_loss_part = (y.B / 32) * ((y.O + 31) / 32);
      y.off_z = take((size_t)y.B * 4 * y.H * 4);
      // stages of one chunk of S steps for the weight-gradient contractions
      y.S = stepwise_chunk_steps(y.B);
      const size_t rows = (size_t)y.S * y.B;
      y.off_st_dz = take((size_t)y.L * rows * 4 * y.H * 2);
      y.off_st_in = take(rows * y.I * 2 + (size_t)(y.L - 1) * rows * y.H * 2);
      y.off_st_hp = take((size_t)y.L * rows * y.H * 2);
      y.off_st_dy = take(rows * y.O * 2);
      y.off_st_h = take(rows * y.H * 2);
      // a run of up to S consecutive operations, one layer at a time: pre-activations of the run,
      // the layer's h_k (the next layer's input), the gradient entering the layer at every step
      y.off_zrun = take(rows * 4 * y.H * 4);
      y.off_hrun = take(rows * y.H * 2);
      y.off_dha_run = take(rows * y.H * 4);
      // split-K scratch: a wave of 128 x 128 float32 tiles for one step, times the 8 row tiles of
      // a whole run (its products are split like a single step's, to sum in the same order)
      y.split_floats = (size_t)148 * 128 * 128 * ((rows + 127) / 128);
      y.off_split = take(y.split_floats * 4);
      y.off_split_dh = take((size_t)y.L * 148 * 128 * 128 * 4);   // per layer: the parts of dh = dz W_hh
    }
    if (y.stepwise_x3) {
      const size_t G = 4 * (size_t)y.H, Kmax = (size_t)(y.I > y.H ? y.I : y.H) + y.H;
      y.n_loss_part = (y.B / 32) * ((y.O + 31) / 32);
      y.S = stepwise_chunk_steps(y.B);
      const size_t rows = (size_t)y.S * y.B;
      y.off_z = take((size_t)y.B * G * 4);
      // the readout of a run of up to S steps at once; its split-K scratch as on the bfloat16 path
      y.off_a3_run = take(rows * 3 * Kmax * 2);
      y.off_hrun = take(y.L > 1 ? rows * y.H * 4 : 0);
      y.off_dy_run = take(rows * y.O * 4);
      y.off_dha_run = take(rows * y.H * 4);
      y.split_floats = (size_t)148 * 128 * 128 * ((rows + 127) / 128);
      y.off_split = take(y.split_floats * 4);
      y.off_split_dh = take((size_t)y.L * 148 * 128 * 128 * 4);
      y.off_a3 = take((size_t)y.B * 3 * Kmax * 2);
      y.off_w3 = take(3 * y.w_total_elems() * 2);
      y.off_wmn3 = take(3 * y.w_total_elems() * 2);
      y.off_wout3 = take((size_t)3 * y.O * y.H * 2);
      y.off_woutmn3 = take((size_t)3 * y.O * y.H * 2);
      y.off_st_dz = take((size_t)y.L * rows * 3 * G * 2);
      y.off_st_in = take(rows * 2 * y.I * 2 + (size_t)(y.L - 1) * rows * 2 * y.H * 2);
      y.off_st_hp = take((size_t)y.L * rows * 2 * y.H * 2);
      y.off_st_dy = take(rows * 3 * y.O * 2);
      y.off_st_h = take(rows * 3 * y.H * 2);
    }
    y.off_loss_part = take((size_t)y.n_loss_part * 4 * ((y.stepwise_tc || y.stepwise_x3) ? y.S : 1));
    y.off_status = take(256);
  } else {
    const size_t G = (size_t)4 * y.H;
    // steps per chunk (and at most per persistent launch): 2048 rows of the batched GEMMs.  Longer
    // chunks mean fewer launches and longer contractions for the weight gradients, at the price of
    // staging memory (measured at config 3, MSM m = 100: 1024 rows 22.9 ms and 102 MB of working
    // memory, 2048 rows 21.6 ms and 173 MB, 4096 rows 21.9 ms and 316 MB)
    y.S = 2048 / y.B > 0 ? 2048 / y.B : 1;
    if (y.S > 64) y.S = 64;
    const size_t SB = (size_t)y.S * y.B;
    y.off_init = take(y.unit);
    y.off_wp_ih = take(G * y.I * 2);
    y.off_wp_hh = take(G * y.H * 2);
    y.off_wpT_hh = take(G * y.H * 2);
    y.off_wpT_ih = take(d->want_dx ? G * y.I * 2 : 0);
    y.off_bias_p = take(G * 4);
    y.off_woutT = take((size_t)y.O * y.H * 2);
    // two copies: the projections of the next window are computed while the runs read this one's
    y.off_zx = take(2 * SB * G * 4);
    // two copies of what the weight-gradient GEMMs read: they may still be running (on the
    // library's side stream) while the backward pass fills the stages of the next chunk
    y.off_dz = take(2 * SB * G * 2);
    y.off_hprev = take(2 * SB * y.H * 2);
    y.off_hk = take(2 * SB * y.H * 2);
    y.off_y = take(SB * y.O * 4);
    y.off_dy = take(2 * SB * y.O * 2);
    y.off_dha = take(SB * y.H * 4);
    y.off_zleaf = take(SB * G * 4);   // pre-activations of a batch of leaves
    y.off_loss_part = take((size_t)y.S * loss_parts_per_step(y.B, y.O) * 4);
    y.n_sync = 64 * (work_items(p, y.S).size() + 1);   // two 128-byte lines per persistent launch (one per group of CTAs)
    y.off_sync = take(y.n_sync * 4);
    y.tape_bytes = (size_t)p->tape.size() * 32 * 2;   // the tape, and the compacted entries of leaf batches
    y.off_tape = take(y.tape_bytes);
    y.off_status = take(256);
  }
  y.total = o;
}

}  // namespace mebptt
