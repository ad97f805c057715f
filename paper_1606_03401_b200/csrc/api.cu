// C interface: execution.  Walks the tape of a plan and enqueues the device work of one
// training step on the caller's stream; nothing here waits for the device.
#include <cuda_runtime.h>

#include <cstdint>
#include <cstdlib>
#include <cstring>
#include <vector>

#include "env.hpp"
#include "kernels.hpp"
#include "layout.hpp"
#include "mebptt.h"
#include "plan.hpp"
#include "tc.hpp"

using namespace mebptt;

namespace {

using StepIO = tc::StepPtrs;

// Base address of the hidden block (or record) at a tape location; LOC_INIT has none.
inline char* loc_base(const Layout& y, char* ws, int32_t loc) {
  switch (loc) {
    case MEBPTT_LOC_PING: return ws + y.off_ping;
    case MEBPTT_LOC_PONG: return ws + y.off_pong;
    case MEBPTT_LOC_CORE: return ws + y.off_core;
    default: return ws + y.off_arena + (size_t)loc * y.loc_bytes;
  }
}

inline void hidden_at(const Layout& y, const StepIO& io, int32_t loc, int l, const void** h, const float** c) {
  const size_t bh = (size_t)y.B * y.H;
  if (loc == MEBPTT_LOC_INIT) {
    *h = io.h0 + (size_t)l * bh * y.esz;
    *c = io.c0 + (size_t)l * bh;
  } else {
    char* base = loc_base(y, io.ws, loc);
    *h = base + y.h_off(l);
    *c = reinterpret_cast<const float*>(base + y.c_off(l));
  }
}

// Where layer l of a forward operation finds its input state and puts its output state.
struct FwdPtrs {
  const void* h_prev; const float* c_prev;
  void* h_out; float* c_out;
  void* gates;                       // NULL: the destination holds a hidden state only
  void* h_in_copy; float* c_in_copy; // NULL unless the destination is a whole internal state
};
inline FwdPtrs fwd_ptrs(const Layout& y, const StepIO& io, const mebptt_op& op, int l) {
  FwdPtrs f{};
  char* dst = loc_base(y, io.ws, op.dst);
  hidden_at(y, io, op.src, l, &f.h_prev, &f.c_prev);
  f.h_out = dst + y.h_off(l);
  f.c_out = reinterpret_cast<float*>(dst + y.c_off(l));
  if (op.dst_fmt != MEBPTT_FMT_HIDDEN) f.gates = dst + y.rec_gates + (size_t)l * y.gsz;
  if (op.dst_fmt == MEBPTT_FMT_INTERNAL) {
    f.h_in_copy = dst + y.rec_in + y.h_off(l);
    f.c_in_copy = reinterpret_cast<float*>(dst + y.rec_in + y.c_off(l));
  }
  return f;
}
// What layer l of a backward operation reads of its internal state, and the layer's input at that step.
struct BwdPtrs {
  const void* gates; const float* c_t;
  const void* h_prev; const float* c_prev;
  const void* in;
};
inline BwdPtrs bwd_ptrs(const Layout& y, const StepIO& io, const mebptt_op& op, int l) {
  BwdPtrs b{};
  char* rec = loc_base(y, io.ws, op.src);
  b.gates = rec + y.rec_gates + (size_t)l * y.gsz;
  b.c_t = reinterpret_cast<const float*>(rec + y.c_off(l));
  if (op.dst_fmt == MEBPTT_FMT_INTERNAL) {
    b.h_prev = rec + y.rec_in + y.h_off(l);
    b.c_prev = reinterpret_cast<const float*>(rec + y.rec_in + y.c_off(l));
  } else {
    hidden_at(y, io, op.aux, l, &b.h_prev, &b.c_prev);
  }
  b.in = (l == 0) ? (const void*)(io.x + (size_t)(op.k - 1) * y.B * y.I * y.esz) : (const void*)(rec + y.h_off(l - 1));
  return b;
}

int check_common(const mebptt_lstm_desc* desc, const mebptt_plan_t* plan) {
  if (!valid_desc(desc) || !plan) return MEBPTT_ERR_ARG;
  const Plan* p = reinterpret_cast<const Plan*>(plan);
  if (p->t != desc->t) return MEBPTT_ERR_ARG;
  // the plan's sizes must hold this layout's states: a hidden state is sigma units of the plan, and
  // its internal states (alpha units; beta without the input hidden state) must fit theirs.  With
  // sigma = 1 that is alpha >= 4 and beta >= 3 for every layout of this library.
  Layout y;
  state_layout(desc, y);
  const size_t sg = (size_t)(p->sigma > 0 ? p->sigma : 1);
  if (y.unit % sg != 0 || (y.unit / sg) % y.granule != 0) return MEBPTT_ERR_UNSUPPORTED;
  const size_t loc_bytes = y.unit / sg;
  if (p->mode != MEBPTT_HSM && (size_t)p->alpha * loc_bytes < y.rec) return MEBPTT_ERR_UNSUPPORTED;
  if (p->mode == MEBPTT_MSM && p->beta != 0 && (size_t)p->beta * loc_bytes < y.rec_in) return MEBPTT_ERR_UNSUPPORTED;
  return MEBPTT_OK;
}

int run_step(const mebptt_lstm_desc* desc, const Plan* p, const Layout& y, const StepIO& io, cudaStream_t s,
             bool side_stream = true) {
  if (y.tensor_path) {
    return (int)tc::run_step(y, p, io, desc->want_dx != 0, s, false, side_stream && !env::no_overlap());
  }
  const size_t bh = (size_t)y.B * y.H;
  const size_t plane_elems = y.plane / y.esz;
  char* ws = io.ws;
  float* dh_rec = reinterpret_cast<float*>(ws + y.off_dh);
  float* dc_rec = reinterpret_cast<float*>(ws + y.off_dc);
  float* dha = reinterpret_cast<float*>(ws + y.off_dha);
  float* dz = reinterpret_cast<float*>(ws + y.off_dz);
  float* dy = reinterpret_cast<float*>(ws + y.off_dy);
  float* loss_part = reinterpret_cast<float*>(ws + y.off_loss_part);
  float* loss_t = reinterpret_cast<float*>(ws + y.off_loss_t);
  int* status = reinterpret_cast<int*>(ws + y.off_status);
  // where each layer's dh of the latest backward operation lies: in its buffer (zero at first), or
  // in the parts of a contraction split along K
  std::vector<tc::SplitParts> dh_parts((size_t)y.L);
  stepwise::Scratch tcw{};
  if (y.stepwise_tc) {
    tcw.z = reinterpret_cast<float*>(ws + y.off_z);
    tcw.status = status;
    tcw.S = y.S; tcw.I0 = y.I;
    tcw.st_dz = reinterpret_cast<__nv_bfloat16*>(ws + y.off_st_dz);
    tcw.st_in = reinterpret_cast<__nv_bfloat16*>(ws + y.off_st_in);
    tcw.st_hp = reinterpret_cast<__nv_bfloat16*>(ws + y.off_st_hp);
    tcw.st_dy = reinterpret_cast<__nv_bfloat16*>(ws + y.off_st_dy);
    tcw.st_h = reinterpret_cast<__nv_bfloat16*>(ws + y.off_st_h);
    tcw.split = tc::SplitWs{reinterpret_cast<float*>(ws + y.off_split), (size_t)148 * 128 * 128};
    tcw.split_run = tc::SplitWs{reinterpret_cast<float*>(ws + y.off_split), y.split_floats};
    tcw.zrun = reinterpret_cast<float*>(ws + y.off_zrun);
    tcw.hrun = reinterpret_cast<__nv_bfloat16*>(ws + y.off_hrun);
    tcw.dha_run = reinterpret_cast<float*>(ws + y.off_dha_run);
    tcw.loss_part = loss_part;
    tcw.split_dh = reinterpret_cast<float*>(ws + y.off_split_dh);
    tcw.dh_parts = dh_parts.data();
  }
  stepwise3::Scratch x3{};
  size_t w_off[16];
  for (int l = 0; l < y.L; ++l) w_off[l] = y.w_layer_offset(l);
  auto bf = [&](size_t off) { return reinterpret_cast<__nv_bfloat16*>(ws + off); };
  if (y.stepwise_x3) {
    x3.z = reinterpret_cast<float*>(ws + y.off_z);
    x3.status = status;
    x3.split = tc::SplitWs{reinterpret_cast<float*>(ws + y.off_split), (size_t)148 * 128 * 128};
    x3.S = y.S; x3.I0 = y.I;
    x3.a3 = bf(y.off_a3); x3.w3 = bf(y.off_w3); x3.wmn3 = bf(y.off_wmn3);
    x3.wout3 = bf(y.off_wout3); x3.woutmn3 = bf(y.off_woutmn3);
    x3.st_dz3 = bf(y.off_st_dz); x3.st_in2 = bf(y.off_st_in); x3.st_hp2 = bf(y.off_st_hp);
    x3.st_dy3 = bf(y.off_st_dy); x3.st_h3 = bf(y.off_st_h);
    x3.split_run = tc::SplitWs{reinterpret_cast<float*>(ws + y.off_split), y.split_floats};
    x3.dy_run = reinterpret_cast<float*>(ws + y.off_dy_run);
    x3.dha_run = reinterpret_cast<float*>(ws + y.off_dha_run);
    x3.loss_part = loss_part;
    x3.split_dh = reinterpret_cast<float*>(ws + y.off_split_dh);
    x3.dh_parts = dh_parts.data();
    x3.a3_run = bf(y.off_a3_run);
    x3.h_run = reinterpret_cast<float*>(ws + y.off_hrun);
  }
  const bool staged = y.stepwise_tc || y.stepwise_x3;   // weight gradients per chunk of S steps
  int rc = MEBPTT_OK;

  cudaMemsetAsync(status, 0, 256, s);
  cudaMemsetAsync(dh_rec, 0, (size_t)y.L * bh * 4, s);
  cudaMemsetAsync(dc_rec, 0, (size_t)y.L * bh * 4, s);
  cudaMemsetAsync(io.dW, 0, y.w_total_elems() * 4, s);
  cudaMemsetAsync(io.db, 0, (size_t)y.L * y.NG * y.H * 4, s);
  cudaMemsetAsync(io.dW_out, 0, (size_t)y.O * y.H * 4, s);
  cudaMemsetAsync(io.db_out, 0, (size_t)y.O * 4, s);
  cudaMemsetAsync(io.counters, 0, 8 * sizeof(int64_t), s);

  if (y.stepwise_x3)
    stepwise3::pack_weights(x3, y.L, y.I, y.H, y.O, reinterpret_cast<const float*>(io.W), w_off,
                            reinterpret_cast<const float*>(io.W_out), s);
  auto run_op = [&](const mebptt_op& op) {
    const int64_t k = op.k;
    const char* x_k = io.x + (size_t)(k - 1) * y.B * y.I * y.esz;
    if (op.kind == MEBPTT_OP_FWD) {
      char* dst = loc_base(y, ws, op.dst);
      for (int l = 0; l < y.L; ++l) {
        generic::FwdArgs a{};
        const FwdPtrs f = fwd_ptrs(y, io, op, l);
        a.h_prev = f.h_prev; a.c_prev = f.c_prev; a.h_out = f.h_out; a.c_out = f.c_out;
        a.gates = f.gates; a.h_in_copy = f.h_in_copy; a.c_in_copy = f.c_in_copy;
        a.in = (l == 0) ? (const void*)x_k : (const void*)(dst + y.h_off(l - 1));
        a.I = (l == 0) ? y.I : y.H;
        a.W = io.W + y.w_layer_offset(l) * y.esz;
        a.bias = io.b + (size_t)l * y.NG * y.H;
        a.plane_elems = plane_elems;
        a.B = y.B; a.H = y.H;
        a.counters = (l == 0) ? io.counters : nullptr;
        if (y.stepwise_x3) rc = stepwise3::forward_step(a, x3, l, w_off[l], s);
        else if (y.stepwise_tc) rc = stepwise::forward_step(a, tcw, s);
        else if (y.gru) generic::gru_forward_step(y.dtype, a, s);
        else generic::forward_step(y.dtype, a, s);
        if (rc != MEBPTT_OK) break;
      }
    } else {
      char* rec = loc_base(y, ws, op.src);
      // readout of the top layer, loss term, dy and the gradient entering the top layer
      generic::ReadoutArgs r{};
      r.h = rec + y.h_off(y.L - 1);
      r.W_out = io.W_out; r.b_out = io.b_out;
      r.target = io.targets + (size_t)(k - 1) * y.B * y.O;
      r.dy = dy; r.loss_part = loss_part; r.n_loss_part = y.n_loss_part;
      r.loss_k = loss_t + (k - 1);
      r.dha = dha; r.dW_out = io.dW_out; r.db_out = io.db_out;
      r.B = y.B; r.H = y.H; r.O = y.O;
      const int sidx = staged ? (int)((k - 1) % y.S) : 0;
      if (y.stepwise_x3) rc = stepwise3::readout(r, x3, sidx, s);
      else if (y.stepwise_tc) rc = stepwise::readout(r, tcw, sidx, s);
      else generic::readout(y.dtype, r, s);
      if (rc != MEBPTT_OK) return;
      for (int l = y.L - 1; l >= 0; --l) {
        generic::BwdArgs a{};
        a.dha = dha;
        a.dh_rec = dh_rec + (size_t)l * bh;
        a.dc_rec = dc_rec + (size_t)l * bh;
        const BwdPtrs q = bwd_ptrs(y, io, op, l);
        a.gates = q.gates; a.c_t = q.c_t; a.h_prev = q.h_prev; a.c_prev = q.c_prev; a.in = q.in;
        a.plane_elems = plane_elems;
        a.I = (l == 0) ? y.I : y.H;
        a.W = io.W + y.w_layer_offset(l) * y.esz;
        a.dz = dz;
        a.dW = io.dW + y.w_layer_offset(l);
        a.db = io.db + (size_t)l * y.NG * y.H;
        a.d_lo = (l > 0) ? dha : (desc->want_dx ? io.dx + (size_t)(k - 1) * y.B * y.I : nullptr);
        a.B = y.B; a.H = y.H;
        a.counters = (l == y.L - 1) ? io.counters : nullptr;
        if (y.stepwise_x3) rc = stepwise3::backward_layer(a, x3, l, w_off[l], sidx, s);
        else if (y.stepwise_tc) rc = stepwise::backward_layer(a, tcw, l, sidx, s);
        else if (y.gru) generic::gru_backward_layer(y.dtype, a, s);
        else generic::backward_layer(y.dtype, a, s);
        if (rc != MEBPTT_OK) break;
      }
      if (staged && sidx == 0 && rc == MEBPTT_OK) {
        // the chunk's first step has been backpropagated: its weight gradients in one go
        const int64_t chunk = (k - 1) / y.S;
        const int steps = (int)((chunk + 1) * y.S <= y.t ? y.S : y.t - chunk * y.S);
        rc = y.stepwise_x3 ? stepwise3::flush_chunk(x3, steps, y.L, y.B, y.I, y.H, y.O, w_off, io.dW, io.dW_out, io.db, io.db_out, s)
                           : stepwise::flush_chunk(tcw, steps, y.L, y.B, y.I, y.H, y.O, w_off, io.dW, io.dW_out, io.db, io.db_out, s);
      }
    }
  };

  // The bfloat16 step-by-step path takes runs of consecutive operations one layer at a time (the
  // input products, the readout and the gradients handed down are then batched over the run);
  // everything else, and the leaves of the recursion, go operation by operation.  Both give the
  // same bits; MEBPTT_STEPWISE_PER_OP=1 keeps to single operations (the tests compare the two).
  const bool per_op_only = env::stepwise_per_op();
  if (!(y.stepwise_tc || y.stepwise_x3) || per_op_only) {
    for (const mebptt_op& op : p->tape) {
      if (rc != MEBPTT_OK) break;
      run_op(op);
    }
  } else {
    const std::vector<WorkItem> items = work_items(p, y.S);
    std::vector<stepwise::FwdRunStep> fst((size_t)y.S);
    std::vector<stepwise::BwdRunStep> bst((size_t)y.S);
    std::vector<const void*> h_top((size_t)y.S);
    for (const WorkItem& wi : items) {
      if (rc != MEBPTT_OK) break;
      const mebptt_op* ops = p->tape.data() + wi.i;
      if (wi.kind == WorkItem::LEAF || wi.n == 1) {
        const size_t cnt = wi.kind == WorkItem::LEAF ? 2 * (size_t)wi.n : 1;
        for (size_t j = 0; j < cnt && rc == MEBPTT_OK; ++j) run_op(ops[j]);
      } else if (y.stepwise_x3 && wi.kind == WorkItem::FWD) {
        // float32 storage: a forward operation is one contraction over [input ; h], so nothing of
        // it can be taken out of the recurrence; what a run saves is the splitting of the operands
        // (once for all inputs of the run; h_k by the cell kernel that produces it)
        const int n = wi.n;
        const int64_t k0 = ops[0].k;
        for (int l = 0; l < y.L && rc == MEBPTT_OK; ++l) {
          for (int j = 0; j < n; ++j) {
            const FwdPtrs q = fwd_ptrs(y, io, ops[j], l);
            stepwise::FwdRunStep& f = fst[j];
            f = stepwise::FwdRunStep{};
            f.h_prev = q.h_prev; f.c_prev = q.c_prev; f.h_out = q.h_out; f.c_out = q.c_out;
            f.gates = q.gates; f.h_in_copy = q.h_in_copy; f.c_in_copy = q.c_in_copy;
          }
          const int I_l = l == 0 ? y.I : y.H;
          const float* in = (l == 0) ? reinterpret_cast<const float*>(io.x) + (size_t)(k0 - 1) * y.B * y.I : x3.h_run;
          rc = stepwise3::forward_run_layer(fst.data(), n, in, (int64_t)y.B * I_l, I_l, io.b + (size_t)l * 4 * y.H, y.B,
                                            y.H, plane_elems, l == 0 ? io.counters : nullptr, x3, w_off[l],
                                            l + 1 < y.L ? x3.h_run : nullptr, s);
        }
      } else if (y.stepwise_x3) {
        // float32 storage: the readout of the run at once, then its backward operations one by one
        const int n = wi.n;
        const int64_t k_hi = ops[0].k, k_lo = k_hi - n + 1;
        const int s_lo = (int)((k_lo - 1) % y.S);
        auto op_at = [&](int a) -> const mebptt_op& { return ops[n - 1 - a]; };
        for (int a = 0; a < n; ++a) h_top[a] = loc_base(y, ws, op_at(a).src) + y.h_off(y.L - 1);
        rc = stepwise3::readout_run(reinterpret_cast<const float* const*>(h_top.data()), n, s_lo, io.b_out,
                                    io.targets + (size_t)(k_lo - 1) * y.B * y.O, loss_t + (k_lo - 1), y.B, y.H, y.O, x3, s);
        for (int a = n - 1; a >= 0 && rc == MEBPTT_OK; --a) {
          const mebptt_op& op = op_at(a);
          char* rec = loc_base(y, ws, op.src);
          const char* x_k = io.x + (size_t)(op.k - 1) * y.B * y.I * y.esz;
          for (int l = y.L - 1; l >= 0 && rc == MEBPTT_OK; --l) {
            generic::BwdArgs b{};
            b.dha = (l == y.L - 1) ? x3.dha_run + (size_t)a * bh : dha;
            b.dh_rec = dh_rec + (size_t)l * bh;
            b.dc_rec = dc_rec + (size_t)l * bh;
            const BwdPtrs q = bwd_ptrs(y, io, op, l);
            b.gates = q.gates; b.c_t = q.c_t; b.h_prev = q.h_prev; b.c_prev = q.c_prev; b.in = q.in;
            b.plane_elems = plane_elems;
            b.I = (l == 0) ? y.I : y.H;
            b.W = io.W + y.w_layer_offset(l) * y.esz;
            b.dz = dz;
            b.dW = io.dW + y.w_layer_offset(l);
            b.db = io.db + (size_t)l * 4 * y.H;
            b.d_lo = (l > 0) ? dha : (desc->want_dx ? io.dx + (size_t)(op.k - 1) * y.B * y.I : nullptr);
            b.B = y.B; b.H = y.H;
            b.counters = (l == y.L - 1) ? io.counters : nullptr;
            rc = stepwise3::backward_layer(b, x3, l, w_off[l], s_lo + a, s);
          }
        }
        if (s_lo == 0 && rc == MEBPTT_OK) {
          const int64_t chunk = (k_lo - 1) / y.S;
          const int steps = (int)((chunk + 1) * y.S <= y.t ? y.S : y.t - chunk * y.S);
          rc = stepwise3::flush_chunk(x3, steps, y.L, y.B, y.I, y.H, y.O, w_off, io.dW, io.dW_out, io.db, io.db_out, s);
        }
      } else if (wi.kind == WorkItem::FWD) {
        const int n = wi.n;
        const int64_t k0 = ops[0].k;
        for (int l = 0; l < y.L && rc == MEBPTT_OK; ++l) {
          for (int j = 0; j < n; ++j) {
            const FwdPtrs q = fwd_ptrs(y, io, ops[j], l);
            stepwise::FwdRunStep& f = fst[j];
            f = stepwise::FwdRunStep{};
            f.h_prev = q.h_prev; f.c_prev = q.c_prev; f.h_out = q.h_out; f.c_out = q.c_out;
            f.gates = q.gates; f.h_in_copy = q.h_in_copy; f.c_in_copy = q.c_in_copy;
          }
          const void* in = (l == 0) ? (const void*)(io.x + (size_t)(k0 - 1) * y.B * y.I * y.esz) : (const void*)tcw.hrun;
          rc = stepwise::forward_run_layer(fst.data(), n, in, l == 0 ? y.I : y.H, io.W + y.w_layer_offset(l) * y.esz,
                                           io.b + (size_t)l * 4 * y.H, l + 1 < y.L, y.B, y.H, plane_elems,
                                           l == 0 ? io.counters : nullptr, tcw, s);
        }
      } else {
        // n backward operations, time descending, inside one chunk: index a = step - first step
        const int n = wi.n;
        const int64_t k_hi = ops[0].k, k_lo = k_hi - n + 1;
        const int s_lo = (int)((k_lo - 1) % y.S);
        auto op_at = [&](int a) -> const mebptt_op& { return ops[n - 1 - a]; };
        for (int a = 0; a < n; ++a) h_top[a] = loc_base(y, ws, op_at(a).src) + y.h_off(y.L - 1);
        rc = stepwise::readout_run(h_top.data(), n, s_lo, io.W_out, io.b_out, io.targets + (size_t)(k_lo - 1) * y.B * y.O,
                                   loss_t + (k_lo - 1), y.B, y.H, y.O, tcw, s);
        for (int l = y.L - 1; l >= 0 && rc == MEBPTT_OK; --l) {
          for (int a = 0; a < n; ++a) {
            const BwdPtrs q = bwd_ptrs(y, io, op_at(a), l);
            stepwise::BwdRunStep& b = bst[a];
            b.gates = q.gates; b.c_t = q.c_t; b.h_prev = q.h_prev; b.c_prev = q.c_prev; b.in = q.in;
          }
          float* d_lo = (l > 0) ? tcw.dha_run : (desc->want_dx ? io.dx + (size_t)(k_lo - 1) * y.B * y.I : nullptr);
          rc = stepwise::backward_run_layer(bst.data(), n, s_lo, l, l == 0 ? y.I : y.H, io.W + y.w_layer_offset(l) * y.esz,
                                            dh_rec + (size_t)l * bh, dc_rec + (size_t)l * bh, d_lo, y.B, y.H, plane_elems, l == y.L - 1 ? io.counters : nullptr, tcw, s);
        }
        if (s_lo == 0 && rc == MEBPTT_OK) {
          const int64_t chunk = (k_lo - 1) / y.S;
          const int steps = (int)((chunk + 1) * y.S <= y.t ? y.S : y.t - chunk * y.S);
          rc = stepwise::flush_chunk(tcw, steps, y.L, y.B, y.I, y.H, y.O, w_off, io.dW, io.dW_out, io.db, io.db_out, s);
        }
      }
    }
  }
  if (rc != MEBPTT_OK) return rc;
  generic::finalize_step(loss_t, y.t, io.loss, io.counters, p->peak_units, status, s);
  return cudaGetLastError() == cudaSuccess ? MEBPTT_OK : MEBPTT_ERR_CUDA;
}

// staging area of the host-buffer variant, placed after the ordinary workspace
struct Staging {
  size_t W, b, W_out, b_out, x, targets, h0, c0, loss, dW, db, dW_out, db_out, dx, counters, total;
  size_t nW, nb, nW_out, nb_out, nx, ntargets, nh0, nc0, ndx;  // bytes
};

void staging_layout(const Layout& y, bool want_dx, size_t base, Staging& g) {
  size_t o = base;
  auto take = [&](size_t bytes) { size_t r = o; o = align_up(o + bytes, 256); return r; };
  const size_t bh = (size_t)y.B * y.H;
  g.nW = y.w_total_elems() * y.esz; g.nb = (size_t)y.L * y.NG * y.H * 4;
  g.nW_out = (size_t)y.O * y.H * y.esz; g.nb_out = (size_t)y.O * 4;
  g.nx = (size_t)y.t * y.B * y.I * y.esz; g.ntargets = (size_t)y.t * y.B * y.O * 4;
  g.nh0 = (size_t)y.L * bh * y.esz; g.nc0 = (size_t)y.L * bh * 4;
  g.ndx = want_dx ? (size_t)y.t * y.B * y.I * 4 : 0;
  g.W = take(g.nW); g.b = take(g.nb); g.W_out = take(g.nW_out); g.b_out = take(g.nb_out);
  g.x = take(g.nx); g.targets = take(g.ntargets); g.h0 = take(g.nh0); g.c0 = take(g.nc0);
  g.loss = take(4); g.dW = take(y.w_total_elems() * 4); g.db = take(g.nb);
  g.dW_out = take((size_t)y.O * y.H * 4); g.db_out = take(g.nb_out);
  g.dx = take(g.ndx); g.counters = take(8 * sizeof(int64_t));
  g.total = o;
}

}  // namespace

extern "C" {

size_t mebptt_lstm_unit_bytes(const mebptt_lstm_desc* desc) {
  if (!valid_desc(desc)) return 0;
  Layout y;
  state_layout(desc, y);
  return y.unit;
}

int64_t mebptt_budget_bytes_to_units(const mebptt_lstm_desc* desc, size_t bytes) {
  const size_t u = mebptt_lstm_unit_bytes(desc);
  return u ? (int64_t)(bytes / u) : -1;
}

int mebptt_plan_for_bytes(const mebptt_lstm_desc* desc, size_t budget_bytes, int mode, int include_working,
                          mebptt_plan_t** out) {
  if (!out || !valid_desc(desc) || mode < MEBPTT_HSM || mode > MEBPTT_MSM) return MEBPTT_ERR_ARG;
  *out = nullptr;
  const size_t unit = mebptt_lstm_unit_bytes(desc);
  if (!unit) return MEBPTT_ERR_ARG;
  const size_t per_m = (mode == MEBPTT_ISM) ? 4 * unit : unit;   // what one more of the mode's units costs
  int64_t m = (int64_t)(budget_bytes / per_m);
  for (int round = 0; round < 64 && m >= 1; ++round) {
    mebptt_plan_t* plan = nullptr;
    const int rc = mebptt_plan(desc->t, m, mode, &plan);
    if (rc != MEBPTT_OK) return rc;
    if (!include_working) { *out = plan; return MEBPTT_OK; }
    const size_t need = mebptt_lstm_workspace_bytes(desc, plan);
    if (need == 0) { mebptt_plan_free(plan); return MEBPTT_ERR_UNSUPPORTED; }
    if (need <= budget_bytes) { *out = plan; return MEBPTT_OK; }
    // too large by `need - budget_bytes`: give up that many units (the working memory changes
    // little with m, so this lands on or just above the answer; the loop settles the rest).
    // A budget above the mode's saturation point was clamped by the planner: go on from there.
    const int64_t m_used = mebptt_plan_m(plan);
    mebptt_plan_free(plan);
    const int64_t drop = (int64_t)((need - budget_bytes + per_m - 1) / per_m);
    m = (m_used < m ? m_used : m) - (drop > 0 ? drop : 1);
  }
  return MEBPTT_ERR_BUDGET;
}

int mebptt_plan_bytes_exact(const mebptt_lstm_desc* desc, size_t budget_bytes, int use_beta, int include_working,
                            mebptt_plan_t** out) {
  if (!out || !valid_desc(desc)) return MEBPTT_ERR_ARG;
  *out = nullptr;
  Layout y;
  state_layout(desc, y);
  // the finest unit in which a hidden state, an internal state and one without its input state are
  // all whole: their greatest common divisor (a multiple of the layout's granule, as they are)
  const size_t rec_short = y.rec_in;   // output hidden state + gate planes
  const size_t f = gcd_sz(gcd_sz(y.unit, y.rec), rec_short);
  const int sigma = (int)(y.unit / f), alpha = (int)(y.rec / f), beta = use_beta ? (int)(rec_short / f) : 0;
  if (sigma > 64) return MEBPTT_ERR_UNSUPPORTED;
  int64_t m = (int64_t)(budget_bytes / f);
  for (int round = 0; round < 64 && m >= sigma; ++round) {
    mebptt_plan_t* plan = nullptr;
    const int rc = mebptt_plan_sized(desc->t, m, sigma, alpha, beta, &plan);
    if (rc != MEBPTT_OK) return rc;
    if (!include_working) { *out = plan; return MEBPTT_OK; }
    const size_t need = mebptt_lstm_workspace_bytes(desc, plan);
    if (need == 0) { mebptt_plan_free(plan); return MEBPTT_ERR_UNSUPPORTED; }
    if (need <= budget_bytes) { *out = plan; return MEBPTT_OK; }
    const int64_t m_used = mebptt_plan_m(plan);
    mebptt_plan_free(plan);
    const int64_t drop = (int64_t)((need - budget_bytes + f - 1) / f);
    m = (m_used < m ? m_used : m) - (drop > 0 ? drop : 1);
  }
  return MEBPTT_ERR_BUDGET;
}

size_t mebptt_lstm_workspace_bytes(const mebptt_lstm_desc* desc, const mebptt_plan_t* plan) {
  if (check_common(desc, plan) != MEBPTT_OK) return 0;
  Layout y;
  workspace_layout(desc, reinterpret_cast<const Plan*>(plan), y);
  // the persistent kernels address the workspace in 16-byte units held in 32 bits
  if (y.tensor_path && y.total >= ((size_t)1 << 36)) return 0;
  return y.total;
}

size_t mebptt_lstm_working_bytes(const mebptt_lstm_desc* desc, const mebptt_plan_t* plan) {
  if (check_common(desc, plan) != MEBPTT_OK) return 0;
  Layout y;
  workspace_layout(desc, reinterpret_cast<const Plan*>(plan), y);
  return y.total - y.off_core;
}

int64_t mebptt_lstm_launch_count(const mebptt_lstm_desc* desc, const mebptt_plan_t* plan) {
  if (check_common(desc, plan) != MEBPTT_OK) return -1;
  const Plan* p = reinterpret_cast<const Plan*>(plan);
  Layout y;
  workspace_layout(desc, p, y);
  if (y.tensor_path) return tc::run_step(y, p, StepIO{}, desc->want_dx != 0, nullptr, true, false);
  // forward operation: one kernel per layer; backward operation: 5 for the readout and
  // 4 per layer; one to finalise
  const int64_t L = desc->layers;
  if (y.stepwise_tc) {
    // forward operation: two GEMMs and the cell kernel per layer; readout: GEMM with loss, loss
    // term and stage, dha GEMM; backward operation per layer: gate kernel and one or two d_in GEMMs
    // (a contraction that is split along K takes a second launch to add its parts)
    const size_t pf = (size_t)148 * 128 * 128;
    const int G = 4 * y.H;
    const int64_t to_h = tc::gemm_split_count(false, true, y.B, y.H, G, pf) > 1 ? 2 : 1;   // dz W -> [B][H]
    const int64_t to_x = tc::gemm_split_count(false, true, y.B, y.I, G, pf) > 1 ? 2 : 1;   // dz W -> [B][I]
    const int64_t dha = tc::gemm_split_count(false, true, y.B, y.H, y.O, pf) > 1 ? 2 : 1;
    // (the recurrent dh = dz W_hh is one launch in any case: its parts are added by the next gate kernel)
    const int64_t bwd = L + L + to_h * (L - 1) + (desc->want_dx ? to_x : 0);
    const int64_t chunks = (p->t + y.S - 1) / y.S;   // each flushed by 2 L + 1 GEMMs and L + 1 bias sums
    // runs of n >= 2 operations go layer by layer: one input product per layer and run, the
    // readout once per run (stage, GEMM with loss, loss terms, dha), the gradient handed down
    // once per layer and run
    int64_t n_launch = chunks * (3 * L + 2) + 1;
    for (const WorkItem& wi : work_items(p, y.S)) {
      if (wi.kind == WorkItem::LEAF) n_launch += wi.n * (3 * L + 2 + dha + bwd);
      else if (wi.kind == WorkItem::FWD) n_launch += wi.n == 1 ? 3 * L : L * (1 + 2 * (int64_t)wi.n);
      else if (wi.n == 1) n_launch += 2 + dha + bwd;
      else n_launch += 3 + dha + L * wi.n * 2 + (L - 1) * to_h + (desc->want_dx ? to_x : 0);
    }
    return n_launch;
  }
  if (y.stepwise_x3) {
    // weights: 2 packing kernels per layer and 2 for the readout; forward operation: split, GEMM,
    // cell per layer; readout: split, GEMM, loss sum, split, dha GEMM; backward operation per
    // layer: gate kernel, one or two d_in GEMMs; a chunk: 3 GEMMs per product and L + 1 bias sums
    const size_t pf = (size_t)148 * 128 * 128;
    const int G = 4 * y.H;
    const int64_t to_h = tc::gemm_split_count(false, true, y.B, y.H, 3 * G, pf) > 1 ? 2 : 1;
    const int64_t to_x = tc::gemm_split_count(false, true, y.B, y.I, 3 * G, pf) > 1 ? 2 : 1;
    const int64_t dha = tc::gemm_split_count(false, true, y.B, y.H, 3 * y.O, pf) > 1 ? 2 : 1;
    const int64_t bwd = L + L + to_h * (L - 1) + (desc->want_dx ? to_x : 0);   // dh = dz W_hh: one launch in any case
    const int64_t chunks = (p->t + y.S - 1) / y.S;
    // the readout of a run of n >= 2 backward operations is taken once for the run (the same
    // launches), and a run of n >= 2 forward operations splits its operands once per layer (then
    // GEMM and cell kernel per step)
    int64_t readouts = 0, forwards = 0;
    for (const WorkItem& wi : work_items(p, y.S)) {
      if (wi.kind == WorkItem::LEAF) { readouts += wi.n * (4 + dha); forwards += wi.n * 3 * L; }
      else if (wi.kind == WorkItem::BWD) readouts += 4 + dha;
      else forwards += wi.n == 1 ? 3 * L : L * (1 + 2 * (int64_t)wi.n);
    }
    return 2 * L + 2 + forwards + readouts + p->t * bwd + chunks * (3 * (2 * L + 1) + L + 1) + 1;
  }
  // (a GRU layer's backward operation takes two launches more: its weight gradient comes in three blocks)
  return p->cost * L + p->t * (5 + (y.gru ? 6 : 4) * L) + 1;
}

}  // extern "C"

namespace mebptt {
int train_step_impl(const mebptt_lstm_desc* desc, const mebptt_plan_t* plan, const void* W, const void* b,
                    const void* W_out, const void* b_out, const void* x, const void* targets, const void* h0,
                    const void* c0, void* workspace, size_t workspace_bytes, void* stream, float* loss, float* dW,
                    float* db, float* dW_out, float* db_out, float* dx, int64_t* counters, bool side_stream) {
  int rc = check_common(desc, plan);
  if (rc != MEBPTT_OK) return rc;
  if (!W || !b || !W_out || !b_out || !x || !targets || !h0 || !c0) return MEBPTT_ERR_ARG;
  if (!loss || !dW || !db || !dW_out || !db_out || !counters) return MEBPTT_ERR_ARG;
  if (desc->want_dx && !dx) return MEBPTT_ERR_ARG;
  const Plan* p = reinterpret_cast<const Plan*>(plan);
  Layout y;
  workspace_layout(desc, p, y);
  if (y.tensor_path && y.total >= ((size_t)1 << 36)) return MEBPTT_ERR_UNSUPPORTED;   // 16-byte offsets in 32 bits
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255) || workspace_bytes < y.total)
    return MEBPTT_ERR_WORKSPACE;
  StepIO io{(const char*)W, (const char*)W_out, (const char*)x, (const char*)h0,
            (const float*)b, (const float*)b_out, (const float*)targets, (const float*)c0,
            (char*)workspace, loss, dW, db, dW_out, db_out, dx, counters};
  io.time_runs = (desc->flags & MEBPTT_FLAG_TIME_RUNS) != 0;
  io.pageable_tape = !side_stream;   // the allocation-free entry point (the only caller without side stream) locks no pages
  return run_step(desc, p, y, io, (cudaStream_t)stream, side_stream);
}
}  // namespace mebptt

extern "C" {

int mebptt_lstm_train_step(const mebptt_lstm_desc* desc, const mebptt_plan_t* plan, const void* W,
                           const void* b, const void* W_out, const void* b_out, const void* x,
                           const void* targets, const void* h0, const void* c0, void* workspace,
                           size_t workspace_bytes, void* stream, float* loss, float* dW, float* db,
                           float* dW_out, float* db_out, float* dx, int64_t* counters) {
  return train_step_impl(desc, plan, W, b, W_out, b_out, x, targets, h0, c0, workspace, workspace_bytes, stream, loss,
                         dW, db, dW_out, db_out, dx, counters, true);
}

size_t mebptt_lstm_host_workspace_bytes(const mebptt_lstm_desc* desc, const mebptt_plan_t* plan) {
  if (check_common(desc, plan) != MEBPTT_OK) return 0;
  Layout y;
  workspace_layout(desc, reinterpret_cast<const Plan*>(plan), y);
  Staging g;
  staging_layout(y, desc->want_dx != 0, y.total, g);
  return g.total;
}

int mebptt_lstm_train_step_host(const mebptt_lstm_desc* desc, const mebptt_plan_t* plan, const void* W,
                                const void* b, const void* W_out, const void* b_out, const void* x,
                                const void* targets, const void* h0, const void* c0, void* workspace,
                                size_t workspace_bytes, void* stream, float* loss, float* dW, float* db,
                                float* dW_out, float* db_out, float* dx, int64_t* counters) {
  int rc = check_common(desc, plan);
  if (rc != MEBPTT_OK) return rc;
  if (!W || !b || !W_out || !b_out || !x || !targets || !h0 || !c0) return MEBPTT_ERR_ARG;
  if (!loss || !dW || !db || !dW_out || !db_out || !counters) return MEBPTT_ERR_ARG;
  if (desc->want_dx && !dx) return MEBPTT_ERR_ARG;
  const Plan* p = reinterpret_cast<const Plan*>(plan);
  Layout y;
  workspace_layout(desc, p, y);
  Staging g;
  staging_layout(y, desc->want_dx != 0, y.total, g);
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255) || workspace_bytes < g.total)
    return MEBPTT_ERR_WORKSPACE;
  char* ws = (char*)workspace;
  cudaStream_t s = (cudaStream_t)stream;
  cudaMemcpyAsync(ws + g.W, W, g.nW, cudaMemcpyHostToDevice, s);
  cudaMemcpyAsync(ws + g.b, b, g.nb, cudaMemcpyHostToDevice, s);
  cudaMemcpyAsync(ws + g.W_out, W_out, g.nW_out, cudaMemcpyHostToDevice, s);
  cudaMemcpyAsync(ws + g.b_out, b_out, g.nb_out, cudaMemcpyHostToDevice, s);
  cudaMemcpyAsync(ws + g.h0, h0, g.nh0, cudaMemcpyHostToDevice, s);
  cudaMemcpyAsync(ws + g.c0, c0, g.nc0, cudaMemcpyHostToDevice, s);
  // x is read progressively by the forward pass and the targets not before the first backward
  // operation: the tensor-core path copies both beside the forward pass
  const bool late_targets = y.tensor_path && !env::no_overlap();
  if (!late_targets) {
    cudaMemcpyAsync(ws + g.x, x, g.nx, cudaMemcpyHostToDevice, s);
    cudaMemcpyAsync(ws + g.targets, targets, g.ntargets, cudaMemcpyHostToDevice, s);
  }
  if (cudaGetLastError() != cudaSuccess) return MEBPTT_ERR_CUDA;
  StepIO io{ws + g.W, ws + g.W_out, ws + g.x, ws + g.h0,
            (const float*)(ws + g.b), (const float*)(ws + g.b_out), (const float*)(ws + g.targets),
            (const float*)(ws + g.c0), ws,
            (float*)(ws + g.loss), (float*)(ws + g.dW), (float*)(ws + g.db), (float*)(ws + g.dW_out),
            (float*)(ws + g.db_out), desc->want_dx ? (float*)(ws + g.dx) : nullptr,
            (int64_t*)(ws + g.counters)};
  if (late_targets) {
    io.targets_host = targets; io.targets_bytes = g.ntargets;
    io.x_host = x; io.x_bytes = g.nx;
  }
  io.time_runs = (desc->flags & MEBPTT_FLAG_TIME_RUNS) != 0;
  rc = run_step(desc, p, y, io, s);
  if (rc != MEBPTT_OK) return rc;
  cudaMemcpyAsync(loss, ws + g.loss, 4, cudaMemcpyDeviceToHost, s);
  cudaMemcpyAsync(dW, ws + g.dW, y.w_total_elems() * 4, cudaMemcpyDeviceToHost, s);
  cudaMemcpyAsync(db, ws + g.db, g.nb, cudaMemcpyDeviceToHost, s);
  cudaMemcpyAsync(dW_out, ws + g.dW_out, (size_t)y.O * y.H * 4, cudaMemcpyDeviceToHost, s);
  cudaMemcpyAsync(db_out, ws + g.db_out, g.nb_out, cudaMemcpyDeviceToHost, s);
  if (desc->want_dx) cudaMemcpyAsync(dx, ws + g.dx, g.ndx, cudaMemcpyDeviceToHost, s);
  cudaMemcpyAsync(counters, ws + g.counters, 8 * sizeof(int64_t), cudaMemcpyDeviceToHost, s);
  return cudaGetLastError() == cudaSuccess ? MEBPTT_OK : MEBPTT_ERR_CUDA;
}

int mebptt_lstm_run_times(double* ms, int64_t* launches, int64_t* ops) { return tc::run_times(ms, launches, ops); }

int mebptt_lstm_prepare(const mebptt_lstm_desc* desc, const mebptt_plan_t* plan) {
  const int rc = check_common(desc, plan);
  if (rc != MEBPTT_OK) return rc;
  const Plan* p = reinterpret_cast<const Plan*>(plan);
  Layout y;
  workspace_layout(desc, p, y);
  if (!y.tensor_path) return MEBPTT_OK;   // the other paths walk the plan's tape as it is
  return tc::prepare_host(y, p, desc->want_dx != 0);
}

int mebptt_test_wait_fault(int mask) {
  if (mask < 0 || mask > 7) return MEBPTT_ERR_ARG;
  tc::set_wait_fault_mask(mask);
  return MEBPTT_OK;
}

int mebptt_lstm_prepare_stats(int64_t* out) {
  if (!out) return MEBPTT_ERR_ARG;
  tc::prepare_stats(out);
  return MEBPTT_OK;
}

int mebptt_gemm_bf16(const void* A, int64_t lda, int a_major, const void* B, int64_t ldb, int b_major, float* C,
                     int64_t ldc, int accumulate, const float* bias, int64_t M, int64_t N, int64_t K, int* status,
                     void* stream) {
  if (!A || !B || !C || M < 1 || N < 1 || K < 1 || M > (1 << 30) || N > (1 << 30) || K > (1 << 30))
    return MEBPTT_ERR_ARG;
  if ((lda & 7) || (ldb & 7) || (reinterpret_cast<uintptr_t>(A) & 15) || (reinterpret_cast<uintptr_t>(B) & 15))
    return MEBPTT_ERR_ARG;
  if ((a_major != 0 && a_major != 1) || (b_major != 0 && b_major != 1)) return MEBPTT_ERR_ARG;
  tc::GemmOut out{accumulate ? tc::GemmOut::ACCUM_F32 : tc::GemmOut::STORE_F32, C, ldc, bias, 0};
  return tc::gemm_bf16(A, lda, a_major == 1, B, ldb, b_major == 1, out, (int)M, (int)N, (int)K, status,
                       (cudaStream_t)stream);
}

int mebptt_slot_copy(void* dst, const void* src, size_t bytes, void* stream) {
  if (!dst || !src) return MEBPTT_ERR_ARG;
  if ((reinterpret_cast<uintptr_t>(dst) & 15) || (reinterpret_cast<uintptr_t>(src) & 15) || (bytes & 15))
    return MEBPTT_ERR_ARG;
  generic::copy_bytes(dst, src, bytes, (cudaStream_t)stream);
  return cudaGetLastError() == cudaSuccess ? MEBPTT_OK : MEBPTT_ERR_CUDA;
}

}  // extern "C"
