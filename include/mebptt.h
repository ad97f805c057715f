/*
 * mebptt.h -- memory-efficient backpropagation through time for LSTMs on one GPU.
 *
 * C interface of libmebptt.  Two groups of calls:
 *
 *   1. Planning (host only, no CUDA): solve the dynamic programs of the paper for a sequence
 *      of length t and a memory budget m, in one of three schemes -- hidden-state
 *      memorisation (BPTT-HSM, Section 3.1), internal-state memorisation (BPTT-ISM,
 *      Section 3.2) or mixed memorisation (BPTT-MSM, Sections 3.3 and 3.4) -- and unroll the
 *      execution protocol (Algorithm 2; Section 3.2 steps 1-4) into a linear tape.
 *
 *   2. Execution (device): one LSTM training step -- forward steps, recomputed forward
 *      steps and backward steps in the order of the tape -- producing the loss and the
 *      gradients of ordinary BPTT (Section 2.1) while holding no more than the budget.
 *
 * Conventions
 *   - Every function returns an int status (MEBPTT_OK = 0, errors < 0) unless it returns a
 *     value that cannot fail.  Nothing aborts, nothing throws.
 *   - The library never allocates device memory.  The caller owns all device buffers and a
 *     workspace whose size mebptt_lstm_workspace_bytes() reports.  Plans are host objects
 *     owned by the library and released with mebptt_plan_free().
 *   - Device work is enqueued on the caller's stream and the call returns without waiting.
 *     Errors that only the device can see are written to counters[3].
 *   - All matrices are dense and row-major.
 *
 * Units of the budget m (they differ by scheme, as in the paper)
 *   - HSM, MSM: m counts hidden states.  The start state (h0, c0) is one of them; the single
 *     working RNN core is not (Section 3.1: C(t, m) = 2t - 1 needs m >= t).
 *   - ISM: m counts internal states, the one being worked on included; the initial hidden
 *     state is free (Section 3.2: C(t, m) = t needs m >= t).
 *   - An internal state takes alpha hidden-state units (beta when its input hidden state is
 *     already stored and the Section 3.4 variant is on).  For the LSTM layouts of this
 *     library alpha = 4 and beta = 3 (see mebptt_lstm_desc).
 */
#ifndef MEBPTT_H
#define MEBPTT_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* ---- enumerations ------------------------------------------------------------------ */
enum { MEBPTT_HSM = 0, MEBPTT_ISM = 1, MEBPTT_MSM = 2,
       MEBPTT_CHEN_SQRT = 3,      /* reported by plans made with mebptt_plan_chen_sqrt; not accepted by mebptt_plan */
       MEBPTT_CHEN_RECURSIVE = 4  /* likewise for mebptt_plan_chen_recursive */ };

enum {
  MEBPTT_OK = 0,
  MEBPTT_ERR_ARG = -1,         /* null pointer, non-positive size, unknown enum value       */
  MEBPTT_ERR_BUDGET = -2,      /* m < 1: no policy exists                                   */
  MEBPTT_ERR_WORKSPACE = -3,   /* workspace missing, misaligned (256 B) or too small         */
  MEBPTT_ERR_UNSUPPORTED = -4, /* shape / precision / plan this build cannot run             */
  MEBPTT_ERR_CUDA = -5,        /* a CUDA runtime call failed                                 */
  MEBPTT_ERR_TIMEOUT = -6,     /* a bounded device-side wait expired (reported in counters)  */
  MEBPTT_ERR_OOM = -7,         /* host allocation failed                                     */
  MEBPTT_ERR_PLAN = -8         /* tape failed validation                                     */
};

enum { MEBPTT_FP32 = 0, MEBPTT_TF32 = 1, MEBPTT_BF16 = 2 };

/* ---- the tape ---------------------------------------------------------------------- */
/*
 * Algorithm 2 recurses on (t, m, s); its shape depends on the tables only, never on data, so
 * it is unrolled once into a list of operations.  Two kinds exist:
 *
 *   MEBPTT_OP_FWD  one forward operation (the unit of cost, Section 3.1): reads the hidden
 *                  state of step k-1 at location `src`, writes the state of step k at `dst`.
 *                  dst_fmt tells what is written: MEBPTT_FMT_HIDDEN (h_k, c_k only),
 *                  MEBPTT_FMT_INTERNAL (the whole internal state of Definition 3) or
 *                  MEBPTT_FMT_INTERNAL_NOINPUT (the same without the copy of the input hidden
 *                  state, Section 3.4).
 *   MEBPTT_OP_BWD  one backward operation over step k: reads the internal state at `src`
 *                  (and, for FMT_INTERNAL_NOINPUT, the hidden state of step k-1 at `aux`).
 *
 * Locations: >= 0 is an offset, in hidden-state units, into the slot arena (a stack: states are
 * read in the reverse order of writing, Section 3.1); negative values name buffers outside the
 * budget: the caller's initial state, the two scratch hidden states a forward sweep alternates
 * between, and the working core (the one RNN core that Section 3.1 keeps for intermediate calculations,
 * outside the budget m).  A memorisation is therefore not a copy: the forward operation
 * that produces the state writes it where it will be kept (Push), and the next forward
 * operation reads it from there (Peek).
 */
enum { MEBPTT_OP_FWD = 1, MEBPTT_OP_BWD = 2 };
enum { MEBPTT_FMT_HIDDEN = 0, MEBPTT_FMT_INTERNAL = 1, MEBPTT_FMT_INTERNAL_NOINPUT = 2 };
enum { MEBPTT_LOC_INIT = -1, MEBPTT_LOC_PING = -2, MEBPTT_LOC_PONG = -3, MEBPTT_LOC_CORE = -4 };

typedef struct {
  int32_t kind;     /* MEBPTT_OP_FWD or MEBPTT_OP_BWD                          */
  int32_t k;        /* time step, 1 .. t                                       */
  int32_t src;      /* location read                                           */
  int32_t dst;      /* FWD: location written; BWD: unused (0)                  */
  int32_t dst_fmt;  /* FWD: MEBPTT_FMT_*; BWD: format of the record at src     */
  int32_t aux;      /* BWD with FMT_INTERNAL_NOINPUT: location of state k-1    */
  int32_t units;    /* arena units in use (paper's accounting) after this op   */
  int32_t reserved;
} mebptt_op;

/* ---- planning ---------------------------------------------------------------------- */
typedef struct mebptt_plan mebptt_plan_t; /* opaque, host memory, library-owned */

/*
 * Solve the DP for (t, m, mode) and build the tape.
 *   HSM: Eqs. (1)-(3) with C(t,1) = t(t+1)/2, C(1,m) = 1            (Section 3.1, Algorithm 1)
 *   ISM: Eqs. (4)-(5) with C(0,m) = 0                               (Section 3.2)
 *   MSM: Eqs. (6)-(9) with C(0,.) = 0, C(t>0, m<=0) = inf           (Section 3.3)
 * alpha = 4, the Section 3.4 variant off.  argmin ties: smallest y (Algorithm 1 scans upward
 * with a strict <); hidden state before internal state.
 * t >= 1.  m < 1 gives MEBPTT_ERR_BUDGET.  m above the point where the cost stops falling
 * (t for HSM/ISM, alpha (t-1) + 1 for MSM) is clamped to it: same policy, same cost.
 * *out receives the plan; the caller releases it with mebptt_plan_free.
 */
int mebptt_plan(int64_t t, int64_t m, int mode, mebptt_plan_t **out);

/*
 * As above with explicit alpha >= 2 (Section 3.3) and beta: 0 switches the Section 3.4 variant
 * off, 1 <= beta <= alpha switches it on (Eq. (10): an internal state pushed at y = 1 is charged
 * beta units because its input hidden state is the stored start state).  Ignored for HSM; ISM
 * uses alpha only to size its slots.
 */
int mebptt_plan_ex(int64_t t, int64_t m, int mode, int alpha, int beta, mebptt_plan_t **out);

/*
 * Chen's sqrt(t) schedule (Section 2.2) as a plan for the same executor, for comparison with the
 * DP policies (Sections 4.1, 4.2): segments of ceil(sqrt(t)) steps, hidden states memorised at the
 * segment boundaries in one forward pass, then every internal state of one segment at a time.
 * beta > 0: internal states are stored without their input hidden state (beta units each, the
 * accounting of Section 4.2); beta = 0: with it (alpha units each).  The plan's m is set to the
 * memory the schedule needs (mebptt_plan_peak_units); its cost is t plus the length of all
 * segments but the last.  It carries no DP tables (mebptt_plan_tables returns NULL pointers).
 */
int mebptt_plan_chen_sqrt(int64_t t, int alpha, int beta, mebptt_plan_t **out);

/*
 * Chen's recursive schedule (Section 2.2), likewise: a sequence of more than k steps is cut into
 * k + 1 parts as equal as they come (the first ones a step longer), one forward pass memorises the
 * hidden states at the k cuts, and the parts are treated the same way from the last to the first;
 * a sequence of at most k steps is run forward keeping every internal state and backpropagated.
 * k = 1 is bisection, the least memory the scheme can do with (about log2 t hidden states).
 * Reading of the paper's one-paragraph summary: "k" counts the states memorised per level, which
 * is what its memory figure O(k log_{k+1} t) and its minimum log2 t at k = 1 need.
 * alpha, beta, m, cost and tables as for mebptt_plan_chen_sqrt.  1 <= k <= 4096.
 */
int mebptt_plan_chen_recursive(int64_t t, int k, int alpha, int beta, mebptt_plan_t **out);

void mebptt_plan_free(mebptt_plan_t *plan);

/* C(t, m): the predicted number of forward operations (Section 3.1). */
int64_t mebptt_plan_cost(const mebptt_plan_t *plan);
/* Number of tape entries: C(t, m) forward + t backward operations. */
int64_t mebptt_plan_num_ops(const mebptt_plan_t *plan);
/* The tape (host memory, valid until mebptt_plan_free). */
const mebptt_op *mebptt_plan_tape(const mebptt_plan_t *plan);
/* Peak memory in the paper's units for this scheme (see "Units" above); <= m. */
int64_t mebptt_plan_peak_units(const mebptt_plan_t *plan);
/* Hidden-state units the slot arena must physically hold (the caller's start state is read in
 * place, so this is peak - 1 for HSM/MSM and alpha * peak for ISM). */
int64_t mebptt_plan_arena_units(const mebptt_plan_t *plan);
/* Parameters after clamping. */
int64_t mebptt_plan_t_len(const mebptt_plan_t *plan);
int64_t mebptt_plan_m(const mebptt_plan_t *plan);
int mebptt_plan_mode(const mebptt_plan_t *plan);
int mebptt_plan_alpha(const mebptt_plan_t *plan);
int mebptt_plan_beta(const mebptt_plan_t *plan);

/*
 * Borrowed pointers to the DP tables, row-major [t_dim][m_dim] with t_dim = t + 1 and
 * m_dim = m + 1 (row / column 0 included).  C: costs, MEBPTT_INF where infeasible.
 * D: position of the first push (HSM, ISM: Eq. (3), (5); MSM: D1 of Eq. (8)).
 * D2, H: MSM only (Eq. (8), (9); H is 1 = hidden, 2 = internal), NULL otherwise.
 * Any output pointer may be NULL.
 */
#define MEBPTT_INF ((int64_t)1 << 60)
int mebptt_plan_tables(const mebptt_plan_t *plan, const int64_t **C, const int32_t **D,
                       const int32_t **D2, const uint8_t **H, int64_t *t_dim, int64_t *m_dim);

/*
 * Replay the tape on the host with integer bookkeeping: every forward operation must find
 * its input state, every backward operation its internal state, live states are never
 * overwritten, backward operations come in the order t .. 1, the forward count equals
 * C(t, m) and the units in use never exceed m.  MEBPTT_OK or MEBPTT_ERR_PLAN.
 * mebptt_plan() already ran it; the call exists for tapes' users and tests.
 */
int mebptt_plan_validate(const mebptt_plan_t *plan);

/* ---- execution --------------------------------------------------------------------- */
/*
 * A stack of `layers` LSTM cells without peepholes (the paper names the LSTM, Section 4,
 * without printing it), gate order i, f, g, o:
 *     z = W [in_t ; h_{t-1}] + b,  i,f,o = sigmoid, g = tanh,
 *     c_t = f c_{t-1} + i g,  h_t = o tanh(c_t),
 * in_t = x_t for layer 0 and the h_t of the layer below otherwise; the RNN core of
 * Definition 1 is the whole stack at one time step and its hidden state (Definition 2) is
 * (h, c) of every layer.  On top: y_t = W_out h_t + b_out (last layer) and the loss
 *     L = sum_t 1/(batch*readout) sum (y_t - target_t)^2,
 * a sum of per-step terms as Algorithm 2 requires (the output gradient is asked for at each
 * step).
 *
 * dtype selects storage and arithmetic:
 *   MEBPTT_FP32  everything float32, FMA arithmetic.
 *   MEBPTT_TF32  everything stored as float32; contractions on tensor cores (each float32
 *                product as three bfloat16 products of 16-bit-mantissa halves, float32
 *                accumulation: at least tf32 accuracy) where the widths are multiples of 8
 *                and the batch a multiple of 32, in float32 FMA arithmetic elsewhere.
 *   MEBPTT_BF16  operands (W, W_out, x, h0 and every stored h and gate) bfloat16; b, b_out,
 *                targets, c0, every stored c, all accumulation and all gradients float32.
 * With these layouts an internal state (h_t, c_t, the four gates, h_{t-1}, c_{t-1}) fits in
 * alpha = 4 hidden-state units, beta = 3 without the input hidden state; plans made with a
 * smaller alpha are refused (MEBPTT_ERR_UNSUPPORTED).
 */
typedef struct {
  int32_t layers;   /* >= 1                                           */
  int32_t input;    /* I: width of x_t                                */
  int32_t hidden;   /* H: per layer                                   */
  int32_t readout;  /* O: width of y_t and of the targets             */
  int32_t batch;    /* B                                              */
  int32_t dtype;    /* MEBPTT_FP32 | MEBPTT_TF32 | MEBPTT_BF16        */
  int32_t want_dx;  /* 1: also return dL/dx                           */
  int32_t flags;    /* MEBPTT_FLAG_* or 0                             */
  int64_t t;        /* sequence length; must equal the plan's         */
} mebptt_lstm_desc;

/* Run on the CUDA-core kernels even where the tensor-core kernels cover the shape (the two
 * paths round differently; results are deterministic within each). */
enum { MEBPTT_FLAG_NO_TENSOR_CORES = 1 };
/* Measurement aid: bracket every launch of the two persistent kernels of the tensor-core path
 * (forward runs, backward runs) with a pair of CUDA events on the caller's stream, to be
 * collected by mebptt_lstm_run_times.  Each pair costs a few microseconds of stream time, so a
 * step that is timed as a whole should not set it.  Ignored by the CUDA-core path. */
enum { MEBPTT_FLAG_TIME_RUNS = 2 };
/* The recurrent core is a GRU instead of an LSTM (Section 1: the method does not depend on the
 * architecture of the core; plans, tape, budgets and every entry point are the same):
 *     r = sigmoid(W_r [x_t ; h_{t-1}] + b_r),   z = sigmoid(W_z [x_t ; h_{t-1}] + b_z),
 *     q = W_hn h_{t-1},   n = tanh(W_xn x_t + b_n + r q),   h_t = (1 - z) n + z h_{t-1}.
 * W is then [3H][I_l + H] per layer (row blocks r, z, n), b [3H], and so are dW, db.  The hidden
 * state is h alone: c0 is not read, and the cell-state part of a memory slot stays unused, so the
 * sizes of slots and the units of m are those of the LSTM layout (alpha = 4: h_t, the planes r, z,
 * n, q, and h_{t-1}).  Runs on the CUDA-core kernels in every precision (MEBPTT_TF32 = MEBPTT_FP32). */
enum { MEBPTT_FLAG_GRU = 4 };

/* Bytes of one hidden-state unit (all layers) for this descriptor; 0 on a bad descriptor. */
size_t mebptt_lstm_unit_bytes(const mebptt_lstm_desc *desc);

/* Budget given in bytes -> hidden-state units (floor); the working memory outside the budget
 * is not counted (Section 3.1 sets the working core apart). */
int64_t mebptt_budget_bytes_to_units(const mebptt_lstm_desc *desc, size_t bytes);

/*
 * Plan from a budget given in bytes (config 5 of the benchmark states its budgets that way).
 * The bytes are turned into the mode's own unit -- hidden-state units for HSM and MSM, internal
 * states (alpha = 4 units each) for ISM -- and the policy is that of mebptt_plan for that m.
 *   include_working = 0: the budget is what the paper budgets, the memorised states only
 *                        (Section 3 keeps the working core outside m).
 *   include_working = 1: the budget is the whole device workspace of a training step: the largest
 *                        m is taken for which mebptt_lstm_workspace_bytes of the resulting plan
 *                        still fits.  (Appendix C notes that the working memory has to be part
 *                        of the allowance once it is not negligible; here it is not: staging for
 *                        a chunk of time steps, packed weights.)
 * MEBPTT_ERR_BUDGET if not even m = 1 fits.  *out as for mebptt_plan.
 */
int mebptt_plan_for_bytes(const mebptt_lstm_desc *desc, size_t budget_bytes, int mode, int include_working,
                          mebptt_plan_t **out);

/* Size of the device workspace mebptt_lstm_train_step needs: the slot arena sized by the plan
 * plus working memory outside the budget.  0 on error. */
size_t mebptt_lstm_workspace_bytes(const mebptt_lstm_desc *desc, const mebptt_plan_t *plan);
/* The part of that workspace that is not the slot arena. */
size_t mebptt_lstm_working_bytes(const mebptt_lstm_desc *desc, const mebptt_plan_t *plan);

/* Number of kernel launches one mebptt_lstm_train_step enqueues for this descriptor and plan
 * (memsets not counted); -1 on error. */
int64_t mebptt_lstm_launch_count(const mebptt_lstm_desc *desc, const mebptt_plan_t *plan);

/*
 * One training step under the plan (Algorithm 2 for HSM; the four steps of Section 3.2 for
 * ISM; Section 3.3 for MSM).  All pointers are DEVICE pointers unless said otherwise.
 *
 * Read-only inputs (never written):
 *   W        layers concatenated; layer l is [4H][I_l + H] with I_0 = I, I_l = H; operand type
 *   b        [layers][4H] float32
 *   W_out    [O][H] operand type;  b_out [O] float32
 *   x        [t][B][I] operand type;  targets [t][B][O] float32
 *   h0       [layers][B][H] operand type;  c0 [layers][B][H] float32
 * Workspace: caller-owned, 256-byte aligned, >= mebptt_lstm_workspace_bytes(); contents on
 *   entry do not matter and are undefined on exit.
 * stream: a cudaStream_t (NULL = the default stream).
 * Streams and events owned by the library: on the tensor-core path for one-layer bfloat16
 *   problems, the first step on a device creates, and keeps until the process ends, four
 *   non-blocking streams and 28 events without timing.  On the first (lowest priority) run the
 *   weight-gradient contractions and bias sums of a finished chunk of time steps, inside the
 *   caller's workspace and output buffers, while the caller's stream goes on with the next chunk;
 *   events order them after the backward steps they read and before the reuse of their staging
 *   buffers, and the caller's stream waits for them before the step's last kernel.  The second
 *   (middle priority) computes the input projections of the window of time steps after the one
 *   the forward runs are reading, into the other of two copies of the window buffer inside the
 *   workspace; every forward run that opens a window waits for its projections first, so nothing
 *   of it is left when the step ends.  The third carries the host-to-device copies of
 *   mebptt_lstm_train_step_host that overlap the forward pass.  The fourth (most urgent
 *   priority) is used only on request (MEBPTT_PRIORITY=1 in the environment): the step then runs
 *   there, ordered after what `stream` holds and joined to `stream` at its end.  Everything the
 *   call enqueues is therefore complete when `stream` has reached the end of the call's work; the
 *   caller needs no knowledge of these streams, but must not use the workspace or the outputs on
 *   other streams before that.  mebptt_lstm_train_step_static uses none of them.
 * Outputs (overwritten, not accumulated; all float32):
 *   loss [1]; dW like W; db like b; dW_out [O][H]; db_out [O]; dx [t][B][I] or NULL.
 *   counters: int64[8] -- [0] forward operations executed, [1] backward operations executed,
 *   [2] peak units (paper's accounting), [3] device status (MEBPTT_OK or an error code),
 *   [4..7] reserved.  counters[0] equals mebptt_plan_cost(plan) after a successful step.
 * Determinism: no atomics; for a fixed descriptor and inputs every plan yields bit-identical
 *   outputs (each backward step sees bit-identical internal states whether they were stored
 *   or recomputed, and all accumulations run in the order t .. 1).
 * Returns MEBPTT_OK once everything is enqueued, or an error with nothing enqueued.
 */
int mebptt_lstm_train_step(const mebptt_lstm_desc *desc, const mebptt_plan_t *plan,
                           const void *W, const void *b, const void *W_out, const void *b_out,
                           const void *x, const void *targets, const void *h0, const void *c0,
                           void *workspace, size_t workspace_bytes, void *stream,
                           float *loss, float *dW, float *db, float *dW_out, float *db_out,
                           float *dx, int64_t *counters);

/*
 * The same step for callers whose data lives in HOST memory.  Inputs and outputs are host
 * pointers (pinned memory makes the copies asynchronous); `workspace` is still a DEVICE buffer,
 * of at least mebptt_lstm_host_workspace_bytes(), in which the call stages its copies of the
 * inputs and outputs around the train step.  The call enqueues host-to-device copies, the step
 * and device-to-host copies on `stream`; results are valid after the stream is synchronised.
 */
size_t mebptt_lstm_host_workspace_bytes(const mebptt_lstm_desc *desc, const mebptt_plan_t *plan);
int mebptt_lstm_train_step_host(const mebptt_lstm_desc *desc, const mebptt_plan_t *plan,
                                const void *W, const void *b, const void *W_out,
                                const void *b_out, const void *x, const void *targets,
                                const void *h0, const void *c0,
                                void *workspace, size_t workspace_bytes, void *stream,
                                float *loss, float *dW, float *db, float *dW_out, float *db_out,
                                float *dx, int64_t *counters);

/*
 * Mixed memorisation over the layout's real sizes.  Section 3.3 counts memory in hidden states and
 * wants the internal state to be a whole number alpha of them; where it is not (bfloat16 h and
 * gates with a float32 cell state: 20/6 of a hidden state, 14/6 without the input state) rounding
 * up plans memory that is never used.  Section 3.3 calls alpha application-specific and Appendix C
 * works with slots of arbitrary sizes; here the recursion of Eqs. (6)-(10) runs over a finer unit:
 *
 *   mebptt_plan_sized(t, m, sigma, alpha, beta)  BPTT-MSM where a hidden state takes sigma units of
 *       m, an internal state alpha, one without its input hidden state beta (0: Section 3.4 off);
 *       Q1 recurses on m - sigma, the start state occupies sigma units.  sigma = 1 is
 *       mebptt_plan_ex(MEBPTT_MSM).  1 <= sigma <= 64, sigma <= alpha <= 64 sigma.  Tape locations,
 *       peak and arena units of such a plan are in the same finer unit.
 *   mebptt_plan_bytes_exact(desc, bytes, use_beta, include_working)  takes as the unit the
 *       greatest common divisor of the byte sizes of the three kinds of state in desc's layout
 *       (config 5: 1 MiB, sizes 3 : 10 : 7), converts the byte budget and plans as above; with
 *       include_working the budget covers the whole device workspace, as in mebptt_plan_for_bytes.
 *   mebptt_plan_sigma  the sigma of a plan (1 for every other constructor).
 *
 * A plan can be executed with a descriptor whose layout fits its sizes (checked; else
 * MEBPTT_ERR_UNSUPPORTED).
 */
int mebptt_plan_sized(int64_t t, int64_t m, int sigma, int alpha, int beta, mebptt_plan_t **out);
int mebptt_plan_bytes_exact(const mebptt_lstm_desc *desc, size_t budget_bytes, int use_beta,
                            int include_working, mebptt_plan_t **out);
int mebptt_plan_sigma(const mebptt_plan_t *plan);

/*
 * What a training step derives from (descriptor, plan, workspace address, device) alone -- the
 * runs the tape of Algorithm 2 is cut into, the tape in the form the kernels read, the kernel
 * variants the device can keep resident, the TMA tensor maps -- is prepared once and kept in a
 * small cache inside the library (eight sets, least recently used out first); mebptt_plan_free
 * drops the sets of its plan.  The first mebptt_lstm_train_step of a combination therefore costs
 * some host time (page-locked memory is allocated for the tape); later ones only look the set up,
 * copy the tape asynchronously and enqueue.  (The paper has no counterpart: its Algorithm 2
 * walks the policy tables on the host at every step.)
 *
 * mebptt_lstm_prepare makes the host part of a set ahead of time, or finds it; it needs no GPU
 * and returns a status.  mebptt_lstm_prepare_stats fills out[0..3] (host array) with: sets built
 * since the library was loaded, look-ups served from the cache, sets whose tape lies in
 * page-locked memory, sets held now.
 */
int mebptt_lstm_prepare(const mebptt_lstm_desc *desc, const mebptt_plan_t *plan);
int mebptt_lstm_prepare_stats(int64_t *out);

/*
 * The training step for callers that cannot allocate device memory.  (The paper has no
 * counterpart: it never says where the working memory of an implementation comes from.)
 *
 * mebptt_lstm_train_step wants a workspace from its caller, and a caller normally gets one from
 * cudaMalloc or from an allocator built on it.  That is not always possible where the step runs:
 * a process that has already given all free device memory to something else, a plug-in whose host
 * application hands it input and output buffers and nothing more, or a service in which an
 * allocation would stall the other streams of the device.  This entry point takes the same inputs
 * and outputs and no workspace; it uses a fixed array of MEBPTT_STATIC_WORKSPACE_BYTES that is part
 * of the library image.  It calls no cudaMalloc, cudaFree or other allocating routine, and creates
 * no stream or event.
 *
 *   - Problems whose workspace (mebptt_lstm_workspace_bytes) exceeds the array are refused with
 *     MEBPTT_ERR_WORKSPACE and nothing is enqueued; use mebptt_lstm_train_step for those.
 *   - The first call on each device is a set-up call: it looks up the array's device address
 *     (with that device current).  With CUDA's default lazy module loading that look-up is also
 *     the moment the driver places the array -- and, at their first launch, the code of the
 *     kernels -- in device memory; only with CUDA_MODULE_LOADING=EAGER does this happen when the
 *     library is loaded.  So make one call (any small problem will do) per device while device
 *     memory is still to be had, and before starting any stream capture; it fails with
 *     MEBPTT_ERR_CUDA if the array cannot be placed.  From then on the GPU holds the array until
 *     the process exits, and later calls reserve nothing.
 *   - A descriptor with MEBPTT_FLAG_TIME_RUNS is refused with MEBPTT_ERR_ARG: per-launch timing
 *     creates CUDA events, which this entry point promises not to do.
 *   - All calls on a device share the one array.  Each call clears the parts that must start at
 *     zero, so leftovers of the previous call do not matter, but two calls whose device work
 *     overlaps (different streams, or the ordinary entry point given this memory) race: keep
 *     calls on one stream or order them with events.
 *   - Arguments, layouts, outputs, counters and determinism are those of mebptt_lstm_train_step.
 */
#define MEBPTT_STATIC_WORKSPACE_BYTES (32u << 20)
int mebptt_lstm_train_step_static(const mebptt_lstm_desc *desc, const mebptt_plan_t *plan,
                                  const void *W, const void *b, const void *W_out, const void *b_out,
                                  const void *x, const void *targets, const void *h0, const void *c0,
                                  void *stream,
                                  float *loss, float *dW, float *db, float *dW_out, float *db_out,
                                  float *dx, int64_t *counters);

/*
 * Push / Pop of Algorithm 2 as an explicit copy, for callers that keep states in a pool of
 * their own: copies `bytes` bytes from src to dst (device pointers, both 16-byte aligned,
 * bytes a multiple of 16) on `stream`.  The train step itself writes memorised states in
 * place and does not call this.
 */
int mebptt_slot_copy(void *dst, const void *src, size_t bytes, void *stream);

/*
 * Collects the event pairs recorded on the current device by steps whose descriptor carried
 * MEBPTT_FLAG_TIME_RUNS since the last call: waits for each pair, and returns per class
 * (index 0: forward runs, one launch executes a run of consecutive forward operations of
 * Algorithm 1-3's "execute" steps; index 1: backward runs) the summed elapsed milliseconds,
 * the number of launches and the number of operations they executed.  ms, launches and ops are
 * host arrays of 2 elements.  Returns MEBPTT_OK, MEBPTT_ERR_ARG on a null pointer, or
 * MEBPTT_ERR_CUDA if an event could not be read (the other pairs are still returned).  The
 * paper has no counterpart; it serves the per-kernel figures of a benchmark.
 */
int mebptt_lstm_run_times(double *ms, int64_t *launches, int64_t *ops);

/*
 * The batched contraction the training step uses for everything that is off the recurrence
 * (input projections, readout, weight gradients), exposed for testing and reuse:
 *     C[M][N] (+)= sum_k A(m,k) B(n,k)
 * over bfloat16 operands with float32 accumulation on the tensor cores.  a_major / b_major:
 * 0 = the operand is stored [m][k] (contraction index contiguous), 1 = stored [k][m].
 * lda / ldb: row strides in elements, multiples of 8; A, B 16-byte aligned.  C is float32
 * [M][ldc]; accumulate != 0 adds to it.  bias (nullable): float32 [N], added per column.
 * status (nullable): device int, set to MEBPTT_ERR_TIMEOUT if a bounded wait expires.
 * All pointers are device pointers.  No counterpart in the paper beyond "the RNN core".
 */
int mebptt_gemm_bf16(const void *A, int64_t lda, int a_major, const void *B, int64_t ldb, int b_major,
                     float *C, int64_t ldc, int accumulate, const float *bias,
                     int64_t M, int64_t N, int64_t K, int *status, void *stream);

/*
 * Testing aid for the bounded waits of the tensor-core kernels (no counterpart in the paper).
 * Every wait of those kernels on a step counter or a barrier gives up after a bounded number of
 * polls, reports MEBPTT_ERR_TIMEOUT through the status word (counters[3], or `status` of
 * mebptt_gemm_bf16) and lets the kernel end in the ordinary way.  To see that path run without
 * anything being wrong, a test sets a mask: bit 0 makes the forward run kernel's step counter wait
 * for one CTA more than exist, bit 1 does the same to the backward run kernels, bit 2 makes the
 * first pipeline stage of the batched contraction wait for 16 bytes more than its copies bring;
 * the waits concerned then give up after a few thousand polls.  No memory is touched that an
 * ordinary run would not touch.  mask = 0 restores normal behaviour; the setting is per process
 * and meant for single-threaded tests only.  Returns MEBPTT_ERR_ARG for a mask outside 0..7.
 */
int mebptt_test_wait_fault(int mask);

const char *mebptt_strerror(int status);

#ifdef __cplusplus
}
#endif
#endif /* MEBPTT_H */
