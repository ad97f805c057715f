// Host-side planner: the dynamic programs of Sections 3.1-3.4 and the unrolling of the
// execution protocol (Algorithm 2; Section 3.2, steps 1-4) into a linear tape.
//
// Tables are kept column-major while they are filled (for a fixed budget m the scan over the
// split point y walks one column forwards and one backwards), then transposed once into the
// row-major layout the C interface documents.
#include "plan.hpp"
#include "env.hpp"

#include <algorithm>
#include <atomic>
#include <cstdlib>
#include <cstring>
#include <limits>
#include <new>
#include <system_error>
#include <thread>

namespace mebptt {
namespace tc { void forget_plan(uint64_t plan_id); }
namespace {
Plan* new_plan() {
  static std::atomic<uint64_t> next_id{1};
  Plan* p = new (std::nothrow) Plan();
  if (p) p->id = next_id.fetch_add(1);
  return p;
}
}  // namespace
}  // namespace mebptt

namespace mebptt {

namespace {

// ---------------------------------------------------------------------------------------
// min / first-argmin of  base + i + a[i] + b[-i]  over i = 0 .. n-1  (a ascending, b descending)
// Two passes: a vectorisable reduction, then a search for the first index that attains it.
// ---------------------------------------------------------------------------------------
template <class T>
#if defined(__GNUC__) && defined(__x86_64__)
__attribute__((target_clones("avx2", "default")))
#endif
T scan_min(const T* a, const T* b_last, int64_t n, T base) {
  T best = std::numeric_limits<T>::max();
  for (int64_t i = 0; i < n; ++i) {
    T v = (T)(base + (T)i + a[i] + b_last[-i]);
    best = v < best ? v : best;
  }
  return best;
}

template <class T>
int64_t first_index(const T* a, const T* b_last, int64_t n, T base, T value) {
  for (int64_t i = 0; i < n; ++i)
    if ((T)(base + (T)i + a[i] + b_last[-i]) == value) return i;
  return -1;
}

// First argmin of  i + a[i] + b[-i]  over i = 0 .. n-1 when that sequence is convex in i: a local
// minimum is then the global one, and walking from a nearby guess (the answer for the previous
// t) costs O(1) on average instead of a scan.  Left first, through ties, so that the smallest
// index wins exactly as in the scan.
template <class T>
int64_t convex_first_argmin(const T* a, const T* b_last, int64_t n, int64_t guess) {
  auto f = [&](int64_t j) { return (T)((T)j + a[j] + b_last[-j]); };
  int64_t i = guess < 0 ? 0 : (guess > n - 1 ? n - 1 : guess);
  T v = f(i);
  bool moved = false;
  while (i > 0) {
    const T w = f(i - 1);
    if (w > v) break;
    v = w; --i; moved = true;
  }
  if (!moved) {
    while (i < n - 1) {
      const T w = f(i + 1);
      if (w >= v) break;
      v = w; ++i;
    }
  }
  return i;
}

// A column of costs seen as a sequence in t: the longest prefix lo .. hi of it that is finite and
// convex (second differences >= 0), extended one element at a time.  Appendix A remarks that the
// O(t^2 m) scan can be brought down to O(t m) through convexity in t; the paper does not
// prove convexity, so it is checked on the numbers before it is used, and wherever it fails the
// scan is kept.
template <class T>
struct ConvexPrefix {
  const T* c;
  int64_t lo, hi;   // c[lo .. hi] is finite and convex; hi = lo - 1 while empty
  ConvexPrefix(const T* col, int64_t first) : c(col), lo(first), hi(first - 1) {}
  // c[t] has just been written (or is being read in order); returns whether the prefix now reaches t
  bool extend(int64_t t, T inf) {
    if (hi != t - 1 || c[t] >= inf) return false;
    if (t - lo >= 2 && (int64_t)c[t] - c[t - 1] < (int64_t)c[t - 1] - c[t - 2]) return false;
    hi = t;
    return true;
  }
  void extend_to(int64_t t_max, T inf) {
    for (int64_t t = hi + 1; t <= t_max && extend(t, inf); ++t) {}
  }
};

// verification aid: keeps the plain scan everywhere (the tests compare the two)
inline bool plan_scan_only() { return env::plan_scan(); }

template <class T>
struct Inf;
template <>
struct Inf<int32_t> {
  static constexpr int32_t v = 1 << 29;  // three of them fit
};
template <>
struct Inf<int64_t> {
  static constexpr int64_t v = (int64_t)1 << 60;
};

// Column-major working tables: col(m)[t].
template <class T>
struct Cols {
  int64_t t_dim, m_dim;
  std::vector<T> v;
  Cols(int64_t t, int64_t m, T fill) : t_dim(t + 1), m_dim(m + 1), v((size_t)(t + 1) * (m + 1), fill) {}
  T* col(int64_t m) { return v.data() + (size_t)m * t_dim; }
};

template <class T>
void solve_hsm(int64_t t_max, int64_t m_max, Cols<T>& C, Cols<int32_t>& D) {
  // Section 3.1: C(1, m) = 1, C(t, 1) = t (t + 1) / 2,
  // C(t, m) = min_{1 <= y < t} y + C(t - y, m - 1) + C(y, m).
  const T INF = Inf<T>::v;
  const bool scan_only = plan_scan_only();
  for (int64_t m = 1; m <= m_max; ++m) {
    T* c = C.col(m);
    int32_t* d = D.col(m);
    std::fill(d, d + t_max + 1, 0);
    c[1] = 1;
    if (m == 1) {
      for (int64_t t = 1; t <= t_max; ++t) c[t] = (T)(t * (t + 1) / 2);
      continue;
    }
    const T* cm1 = C.col(m - 1);
    ConvexPrefix<T> cur(c, 1), prev(cm1, 1);
    if (!scan_only) prev.extend_to(t_max, INF);
    cur.extend(1, INF);
    int64_t guess = 0;
    for (int64_t t = 2; t <= t_max; ++t) {
      // y = 1 + i, i = 0 .. t-2 :  (1 + i) + c[1 + i] + cm1[t - 1 - i]
      if (!scan_only && cur.hi >= t - 1 && prev.hi >= t - 1) {
        // c on [1, t-1] and cm1 on [1, t-1] are convex, hence so is the sum over the split point
        guess = convex_first_argmin<T>(c + 1, cm1 + (t - 1), t - 1, guess);
        c[t] = (T)((T)1 + (T)guess + c[1 + guess] + cm1[t - 1 - guess]);
        d[t] = (int32_t)(1 + guess);
      } else {
        T best = scan_min<T>(c + 1, cm1 + (t - 1), t - 1, (T)1);
        if (best >= INF) { c[t] = INF; continue; }
        c[t] = best;
        guess = first_index<T>(c + 1, cm1 + (t - 1), t - 1, (T)1, best);
        d[t] = (int32_t)(1 + guess);
      }
      cur.extend(t, INF);
    }
  }
}

template <class T>
void solve_ism(int64_t t_max, int64_t m_max, Cols<T>& C, Cols<int32_t>& D) {
  // Section 3.2: C(0, m) = 0, C(t > 0, 0) = inf,
  // C(t, m) = min_{1 <= y <= t} y + C(y - 1, m) + C(t - y, m - 1).
  const T INF = Inf<T>::v;
  const bool scan_only = plan_scan_only();
  for (int64_t m = 0; m <= m_max; ++m) {
    C.col(m)[0] = 0;
    std::fill(D.col(m), D.col(m) + t_max + 1, 0);
  }
  for (int64_t m = 1; m <= m_max; ++m) {
    T* c = C.col(m);
    int32_t* d = D.col(m);
    const T* cm1 = C.col(m - 1);
    ConvexPrefix<T> cur(c, 0), prev(cm1, 0);
    if (!scan_only) prev.extend_to(t_max, INF);
    cur.extend(0, INF);
    int64_t guess = 0;
    for (int64_t t = 1; t <= t_max; ++t) {
      // y = 1 + i, i = 0 .. t-1 :  (1 + i) + c[i] + cm1[t - 1 - i]
      if (!scan_only && cur.hi >= t - 1 && prev.hi >= t - 1) {
        guess = convex_first_argmin<T>(c, cm1 + (t - 1), t, guess);
        c[t] = (T)((T)1 + (T)guess + c[guess] + cm1[t - 1 - guess]);
        d[t] = (int32_t)(1 + guess);
      } else {
        T best = scan_min<T>(c, cm1 + (t - 1), t, (T)1);
        if (best >= INF) { c[t] = INF; continue; }
        c[t] = best;
        guess = first_index<T>(c, cm1 + (t - 1), t, (T)1, best);
        d[t] = (int32_t)(1 + guess);
      }
      cur.extend(t, INF);
    }
  }
}

template <class T>
void solve_msm(int64_t t_max, int64_t m_max, int alpha, int beta, int sigma, Cols<T>& C, Cols<int32_t>& D1,
               Cols<int32_t>& D2, Cols<uint8_t>& H) {
  // Section 3.3 with the reading C(0, m) = 0 for every m (also m <= 0) and C(t > 0, m <= 0) = inf.
  // Q1 = y + C(y, m) + C(t - y, m - 1), 1 <= y < t;  Q2 = y + C(y - 1, m) + C(t - y, m - a(y)),
  // 1 <= y <= t, a(y) = alpha, or beta at y = 1 when the Section 3.4 variant is on.
  // sigma generalises the unit: where an internal state is no whole number of hidden states
  // (Section 3.3 calls alpha application-specific; Appendix C has slots of arbitrary sizes), m is
  // counted in a finer unit in which a hidden state takes sigma, an internal state alpha and one
  // without its input state beta: Q1 then recurses on m - sigma, and a budget below sigma cannot
  // even hold the start state of a sequence.
  const T INF = Inf<T>::v;
  std::vector<T> nonpos((size_t)t_max + 1, INF);  // the column of any budget <= 0
  nonpos[0] = 0;
  for (int64_t m = 0; m <= m_max; ++m) {
    C.col(m)[0] = 0;
    std::fill(D1.col(m), D1.col(m) + t_max + 1, 0);
    std::fill(D2.col(m), D2.col(m) + t_max + 1, 0);
    std::fill(H.col(m), H.col(m) + t_max + 1, (uint8_t)0);
  }
  auto column = [&](int64_t m) -> const T* { return m < sigma ? nonpos.data() : C.col(m); };
  // The columns of this mode are not convex in t, so every cell is a scan; what is left to gain is
  // that cell (t, m) needs the columns m - 1, m - alpha, m - beta only up to row t - 1.  Several
  // threads therefore fill consecutive columns at once, each a few rows behind the columns it
  // reads (rows[m]: how far column m has got).  The values are those of the plain loop.
  std::vector<std::atomic<int64_t>> rows((size_t)m_max + 1);
  for (auto& r : rows) r.store(0, std::memory_order_relaxed);
  auto wait_for = [&](int64_t m, int64_t upto) -> int64_t {   // until column m is filled up to row `upto`; how far it is
    if (m < sigma) return t_max;
    int64_t got;
    while ((got = rows[(size_t)m].load(std::memory_order_acquire)) < upto) std::this_thread::yield();
    return got;
  };
  std::atomic<int64_t> next_column{sigma};   // columns below sigma stay infinite (row 0 apart)
  auto worker = [&]() {
   for (;;) {
    const int64_t m = next_column.fetch_add(1, std::memory_order_relaxed);
    if (m > m_max) return;
    T* c = C.col(m);
    const T* cm1 = column(m - sigma);
    const T* cma = column(m - alpha);
    const T* cmb = beta > 0 ? column(m - beta) : nullptr;
    int64_t sure = 0;   // rows of the columns read that are known to be there
    for (int64_t t = 1; t <= t_max; ++t) {
      if (sure < t - 1) {
        sure = std::min(wait_for(m - sigma, t - 1), wait_for(m - alpha, t - 1));
        if (cmb) sure = std::min(sure, wait_for(m - beta, t - 1));
      }
      T c1 = INF, c2 = INF;
      int32_t y1 = 0, y2 = 0;
      if (t >= 2) {
        c1 = scan_min<T>(c + 1, cm1 + (t - 1), t - 1, (T)1);
        if (c1 < INF) y1 = (int32_t)(1 + first_index<T>(c + 1, cm1 + (t - 1), t - 1, (T)1, c1));
        else c1 = INF;
      }
      if (cmb) {
        // y = 1 charged beta, y >= 2 charged alpha; keep the smallest y on ties
        T q1 = (T)std::min<int64_t>((int64_t)1 + c[0] + cmb[t - 1], INF);
        T rest = INF;
        if (t >= 2) rest = scan_min<T>(c + 1, cma + (t - 2), t - 1, (T)2);
        if (rest >= INF) rest = INF;
        if (q1 <= rest) { c2 = q1; y2 = 1; }
        else { c2 = rest; y2 = (int32_t)(2 + first_index<T>(c + 1, cma + (t - 2), t - 1, (T)2, rest)); }
        if (c2 >= INF) { c2 = INF; y2 = 0; }
      } else {
        c2 = scan_min<T>(c, cma + (t - 1), t, (T)1);
        if (c2 < INF) y2 = (int32_t)(1 + first_index<T>(c, cma + (t - 1), t, (T)1, c2));
        else c2 = INF;
      }
      D1.col(m)[t] = y1;
      D2.col(m)[t] = y2;
      if (c1 >= INF && c2 >= INF) c[t] = INF;
      else if (c1 <= c2) { c[t] = c1; H.col(m)[t] = 1; }   // ties: the hidden state (fewer units)
      else               { c[t] = c2; H.col(m)[t] = 2; }
      if ((t & 7) == 0 || t == t_max) rows[(size_t)m].store(t, std::memory_order_release);
    }
   }
  };
  // few, short columns are not worth a thread
  unsigned n_threads = std::thread::hardware_concurrency();
  if (n_threads > 16) n_threads = 16;
  if (n_threads < 1 || plan_scan_only() || t_max * m_max < 200000) n_threads = 1;
  if ((int64_t)n_threads > m_max) n_threads = (unsigned)m_max;
  std::vector<std::thread> pool;
  try {
    for (unsigned i = 1; i < n_threads; ++i) pool.emplace_back(worker);
  } catch (const std::system_error&) {
    // fewer threads than hoped for: the ones that started, and this one, do all the columns
  }
  worker();
  for (std::thread& th : pool) th.join();
}

template <class S, class Dst>
void transpose_into(Cols<S>& src, std::vector<Dst>& dst) {
  dst.resize(src.v.size());
  for (int64_t m = 0; m < src.m_dim; ++m) {
    const S* c = src.col(m);
    for (int64_t t = 0; t < src.t_dim; ++t) dst[(size_t)t * src.m_dim + m] = (Dst)c[t];
  }
}

template <class S>
void transpose_costs(Cols<S>& src, std::vector<int64_t>& dst) {
  transpose_into(src, dst);
  for (int64_t& v : dst)
    if (v >= (int64_t)Inf<S>::v) v = Inf<int64_t>::v;
}

template <class T>
void solve(Plan& p) {
  const int64_t t = p.t, m = p.m;
  Cols<T> C(t, m, Inf<T>::v);
  Cols<int32_t> D(t, m, 0);
  if (p.mode == MEBPTT_HSM) {
    solve_hsm<T>(t, m, C, D);
  } else if (p.mode == MEBPTT_ISM) {
    solve_ism<T>(t, m, C, D);
  } else {
    Cols<int32_t> D2(t, m, 0);
    Cols<uint8_t> H(t, m, 0);
    solve_msm<T>(t, m, p.alpha, p.beta, p.sigma, C, D, D2, H);
    transpose_into(D2, p.D2);
    transpose_into(H, p.H);
  }
  transpose_costs(C, p.C);
  transpose_into(D, p.D);
}

// ---------------------------------------------------------------------------------------
// Unrolling the protocol
// ---------------------------------------------------------------------------------------
struct Emitter {
  Plan& p;
  int64_t units;      // paper's accounting
  int64_t top = 0;    // physical arena top, hidden-state units
  explicit Emitter(Plan& pl) : p(pl), units(pl.mode == MEBPTT_ISM ? 0 : pl.sigma) { p.peak_units = units; }

  int64_t Cat(int64_t t, int64_t m) const { return p.C[(size_t)t * (p.m + 1) + m]; }
  int32_t Dat(int64_t t, int64_t m) const { return p.D[(size_t)t * (p.m + 1) + m]; }
  int32_t D2at(int64_t t, int64_t m) const { return p.D2[(size_t)t * (p.m + 1) + m]; }
  int Hat(int64_t t, int64_t m) const { return p.H[(size_t)t * (p.m + 1) + m]; }

  void fwd(int64_t k, int32_t src, int32_t dst, int fmt) {
    mebptt_op op{};
    op.kind = MEBPTT_OP_FWD; op.k = (int32_t)k; op.src = src; op.dst = dst; op.dst_fmt = fmt;
    op.aux = 0; op.units = (int32_t)units;
    p.tape.push_back(op);
  }
  void bwd(int64_t k, int32_t src, int fmt, int32_t aux) {
    mebptt_op op{};
    op.kind = MEBPTT_OP_BWD; op.k = (int32_t)k; op.src = src; op.dst = 0; op.dst_fmt = fmt;
    op.aux = aux; op.units = (int32_t)units;
    p.tape.push_back(op);
  }
  // n forward operations from the state of step s at `loc`; the last one writes `fmt` to
  // `last_dst`, the others alternate between the two scratch states.  Returns nothing: the
  // caller knows where the last state went.
  void sweep(int64_t s, int64_t n, int32_t loc, int32_t last_dst, int last_fmt) {
    int32_t cur = loc;
    for (int64_t i = 1; i <= n; ++i) {
      if (i == n) { fwd(s + i, cur, last_dst, last_fmt); return; }
      int32_t dst = (cur == MEBPTT_LOC_PING) ? MEBPTT_LOC_PONG : MEBPTT_LOC_PING;
      fwd(s + i, cur, dst, MEBPTT_FMT_HIDDEN);
      cur = dst;
    }
  }
  void grow(int64_t paper_units, int64_t phys_units) {
    units += paper_units; top += phys_units;
    p.peak_units = std::max(p.peak_units, units);
    p.arena_units = std::max(p.arena_units, top);
  }
  void shrink(int64_t paper_units, int64_t phys_units) { units -= paper_units; top -= phys_units; }

  // Algorithm 2.  `loc` holds the hidden state of step s (Peek).
  void hsm(int64_t t, int64_t m, int64_t s, int32_t loc) {
    for (;;) {
      if (t == 0) return;
      if (t == 1) {  // base case: forward and backward on the working core
        fwd(s + 1, loc, MEBPTT_LOC_CORE, MEBPTT_FMT_INTERNAL);
        bwd(s + 1, MEBPTT_LOC_CORE, MEBPTT_FMT_INTERNAL, 0);
        return;
      }
      if (m == 1) {  // boundary C(t, 1): re-run from the start state before every backward step
        for (int64_t k = t; k >= 1; --k) {
          sweep(s, k, loc, MEBPTT_LOC_CORE, MEBPTT_FMT_INTERNAL);
          bwd(s + k, MEBPTT_LOC_CORE, MEBPTT_FMT_INTERNAL, 0);
        }
        return;
      }
      const int64_t y = Dat(t, m);
      const int32_t slot = (int32_t)top;
      grow(1, 1);
      // the sweep runs y operations (the printed bound t - 1 contradicts the cost y of
      // Eq. (1)); its last one writes h_{s+y} straight into the slot: that is the Push
      sweep(s, y, loc, slot, MEBPTT_FMT_HIDDEN);
      hsm(t - y, m - 1, s + y, slot);
      shrink(1, 1);  // Pop
      t = y;         // left part, full budget
    }
  }

  // Section 3.2, steps 1-4.
  void ism(int64_t t, int64_t m, int64_t s, int32_t loc) {
    const int a = p.alpha;
    while (t > 0) {
      const int64_t y = Dat(t, m);
      const int32_t slot = (int32_t)top;
      grow(1, a);
      sweep(s, y, loc, slot, MEBPTT_FMT_INTERNAL);          // step 1
      ism(t - y, m - 1, s + y, slot);                        // step 2
      bwd(s + y, slot, MEBPTT_FMT_INTERNAL, 0);              // step 3
      shrink(1, a);
      t = y - 1;                                             // step 4
    }
  }

  // Section 3.3 (and 3.4 when beta > 0).
  void msm(int64_t t, int64_t m, int64_t s, int32_t loc) {
    const int a = p.alpha, b = p.beta, sg = p.sigma;
    while (t > 0) {
      if (Hat(t, m) == 1) {
        const int64_t y = Dat(t, m);
        const int32_t slot = (int32_t)top;
        grow(sg, sg);
        sweep(s, y, loc, slot, MEBPTT_FMT_HIDDEN);
        msm(t - y, m - sg, s + y, slot);
        shrink(sg, sg);
        t = y;
      } else {
        const int64_t y = D2at(t, m);
        if (y == t) {
          // nothing to the right: the internal state never leaves the working core
          sweep(s, y, loc, MEBPTT_LOC_CORE, MEBPTT_FMT_INTERNAL);
          bwd(s + y, MEBPTT_LOC_CORE, MEBPTT_FMT_INTERNAL, 0);
        } else {
          const bool short_form = (b > 0 && y == 1);
          const int u = short_form ? b : a;
          const int fmt = short_form ? MEBPTT_FMT_INTERNAL_NOINPUT : MEBPTT_FMT_INTERNAL;
          const int32_t slot = (int32_t)top;
          grow(u, u);
          sweep(s, y, loc, slot, fmt);
          msm(t - y, m - u, s + y, slot);
          bwd(s + y, slot, fmt, short_form ? loc : 0);
          shrink(u, u);
        }
        t = y - 1;
      }
    }
  }
};

}  // namespace

// Chen's sqrt(t) schedule (Section 2.2) as a tape for the same executor: cut the sequence into
// segments of s = ceil(sqrt(t)) steps; one forward pass memorises the hidden state at every
// segment boundary; then, from the last segment to the first, run forward through the segment
// memorising every internal state (the last segment does this on its first visit) and
// backpropagate through them.  Section 4.1 notes that this is one (suboptimal) policy of the
// mixed scheme; Section 4.2 counts its memory with the input hidden states left out (beta units
// per internal state), which is what beta > 0 selects here.
int build_chen_plan(int64_t t, int alpha, int beta, Plan** out) {
  if (!out) return MEBPTT_ERR_ARG;
  *out = nullptr;
  if (t < 1 || t > (int64_t)1 << 24) return MEBPTT_ERR_ARG;
  if (alpha < 2 || alpha > 64 || beta < 0 || beta > alpha) return MEBPTT_ERR_ARG;
  Plan* p = new_plan();
  if (!p) return MEBPTT_ERR_OOM;
  p->t = t; p->mode = MEBPTT_CHEN_SQRT; p->alpha = alpha; p->beta = beta;
  try {
    int64_t s = 1;
    while (s * s < t) ++s;
    const int64_t nseg = (t + s - 1) / s;
    const int u = beta > 0 ? beta : alpha;
    const int fmt = beta > 0 ? MEBPTT_FMT_INTERNAL_NOINPUT : MEBPTT_FMT_INTERNAL;
    p->m = (int64_t)1 << 40;  // no budget while emitting; set to the peak below
    Emitter e(*p);
    int32_t loc = MEBPTT_LOC_INIT;
    for (int64_t j = 0; j + 1 < nseg; ++j) {
      const int32_t slot = (int32_t)e.top;
      e.grow(1, 1);
      e.sweep(j * s, s, loc, slot, MEBPTT_FMT_HIDDEN);
      loc = slot;
    }
    std::vector<int32_t> slots, prevs;
    for (int64_t j = nseg - 1; j >= 0; --j) {
      const int64_t start = j * s, len = std::min<int64_t>(s, t - start);
      int32_t prev = (j == 0) ? (int32_t)MEBPTT_LOC_INIT : (int32_t)(j - 1);
      slots.clear(); prevs.clear();
      for (int64_t i = 1; i <= len; ++i) {
        const int32_t slot = (int32_t)e.top;
        e.grow(u, u);
        e.fwd(start + i, prev, slot, fmt);
        slots.push_back(slot); prevs.push_back(prev);
        prev = slot;
      }
      for (int64_t i = len; i >= 1; --i) {
        e.bwd(start + i, slots[(size_t)i - 1], fmt, beta > 0 ? prevs[(size_t)i - 1] : 0);
        e.shrink(u, u);
      }
      if (j > 0) e.shrink(1, 1);
    }
    p->cost = 0;
    for (const mebptt_op& op : p->tape) p->cost += (op.kind == MEBPTT_OP_FWD);
    p->m = p->peak_units;
  } catch (const std::bad_alloc&) {
    delete p;
    return MEBPTT_ERR_OOM;
  }
  int rc = validate_plan(*p);
  if (rc != MEBPTT_OK) { delete p; return rc; }
  *out = p;
  return MEBPTT_OK;
}

// Chen's recursive schedule (Section 2.2) as a tape: a sequence of more than k steps is cut into
// k + 1 parts as equal as they come, one forward pass memorises the hidden state at the k cuts,
// and the parts are then treated the same way from the last to the first; a sequence of at most
// k steps is run forward with every internal state kept and backpropagated.  (Section 2.2
// summarises the scheme as a split into k parts that stops when a part is shorter than k;
// k memorised states per level, hence k + 1 parts, is the reading under which its figures --
// memory O(k log_{k+1} t), at least log_2 t for k = 1 -- come out.)
int build_chen_recursive_plan(int64_t t, int k, int alpha, int beta, Plan** out) {
  if (!out) return MEBPTT_ERR_ARG;
  *out = nullptr;
  if (t < 1 || t > (int64_t)1 << 24 || k < 1 || k > 4096) return MEBPTT_ERR_ARG;
  if (alpha < 2 || alpha > 64 || beta < 0 || beta > alpha) return MEBPTT_ERR_ARG;
  Plan* p = new_plan();
  if (!p) return MEBPTT_ERR_OOM;
  p->t = t; p->mode = MEBPTT_CHEN_RECURSIVE; p->alpha = alpha; p->beta = beta;
  try {
    const int u = beta > 0 ? beta : alpha;
    const int fmt = beta > 0 ? MEBPTT_FMT_INTERNAL_NOINPUT : MEBPTT_FMT_INTERNAL;
    p->m = (int64_t)1 << 40;  // no budget while emitting; set to the peak below
    Emitter e(*p);
    struct Frame { int64_t start, len; int32_t loc; int stage; std::vector<int64_t> cut; std::vector<int32_t> locs; int j; };
    std::vector<Frame> stack;
    stack.push_back(Frame{0, t, MEBPTT_LOC_INIT, 0, {}, {}, 0});
    std::vector<int32_t> slots, prevs;
    while (!stack.empty()) {
      Frame& f = stack.back();
      if (f.len <= k) {
        // every internal state of the segment, then back through them
        int32_t prev = f.loc;
        slots.clear(); prevs.clear();
        for (int64_t i = 1; i <= f.len; ++i) {
          const int32_t slot = (int32_t)e.top;
          e.grow(u, u);
          e.fwd(f.start + i, prev, slot, fmt);
          slots.push_back(slot); prevs.push_back(prev);
          prev = slot;
        }
        for (int64_t i = f.len; i >= 1; --i) {
          e.bwd(f.start + i, slots[(size_t)i - 1], fmt, beta > 0 ? prevs[(size_t)i - 1] : 0);
          e.shrink(u, u);
        }
        stack.pop_back();
        continue;
      }
      if (f.stage == 0) {
        // cuts[0] = start, cuts[k + 1] = end; the first len mod (k + 1) parts are one step longer
        const int64_t parts = k + 1, base = f.len / parts, rem = f.len % parts;
        f.cut.assign(1, f.start);
        for (int64_t i = 0; i < parts; ++i) f.cut.push_back(f.cut.back() + base + (i < rem ? 1 : 0));
        f.locs.assign(1, f.loc);
        int32_t cur = f.loc;
        for (int64_t i = 1; i <= k; ++i) {
          const int32_t slot = (int32_t)e.top;
          e.grow(1, 1);
          e.sweep(f.cut[(size_t)i - 1], f.cut[(size_t)i] - f.cut[(size_t)i - 1], cur, slot, MEBPTT_FMT_HIDDEN);
          f.locs.push_back(slot);
          cur = slot;
        }
        f.stage = 1;
        f.j = k;
      } else {
        // part j + 1 has just been backpropagated: the state at its start is no longer needed
        e.shrink(1, 1);
        --f.j;
      }
      if (f.j < 0) { stack.pop_back(); continue; }
      if (f.j == 0) {
        // the first part starts at the state the caller holds: nothing of ours to release after it
        const Frame child{f.cut[0], f.cut[1] - f.cut[0], f.locs[0], 0, {}, {}, 0};
        stack.pop_back();
        stack.push_back(child);
        continue;
      }
      const Frame child{f.cut[(size_t)f.j], f.cut[(size_t)f.j + 1] - f.cut[(size_t)f.j], f.locs[(size_t)f.j], 0, {}, {}, 0};
      stack.push_back(child);
    }
    p->cost = 0;
    for (const mebptt_op& op : p->tape) p->cost += (op.kind == MEBPTT_OP_FWD);
    p->m = p->peak_units;
  } catch (const std::bad_alloc&) {
    delete p;
    return MEBPTT_ERR_OOM;
  }
  int rc = validate_plan(*p);
  if (rc != MEBPTT_OK) { delete p; return rc; }
  *out = p;
  return MEBPTT_OK;
}

int build_plan(int64_t t, int64_t m, int mode, int alpha, int beta, Plan** out, int sigma) {
  if (!out) return MEBPTT_ERR_ARG;
  *out = nullptr;
  if (t < 1 || t > (int64_t)1 << 24) return MEBPTT_ERR_ARG;
  if (mode != MEBPTT_HSM && mode != MEBPTT_ISM && mode != MEBPTT_MSM) return MEBPTT_ERR_ARG;
  if (sigma < 1 || sigma > 64 || (sigma > 1 && mode != MEBPTT_MSM)) return MEBPTT_ERR_ARG;
  if (alpha < 2 || alpha < sigma || alpha > 64 * sigma) return MEBPTT_ERR_ARG;
  if (beta < 0 || beta > alpha || (beta > 0 && beta < sigma)) return MEBPTT_ERR_ARG;
  if (m < 1) return MEBPTT_ERR_BUDGET;
  if (mode != MEBPTT_MSM) beta = 0;
  // beyond saturation more memory changes nothing
  const int64_t sat = (mode == MEBPTT_MSM) ? std::max<int64_t>(1, (int64_t)alpha * (t - 1) + sigma) : t;
  m = std::min(m, sat);
  Plan* p = new_plan();
  if (!p) return MEBPTT_ERR_OOM;
  p->t = t; p->m = m; p->mode = mode; p->alpha = alpha; p->beta = beta; p->sigma = sigma;
  try {
    if (t * (t + 1) / 2 + t < (int64_t)Inf<int32_t>::v) solve<int32_t>(*p);
    else solve<int64_t>(*p);
    p->cost = p->C[(size_t)t * (m + 1) + m];
    if (p->cost >= MEBPTT_INF) { delete p; return MEBPTT_ERR_BUDGET; }
    if (p->cost + t > (int64_t)1 << 28) { delete p; return MEBPTT_ERR_UNSUPPORTED; }  // tape too long
    p->tape.reserve((size_t)(p->cost + t));
    Emitter e(*p);
    if (mode == MEBPTT_HSM) e.hsm(t, m, 0, MEBPTT_LOC_INIT);
    else if (mode == MEBPTT_ISM) e.ism(t, m, 0, MEBPTT_LOC_INIT);
    else e.msm(t, m, 0, MEBPTT_LOC_INIT);
  } catch (const std::bad_alloc&) {
    delete p;
    return MEBPTT_ERR_OOM;
  }
  int rc = validate_plan(*p);
  if (rc != MEBPTT_OK) { delete p; return rc; }
  *out = p;
  return MEBPTT_OK;
}

// ---------------------------------------------------------------------------------------
// Host replay of a tape with integer bookkeeping
// ---------------------------------------------------------------------------------------
int validate_plan(const Plan& p) {
  struct Entry { int64_t off, units, pos; int fmt; };
  std::vector<Entry> arena;            // live records, ascending offsets (a stack)
  int64_t ping = -1, pong = -1;        // step whose hidden state sits there
  int64_t core = -1;                   // step whose internal state the working core holds
  int64_t next_bwd = p.t, forwards = 0, peak = 0;
  const int a = p.alpha, b = p.beta;
  auto rec_units = [&](int fmt) -> int64_t {
    if (fmt == MEBPTT_FMT_HIDDEN) return p.sigma;
    if (fmt == MEBPTT_FMT_INTERNAL) return a;
    return b;
  };
  auto hidden_at = [&](int32_t loc) -> int64_t {  // which step's hidden state is readable at loc
    if (loc == MEBPTT_LOC_INIT) return 0;
    if (loc == MEBPTT_LOC_PING) return ping;
    if (loc == MEBPTT_LOC_PONG) return pong;
    if (loc == MEBPTT_LOC_CORE) return core;
    for (const Entry& e : arena) if (e.off == loc) return e.pos;
    return -1;
  };
  for (const mebptt_op& op : p.tape) {
    if (op.k < 1 || op.k > p.t) return MEBPTT_ERR_PLAN;
    if (op.units < 0 || op.units > p.m) return MEBPTT_ERR_PLAN;
    peak = std::max<int64_t>(peak, op.units);
    if (op.kind == MEBPTT_OP_FWD) {
      if (hidden_at(op.src) != op.k - 1) return MEBPTT_ERR_PLAN;
      if (op.dst == op.src) return MEBPTT_ERR_PLAN;
      ++forwards;
      if (op.dst == MEBPTT_LOC_PING) { if (op.dst_fmt != MEBPTT_FMT_HIDDEN) return MEBPTT_ERR_PLAN; ping = op.k; }
      else if (op.dst == MEBPTT_LOC_PONG) { if (op.dst_fmt != MEBPTT_FMT_HIDDEN) return MEBPTT_ERR_PLAN; pong = op.k; }
      else if (op.dst == MEBPTT_LOC_CORE) { if (op.dst_fmt != MEBPTT_FMT_INTERNAL) return MEBPTT_ERR_PLAN; core = op.k; }
      else if (op.dst >= 0) {
        if (op.dst_fmt == MEBPTT_FMT_INTERNAL_NOINPUT && b <= 0) return MEBPTT_ERR_PLAN;
        const int64_t u = rec_units(op.dst_fmt);
        // writing at an offset retires everything at or above it (stack discipline) ...
        while (!arena.empty() && arena.back().off >= op.dst) arena.pop_back();
        // ... and must not run into what lies below
        if (!arena.empty() && arena.back().off + arena.back().units > op.dst) return MEBPTT_ERR_PLAN;
        if (op.dst + u > p.arena_units) return MEBPTT_ERR_PLAN;
        arena.push_back(Entry{op.dst, u, op.k, op.dst_fmt});
      } else return MEBPTT_ERR_PLAN;
    } else if (op.kind == MEBPTT_OP_BWD) {
      if (op.k != next_bwd) return MEBPTT_ERR_PLAN;
      if (op.src == MEBPTT_LOC_CORE) {
        if (core != op.k || op.dst_fmt != MEBPTT_FMT_INTERNAL) return MEBPTT_ERR_PLAN;
        core = -1;
      } else {
        bool ok = false;
        for (const Entry& e : arena)
          if (e.off == op.src && e.pos == op.k && e.fmt == op.dst_fmt && e.fmt != MEBPTT_FMT_HIDDEN) ok = true;
        if (!ok) return MEBPTT_ERR_PLAN;
        if (op.dst_fmt == MEBPTT_FMT_INTERNAL_NOINPUT && hidden_at(op.aux) != op.k - 1) return MEBPTT_ERR_PLAN;
      }
      --next_bwd;
    } else return MEBPTT_ERR_PLAN;
  }
  if (next_bwd != 0) return MEBPTT_ERR_PLAN;
  if (forwards != p.cost) return MEBPTT_ERR_PLAN;
  if (peak != p.peak_units || peak > p.m) return MEBPTT_ERR_PLAN;
  return MEBPTT_OK;
}

}  // namespace mebptt

// ---------------------------------------------------------------------------------------
// C interface: planning
// ---------------------------------------------------------------------------------------
using mebptt::Plan;

extern "C" {

int mebptt_plan(int64_t t, int64_t m, int mode, mebptt_plan_t** out) {
  return mebptt::build_plan(t, m, mode, 4, 0, reinterpret_cast<Plan**>(out));
}

int mebptt_plan_chen_recursive(int64_t t, int k, int alpha, int beta, mebptt_plan_t** out) {
  return mebptt::build_chen_recursive_plan(t, k, alpha, beta, reinterpret_cast<Plan**>(out));
}
int mebptt_plan_chen_sqrt(int64_t t, int alpha, int beta, mebptt_plan_t** out) {
  return mebptt::build_chen_plan(t, alpha, beta, reinterpret_cast<Plan**>(out));
}

int mebptt_plan_ex(int64_t t, int64_t m, int mode, int alpha, int beta, mebptt_plan_t** out) {
  return mebptt::build_plan(t, m, mode, alpha, beta, reinterpret_cast<Plan**>(out));
}

void mebptt_plan_free(mebptt_plan_t* plan) {
  if (!plan) return;
  mebptt::tc::forget_plan(reinterpret_cast<Plan*>(plan)->id);   // what the executor prepared for this plan goes with it
  delete reinterpret_cast<Plan*>(plan);
}

#define P_(x) (reinterpret_cast<const Plan*>(x))
int64_t mebptt_plan_cost(const mebptt_plan_t* plan) { return plan ? P_(plan)->cost : -1; }
int64_t mebptt_plan_num_ops(const mebptt_plan_t* plan) { return plan ? (int64_t)P_(plan)->tape.size() : -1; }
const mebptt_op* mebptt_plan_tape(const mebptt_plan_t* plan) { return plan ? P_(plan)->tape.data() : nullptr; }
int64_t mebptt_plan_peak_units(const mebptt_plan_t* plan) { return plan ? P_(plan)->peak_units : -1; }
int64_t mebptt_plan_arena_units(const mebptt_plan_t* plan) { return plan ? P_(plan)->arena_units : -1; }
int64_t mebptt_plan_t_len(const mebptt_plan_t* plan) { return plan ? P_(plan)->t : -1; }
int64_t mebptt_plan_m(const mebptt_plan_t* plan) { return plan ? P_(plan)->m : -1; }
int mebptt_plan_mode(const mebptt_plan_t* plan) { return plan ? P_(plan)->mode : -1; }
int mebptt_plan_sized(int64_t t, int64_t m, int sigma, int alpha, int beta, mebptt_plan_t** out) {
  return mebptt::build_plan(t, m, MEBPTT_MSM, alpha, beta, reinterpret_cast<Plan**>(out), sigma);
}
int mebptt_plan_sigma(const mebptt_plan_t* plan) { return plan ? P_(plan)->sigma : -1; }
int mebptt_plan_alpha(const mebptt_plan_t* plan) { return plan ? P_(plan)->alpha : -1; }
int mebptt_plan_beta(const mebptt_plan_t* plan) { return plan ? P_(plan)->beta : -1; }

int mebptt_plan_tables(const mebptt_plan_t* plan, const int64_t** C, const int32_t** D,
                       const int32_t** D2, const uint8_t** H, int64_t* t_dim, int64_t* m_dim) {
  if (!plan) return MEBPTT_ERR_ARG;
  const Plan* p = P_(plan);
  if (C) *C = p->C.empty() ? nullptr : p->C.data();
  if (D) *D = p->D.empty() ? nullptr : p->D.data();
  if (D2) *D2 = p->D2.empty() ? nullptr : p->D2.data();
  if (H) *H = p->H.empty() ? nullptr : p->H.data();
  if (t_dim) *t_dim = p->t + 1;
  if (m_dim) *m_dim = p->m + 1;
  return MEBPTT_OK;
}

int mebptt_plan_validate(const mebptt_plan_t* plan) {
  if (!plan) return MEBPTT_ERR_ARG;
  return mebptt::validate_plan(*P_(plan));
}

const char* mebptt_strerror(int status) {
  switch (status) {
    case MEBPTT_OK: return "ok";
    case MEBPTT_ERR_ARG: return "invalid argument";
    case MEBPTT_ERR_BUDGET: return "memory budget too small: no policy exists";
    case MEBPTT_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case MEBPTT_ERR_UNSUPPORTED: return "unsupported shape, precision or plan";
    case MEBPTT_ERR_CUDA: return "CUDA runtime error";
    case MEBPTT_ERR_TIMEOUT: return "bounded device-side wait expired";
    case MEBPTT_ERR_OOM: return "out of host memory";
    case MEBPTT_ERR_PLAN: return "tape failed validation";
    default: return "unknown status";
  }
}

}  // extern "C"
