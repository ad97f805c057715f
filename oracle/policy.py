"""Oracle: the checkpoint-policy dynamic programs and an integer simulation of the protocol.

Test infrastructure only (see the package docstring).  Integer arithmetic throughout.

Notation follows the paper: ``t`` sequence length, ``m`` memory budget, ``y`` position of the
first memorisation, ``C(t, m)`` optimal number of forward operations, ``D(t, m)`` the optimal
``y``; for the mixed scheme ``alpha`` (``beta``) is the size of an internal state measured in
hidden states (when its input hidden state is already stored), ``H(t, m)`` tells which kind of
state is pushed first and ``D1``/``D2`` where.

Readings taken where the text leaves a choice (each is repeated beside the code it affects):

* ``C(0, m) = 0`` holds for every ``m``, also ``m <= 0`` (Section 3.3 lists it next to
  ``C(., m <= 0) = inf``; the zero wins, an empty sequence costs nothing).
* ``argmin`` ties go to the smallest ``y`` (Algorithm 1 scans upward with a strict ``<``) and
  ties between the two kinds of push go to the hidden state (fewer units for the same cost).
* Units: in HSM and MSM the start state of a (sub)sequence occupies one of its ``m`` units and
  the single working core lives outside the budget (Section 3.1: ``C(t, m) = 2t - 1`` needs
  ``m >= t``).  In ISM the budget counts internal states and the state being worked on is one of
  them (Section 3.2: ``C(t, m) = t`` needs ``m >= t``); the initial hidden state is free.
"""
from __future__ import annotations

import numpy as np

INF = np.int64(1) << np.int64(60)  # "infinity": three of them still fit in int64

HSM, ISM, MSM = 0, 1, 2


def _sat(a):
    """Clamp sums that involved INF back to INF."""
    return np.minimum(a, INF)


# --------------------------------------------------------------------------------------
# Section 3.1, Eqs. (1)-(3): hidden-state memorisation
# --------------------------------------------------------------------------------------
def hsm_tables(t_max: int, m_max: int):
    """C(t, m), D(t, m) for BPTT-HSM, 0 <= t <= t_max, 0 <= m <= m_max.

    Boundaries (Section 3.1): C(1, m) = 1 and C(t, 1) = t (t + 1) / 2.  Elsewhere
    C(t, m) = min over 1 <= y < t of Q(t, m, y) = y + C(t - y, m - 1) + C(y, m).
    C(t, m) = 2 t - 1 for m >= t is *not* imposed; it has to come out of the recursion.
    Row t = 0 and column m = 0 are INF (not used by HSM) and D is 0 where no push happens.
    """
    C = np.full((t_max + 1, m_max + 1), INF, dtype=np.int64)
    D = np.zeros((t_max + 1, m_max + 1), dtype=np.int64)
    for m in range(1, m_max + 1):
        if t_max >= 1:
            C[1, m] = 1
    if m_max >= 1:
        for t in range(1, t_max + 1):
            C[t, 1] = t * (t + 1) // 2
    for m in range(2, m_max + 1):
        for t in range(2, t_max + 1):
            y = np.arange(1, t, dtype=np.int64)
            Q = _sat(y + C[t - y, m - 1] + C[y, m])
            k = int(np.argmin(Q))  # first minimum = smallest y
            C[t, m] = Q[k]
            D[t, m] = y[k]
    return C, D


# --------------------------------------------------------------------------------------
# Section 3.2, Eqs. (4)-(5): internal-state memorisation
# --------------------------------------------------------------------------------------
def ism_tables(t_max: int, m_max: int):
    """C(t, m), D(t, m) for BPTT-ISM.

    C(0, m) = 0; C(t, 0) = INF for t > 0; otherwise the minimum over 1 <= y <= t of
    Q(t, m, y) = y + C(y - 1, m) + C(t - y, m - 1).
    """
    C = np.full((t_max + 1, m_max + 1), INF, dtype=np.int64)
    D = np.zeros((t_max + 1, m_max + 1), dtype=np.int64)
    C[0, :] = 0
    for m in range(1, m_max + 1):
        for t in range(1, t_max + 1):
            y = np.arange(1, t + 1, dtype=np.int64)
            Q = _sat(y + C[y - 1, m] + C[t - y, m - 1])
            k = int(np.argmin(Q))
            C[t, m] = Q[k]
            D[t, m] = y[k]
    return C, D


# --------------------------------------------------------------------------------------
# Sections 3.3 and 3.4, Eqs. (6)-(10): mixed memorisation
# --------------------------------------------------------------------------------------
def msm_tables(t_max: int, m_max: int, alpha: int, beta: int | None = None, sigma: int = 1):
    """C, H, D1, D2 for BPTT-MSM; ``beta`` switches on the variant of Section 3.4.

    Q1(t, m, y) = y + C(y, m) + C(t - y, m - sigma),           1 <= y <  t
    Q2(t, m, y) = y + C(y - 1, m) + C(t - y, m - a(y)),        1 <= y <= t
    with a(y) = alpha, or (Section 3.4) beta when y = 1 and alpha when y > 1.
    C(0, .) = 0 everywhere, C(t > 0, m < sigma) = INF.  H = 1 (hidden) wins ties.

    ``sigma`` is the size of a hidden state in the unit m is counted in.  Section 3.3 measures
    memory "in the units of hidden states", i.e. sigma = 1, and an internal state then has to be
    a whole number alpha of them.  Where it is not -- Section 3.3 calls alpha application-specific,
    and Appendix C has slots of arbitrary sizes s_i -- the same recursion is written over a finer
    unit (the greatest common divisor of the sizes): a hidden state takes sigma units, an internal
    state alpha, one without its input hidden state beta, and the start state of a subsequence,
    which Section 3.1 counts as one of the m hidden states, sigma of the m units.
    """
    if sigma < 1:
        raise ValueError("sigma must be a positive integer")
    if alpha < 2 and sigma == 1:
        raise ValueError("alpha must be an integer >= 2 (Section 3.3)")
    if alpha < sigma:
        raise ValueError("an internal state contains a hidden state: alpha >= sigma")
    if beta is not None and not (1 <= beta <= alpha):
        raise ValueError("need 1 <= beta <= alpha (Section 3.4)")
    C = np.full((t_max + 1, m_max + 1), INF, dtype=np.int64)
    H = np.zeros((t_max + 1, m_max + 1), dtype=np.int64)
    D1 = np.zeros((t_max + 1, m_max + 1), dtype=np.int64)
    D2 = np.zeros((t_max + 1, m_max + 1), dtype=np.int64)
    C[0, :] = 0

    def Cget(tt, mm):
        """C with the conventions for budgets that cannot hold a start state (vectorised over tt)."""
        tt = np.asarray(tt, dtype=np.int64)
        if mm < sigma:
            return np.where(tt == 0, np.int64(0), INF)
        return C[tt, mm]

    for m in range(sigma, m_max + 1):
        for t in range(1, t_max + 1):
            c1 = INF
            if t >= 2:
                y = np.arange(1, t, dtype=np.int64)
                Q1 = _sat(y + C[y, m] + Cget(t - y, m - sigma))
                k1 = int(np.argmin(Q1))
                c1 = Q1[k1]
                D1[t, m] = y[k1]
            y = np.arange(1, t + 1, dtype=np.int64)
            right = Cget(t - y, m - alpha).copy()
            if beta is not None:
                right[0] = Cget(np.int64(t - 1), m - beta)  # y = 1 is charged beta
            Q2 = _sat(y + C[y - 1, m] + right)
            k2 = int(np.argmin(Q2))
            c2 = Q2[k2]
            D2[t, m] = y[k2]
            if c1 <= c2:
                C[t, m], H[t, m] = c1, 1
            else:
                C[t, m], H[t, m] = c2, 2
    return C, H, D1, D2


# --------------------------------------------------------------------------------------
# Section 2.2 / 4.2: Chen's sqrt(t) algorithm, for comparison
# --------------------------------------------------------------------------------------
def chen_sqrt(t: int, alpha: int, beta: int | None = None):
    """Forward operations and memory units of Chen's sqrt(t) schedule.

    The sequence is cut into segments of s = ceil(sqrt(t)) steps.  A first pass runs through all
    segments but the last and keeps the hidden state at each boundary; then every segment, from
    the last to the first, is run forward keeping all its internal states and backpropagated.
    So every step is computed once, and every step outside the last segment a second time.
    Memory (in hidden-state units, the start state included as in the mixed scheme): one unit per
    kept boundary plus, at the worst moment, the internal states of one full segment (beta units
    each when their input hidden states are left out as in Section 4.2, else alpha).
    """
    s = 1
    while s * s < t:
        s += 1
    nseg = -(-t // s)
    last = t - (nseg - 1) * s
    forwards = t + (t - last)
    per = beta if beta is not None else alpha
    # while segment j is processed, the boundaries at its start and below are still kept
    # (j of them, all nseg - 1 for the last segment) next to its internal states
    peak = 1 + max(min(j, nseg - 1) + min(s, t - j * s) * per for j in range(nseg))
    return {"forwards": forwards, "units": peak, "segment": s}


def chen_recursive(t: int, k: int, alpha: int, beta: int | None = None):
    """Forward operations and memory units of Chen's recursive schedule (Section 2.2).

    A sequence of more than k steps is cut into k + 1 parts as equal as they come (the first ones
    one step longer); one pass runs through all parts but the last and keeps the hidden state at
    each of the k cuts; the parts are then treated the same way, last to first, each cut being
    dropped once the part that starts there is done.  A sequence of at most k steps is run forward
    keeping every internal state (beta units each when their input hidden states are left out,
    else alpha) and backpropagated.  Units count the start state, as in the mixed scheme.
    Reading: Section 2.2 summarises the scheme as a split into k parts; k memorised states per level (k + 1
    parts) is what its figures need -- memory O(k log_{k+1} t) and a minimum of log2 t at k = 1.
    """
    per = beta if beta is not None else alpha
    memo = {}

    def rec(n):
        if n in memo:
            return memo[n]
        if n <= k:
            memo[n] = (n, n * per)
            return memo[n]
        base, rem = divmod(n, k + 1)
        sizes = [base + (1 if i < rem else 0) for i in range(k + 1)]
        forwards = sum(sizes[:k])
        peak = k
        for j in range(k, -1, -1):          # while part j is treated, the cuts 1 .. j are still kept
            f, pk = rec(sizes[j])
            forwards += f
            peak = max(peak, j + pk)
        memo[n] = (forwards, peak)
        return memo[n]

    import sys
    sys.setrecursionlimit(max(sys.getrecursionlimit(), 10000))
    f, pk = rec(t)
    return {"forwards": f, "units": 1 + pk}


def saturation_budget(mode: int, t: int, alpha: int = 4) -> int:
    """Smallest budget beyond which more memory cannot lower the cost (used to cap tables)."""
    if mode == MSM:
        return max(1, alpha * (t - 1) + 1)
    return max(1, t)


def plan_tables(mode: int, t: int, m: int, alpha: int = 4, beta: int | None = None, sigma: int = 1):
    """Tables for one (mode, t, m) problem, in a dict (sigma: size of a hidden state, MSM only)."""
    if mode == HSM:
        C, D = hsm_tables(t, m)
        return {"mode": HSM, "C": C, "D": D}
    if mode == ISM:
        C, D = ism_tables(t, m)
        return {"mode": ISM, "C": C, "D": D}
    if mode == MSM:
        C, H, D1, D2 = msm_tables(t, m, alpha, beta, sigma)
        return {"mode": MSM, "C": C, "H": H, "D1": D1, "D2": D2, "alpha": alpha, "beta": beta, "sigma": sigma}
    raise ValueError("unknown mode")


def cost(mode: int, t: int, m: int, alpha: int = 4, beta: int | None = None, sigma: int = 1) -> int:
    """C(t, m): the predicted number of forward operations."""
    return int(plan_tables(mode, t, m, alpha, beta, sigma)["C"][t, m])


# --------------------------------------------------------------------------------------
# Algorithm 2 (HSM) and its ISM / MSM counterparts, with integer bookkeeping only
# --------------------------------------------------------------------------------------
class ProtocolError(AssertionError):
    pass


class _Machine:
    """Abstract machine of the paper's cost model.

    It holds a stack of memorised states, one working core, and the position of the hidden
    state the core last produced.  Each ``forward`` checks that the input hidden state it needs
    is really there; each ``backward`` checks that the internal state is.  No numbers flow.
    """

    def __init__(self, t: int, budget_units: int, start_units: int):
        self.t = t
        self.budget = budget_units
        self.units = start_units      # units in use (the start state in HSM / MSM)
        self.peak = start_units
        self.stack = []               # entries (kind, position, units)
        self.cur = 0                  # hidden state present in the working core: position
        self.core = None              # position whose internal state sits in the core
        self.forwards = 0
        self.ops = []                 # ('F', k, save) and ('B', k, src)
        self.next_backward = t

    def available_hidden(self):
        pos = {0, self.cur}
        for kind, p, _ in self.stack:
            pos.add(p)  # an internal state contains its output hidden state (Definition 3)
        return pos

    def forward(self, k: int, save: str | None):
        """One forward operation producing state k from state k - 1."""
        if (k - 1) not in self.available_hidden():
            raise ProtocolError(f"forward to {k}: hidden state {k - 1} is not in memory")
        self.forwards += 1
        self.cur = k
        self.core = k if save == "core" else None
        self.ops.append(("F", k, save))

    def push(self, kind: str, pos: int, units: int):
        self.units += units
        self.peak = max(self.peak, self.units)
        if self.units > self.budget:
            raise ProtocolError(f"budget exceeded: {self.units} > {self.budget}")
        self.stack.append((kind, pos, units))

    def pop(self):
        kind, pos, units = self.stack.pop()
        self.units -= units
        return kind, pos

    def restore(self, pos: int):
        """Peek: make the stored hidden state at ``pos`` the working hidden state (free)."""
        if pos not in self.available_hidden():
            raise ProtocolError(f"peek of {pos}: not stored")
        self.cur = pos

    def backward(self, k: int):
        if k != self.next_backward:
            raise ProtocolError(f"backward {k} out of order, expected {self.next_backward}")
        if self.core == k:
            src = "core"
        elif self.stack and self.stack[-1][:2] == ("internal", k):
            src = "stack"
        else:
            raise ProtocolError(f"backward {k}: internal state not available")
        self.core = None
        self.next_backward = k - 1
        self.ops.append(("B", k, src))


def simulate(mode: int, t: int, m: int, tables=None, alpha: int = 4, beta: int | None = None, sigma: int = 1):
    """Run the execution protocol for (mode, t, m) and return its integer statistics.

    Returns a dict with ``forwards`` (executed forward operations), ``backwards``,
    ``peak_units`` and ``ops``.  Raises ProtocolError if a state is used that is not stored,
    if the budget is exceeded, or if backward steps do not come in the order t, t-1, ..., 1.
    """
    if tables is None:
        tables = plan_tables(mode, t, m, alpha, beta, sigma)
    sg = tables.get("sigma", 1) if mode == MSM else 1
    if mode == ISM:
        mach = _Machine(t, m, 0)
    else:
        mach = _Machine(t, m, sg)  # the initial hidden state takes the units of one hidden state

    def sweep(s: int, n: int, last_save: str | None):
        """n consecutive forward operations from the stored state at s."""
        mach.restore(s)
        for i in range(1, n + 1):
            mach.forward(s + i, last_save if i == n else None)

    def exec_hsm(t_, m_, s):
        D = tables["D"]
        while True:
            if t_ == 0:
                return
            if t_ == 1:
                # Algorithm 2, base case: forward and backward on the working core
                sweep(s, 1, "core")
                mach.backward(s + 1)
                return
            if m_ == 1:
                # boundary C(t, 1): nothing but the start state is kept, every backward
                # step re-runs the sequence from it (Section 3, first example)
                for k in range(t_, 0, -1):
                    sweep(s, k, "core")
                    mach.backward(s + k)
                return
            y = int(D[t_, m_])
            # Algorithm 2 prints the sweep bound as t - 1; the text of Section 3.1 charges
            # y forward operations for this step and pushes the state at y, so y it is.
            sweep(s, y, None)
            mach.push("hidden", s + y, 1)
            exec_hsm(t_ - y, m_ - 1, s + y)
            mach.pop()
            t_ = y  # left part with the full budget (tail call)

    def exec_ism(t_, m_, s):
        D = tables["D"]
        while t_ > 0:
            y = int(D[t_, m_])
            # the sweep ends in one of the m internal-state slots (the state being worked on
            # counts against the budget in this scheme)
            sweep(s, y, "internal")
            mach.push("internal", s + y, 1)
            exec_ism(t_ - y, m_ - 1, s + y)     # Step 2
            mach.backward(s + y)                # Step 3: no forward operation needed
            mach.pop()
            t_ = y - 1                          # Step 4

    def exec_msm(t_, m_, s):
        Hh, D1, D2 = tables["H"], tables["D1"], tables["D2"]
        a, b = tables["alpha"], tables["beta"]
        while t_ > 0:
            if int(Hh[t_, m_]) == 1:
                y = int(D1[t_, m_])
                sweep(s, y, None)
                mach.push("hidden", s + y, sg)
                exec_msm(t_ - y, m_ - sg, s + y)
                mach.pop()
                t_ = y
            else:
                y = int(D2[t_, m_])
                if y == t_:
                    # nothing lies to the right: the internal state stays in the working
                    # core, which is outside the budget
                    sweep(s, y, "core")
                    mach.backward(s + y)
                else:
                    units = b if (b is not None and y == 1) else a
                    sweep(s, y, "internal")
                    mach.push("internal", s + y, units)
                    exec_msm(t_ - y, m_ - units, s + y)
                    mach.backward(s + y)
                    mach.pop()
                t_ = y - 1

    import sys
    old = sys.getrecursionlimit()
    sys.setrecursionlimit(max(old, 10 * t + 1000))
    try:
        if int(tables["C"][t, m]) >= INF:
            raise ProtocolError("infeasible budget")
        {HSM: exec_hsm, ISM: exec_ism, MSM: exec_msm}[mode](t, m, 0)
    finally:
        sys.setrecursionlimit(old)
    if mach.next_backward != 0:
        raise ProtocolError("not every step was backpropagated")
    if mach.stack:
        raise ProtocolError("stack not empty at the end")
    return {
        "forwards": mach.forwards,
        "backwards": t,
        "peak_units": mach.peak,
        "ops": mach.ops,
    }
