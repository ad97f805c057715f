"""Pins for oracle.policy: brute force, the paper's closed forms, bounds and ordering claims."""
import math
import os

import numpy as np
import pytest

from oracle import bruteforce as BF
from oracle import policy as P

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_policy_facts.txt")


# ---------------------------------------------------------------- brute force
@pytest.mark.parametrize("t", range(1, 9))
def test_hsm_ism_match_unrestricted_search(t):
    C, _ = P.hsm_tables(t, t + 2)
    Ci, _ = P.ism_tables(t, t + 2)
    for m in range(1, t + 3):
        assert BF.hsm_unrestricted(t, m) == C[t, m], (t, m)
        assert BF.ism_unrestricted(t, m) == Ci[t, m], (t, m)


@pytest.mark.parametrize("alpha,beta", [(2, None), (3, None), (4, None), (5, None),
                                        (4, 3), (3, 2), (2, 1), (4, 2)])
def test_msm_matches_protocol_enumeration(alpha, beta):
    for t in range(1, 8):
        mm = alpha * t + 1
        C = P.msm_tables(t, mm, alpha, beta)[0]
        for m in range(1, mm + 1):
            assert BF.msm_protocol(t, m, alpha, beta) == C[t, m], (t, m)


def test_bruteforce_detects_planted_mistakes():
    """A wrong index or a dropped term in the recursion must disagree with the search."""
    def hsm_wrong(t_max, m_max, variant):
        C = np.full((t_max + 1, m_max + 1), P.INF, dtype=np.int64)
        C[1, 1:] = 1
        for t in range(1, t_max + 1):
            C[t, 1] = t * (t + 1) // 2
        for m in range(2, m_max + 1):
            for t in range(2, t_max + 1):
                best = P.INF
                for y in range(1, t):
                    if variant == "no_y":
                        q = C[t - y, m - 1] + C[y, m]
                    elif variant == "swap_m":
                        q = y + C[t - y, m] + C[y, m - 1]
                    else:  # right part keeps the full budget
                        q = y + C[t - y, m] + C[y, m] if t - y < t else P.INF
                    best = min(best, q)
                C[t, m] = best
        return C
    for variant in ("no_y", "swap_m"):
        C = hsm_wrong(7, 5, variant)
        bad = [(t, m) for t in range(2, 8) for m in range(2, 6)
               if BF.hsm_unrestricted(t, m) != C[t, m]]
        assert bad, variant


# ---------------------------------------------------------------- closed forms
def test_hsm_boundaries():
    C, D = P.hsm_tables(120, 130)
    for t in range(1, 121):
        assert C[t, 1] == t * (t + 1) // 2                    # Section 3.1
        for m in range(t, 131):
            assert C[t, m] == 2 * t - 1                       # Section 3.1
        assert all(C[1, 1:] == 1)
    # Algorithm 1 sets D = 1 in the plentiful regime: it must be *an* argmin there
    for t in range(2, 60):
        for m in (t, t + 3):
            assert 1 + C[t - 1, m - 1] + C[1, m] == C[t, m]


def test_ism_boundaries():
    C, _ = P.ism_tables(120, 130)
    assert all(C[0, :] == 0)
    for t in range(1, 121):
        assert C[t, 1] == t * (t + 1) // 2                    # Section 3.2
        assert C[t, 0] >= P.INF
        for m in range(t, 131):
            assert C[t, m] == t                               # Section 3.2
        if t >= 2:
            assert C[t, t - 1] > t


@pytest.mark.parametrize("alpha", [2, 4, 5])
def test_msm_boundaries(alpha):
    t_max = 40
    C, H, D1, D2 = P.msm_tables(t_max, alpha * t_max + 2, alpha)
    for t in range(1, t_max + 1):
        assert C[t, 1] == t * (t + 1) // 2                    # Section 3.3
        for m in range(alpha * t, alpha * t_max + 3):
            assert C[t, m] == t                               # Section 3.3
        assert C[1, 1] == 1
    # the smallest budget that reaches C = t
    for t in range(2, t_max + 1):
        sat = P.saturation_budget(P.MSM, t, alpha)
        assert C[t, sat] == t and C[t, sat - 1] > t


def test_golden_facts_from_the_paper():
    cache = {}
    n = 0
    for line in open(GOLDEN):
        line = line.split("#")[0].split()
        if not line:
            continue
        mode, rel, t, m, val = line[0], line[1], int(line[2]), int(line[3]), int(line[4])
        key = (mode, t, m)
        if key not in cache:
            if mode == "hsm":
                cache[key] = int(P.hsm_tables(t, m)[0][t, m])
            elif mode == "ism":
                cache[key] = int(P.ism_tables(t, m)[0][t, m])
            else:
                cache[key] = int(P.msm_tables(t, m, int(mode[3:]))[0][t, m])
        c = cache[key]
        assert (c == val) if rel == "eq" else (c <= val), (mode, rel, t, m, val, c)
        n += 1
    assert n >= 10


# ---------------------------------------------------------------- bounds of Section 3.5 / App. B
def test_hsm_upper_bounds_and_monotonicity():
    t_max, m_max = 400, 40
    C, _ = P.hsm_tables(t_max, m_max)
    for m in range(1, m_max + 1):
        col = C[1:, m]
        assert np.all(np.diff(col) > 0)                        # increasing in t (App. B.2)
        for t in range(1, t_max + 1):
            bound = t ** (1.0 + 1.0 / m)
            assert C[t, m] <= m * bound + 1e-9                 # Proposition 1
            if m >= 2 or t < 8:
                assert C[t, m] < 4 * bound                     # numerical claim of Section 3.5
    # more memory never hurts
    assert np.all(np.diff(C[1:, 1:], axis=1) <= 0)
    # short-sequence regime: C <= (a + 1) t whenever t <= m^a / a!
    for m in range(2, m_max + 1):
        for a in range(1, 5):
            lim = m ** a / math.factorial(a)
            for t in range(1, t_max + 1):
                if t <= lim:
                    assert C[t, m] <= (a + 1) * t, (t, m, a)


def test_ism_short_sequence_bound():
    t_max, m_max = 300, 30
    C, _ = P.ism_tables(t_max, m_max)
    for m in range(2, m_max + 1):
        for a in range(1, 5):
            lim = m ** a / math.factorial(a)
            for t in range(1, t_max + 1):
                if t <= lim:
                    assert C[t, m] <= a * t, (t, m, a)         # App. B.3
    assert np.all(np.diff(C[:, 1:], axis=0) > 0)
    assert np.all(np.diff(C[1:, 1:], axis=1) <= 0)


def test_ordering_of_the_three_schemes():
    """Section 3.6 and the caption of the ISM/MSM cost figure, alpha = 5."""
    alpha, t_max = 5, 300
    m_hid = 50
    Ch, _ = P.hsm_tables(t_max, m_hid)
    Ci, _ = P.ism_tables(t_max, m_hid // alpha)
    Cm = P.msm_tables(t_max, m_hid, alpha)[0]
    for t in range(1, t_max + 1):
        for m in (5, 10, 25, 50):
            assert Cm[t, m] <= Ch[t, m]
            assert Cm[t, m] <= Ci[t, m // alpha]
    # hidden states win for long sequences, internal states for short ones
    assert Ci[50, 10] < Ch[50, 50]
    Ch1000 = P.hsm_tables(1000, 50)[0]
    Ci1000 = P.ism_tables(1000, 10)[0]
    assert Ch1000[1000, 50] < Ci1000[1000, 10]


# ---------------------------------------------------------------- argmin validity, protocol simulation
def test_tables_are_self_consistent():
    t_max, m_max, alpha = 60, 40, 4
    C, D = P.hsm_tables(t_max, m_max)
    for t in range(2, t_max + 1):
        for m in range(2, m_max + 1):
            y = D[t, m]
            assert 1 <= y < t and y + C[t - y, m - 1] + C[y, m] == C[t, m]
    C, D = P.ism_tables(t_max, m_max)
    for t in range(1, t_max + 1):
        for m in range(1, m_max + 1):
            y = D[t, m]
            assert 1 <= y <= t and y + C[y - 1, m] + C[t - y, m - 1] == C[t, m]


CASES = [(P.HSM, 1, 1), (P.HSM, 2, 1), (P.HSM, 7, 1), (P.HSM, 64, 8), (P.HSM, 50, 50),
         (P.HSM, 33, 2), (P.HSM, 100, 5), (P.ISM, 1, 1), (P.ISM, 64, 8), (P.ISM, 40, 40),
         (P.ISM, 40, 1), (P.ISM, 100, 3), (P.MSM, 1, 1), (P.MSM, 64, 8), (P.MSM, 64, 31),
         (P.MSM, 30, 117), (P.MSM, 30, 1), (P.MSM, 100, 10)]


@pytest.mark.parametrize("mode,t,m", CASES)
def test_protocol_simulation_costs_exactly_C(mode, t, m):
    tabs = P.plan_tables(mode, t, m, alpha=4)
    sim = P.simulate(mode, t, m, tabs)
    assert sim["forwards"] == int(tabs["C"][t, m])
    assert sim["peak_units"] <= m
    assert [op[1] for op in sim["ops"] if op[0] == "B"] == list(range(t, 0, -1))


def test_protocol_simulation_with_beta():
    for t, m in [(20, 7), (50, 12), (30, 90)]:
        tabs = P.plan_tables(P.MSM, t, m, alpha=4, beta=3)
        sim = P.simulate(P.MSM, t, m, tabs)
        assert sim["forwards"] == int(tabs["C"][t, m])
        assert sim["peak_units"] <= m
        assert int(tabs["C"][t, m]) <= P.cost(P.MSM, t, m, alpha=4)


def test_infeasible_budget_is_rejected():
    with pytest.raises(P.ProtocolError):
        P.simulate(P.ISM, 5, 0)


def test_chen_schedules_against_closed_forms():
    """Chen's schedules (Section 2.2) where their cost and memory can be written down by hand.

    sqrt(t) on a perfect square t = s^2: s - 1 segments are run twice, so t + (t - s) forward
    operations, and at the worst moment s - 1 boundaries plus s internal states are kept (plus the
    start state).  Recursive with k = 1 on t = 2^d: every level reruns the first half of each
    piece, t / 2 operations per level over d levels, and keeps one state per level; the last piece
    of one step keeps one internal state.  With k >= t nothing is cut: standard BPTT."""
    for s in (2, 3, 8, 31):
        r = P.chen_sqrt(s * s, 4, 3)
        assert r["forwards"] == 2 * s * s - s and r["units"] == 1 + (s - 1) + 3 * s
        r = P.chen_sqrt(s * s, 4)
        assert r["units"] == 1 + (s - 1) + 4 * s
    for d in (1, 2, 5, 10):
        t = 1 << d
        r = P.chen_recursive(t, 1, 4, 3)
        assert r["forwards"] == t + d * (t // 2) and r["units"] == 1 + d + 3
    for t, k in [(5, 5), (7, 30)]:
        r = P.chen_recursive(t, k, 4)
        assert r["forwards"] == t and r["units"] == 1 + 4 * t
    # k cuts per level: a three-way cut of 9 steps with k = 2 ends in pieces of one step after two
    # levels: passes of 6 and 3 x 2 steps, 9 single steps at the bottom
    r = P.chen_recursive(9, 2, 4, 3)
    assert r["forwards"] == 6 + 3 * 2 + 9 and r["units"] == 1 + 2 + 2 + 3
    # the paper's figures: memory grows like k log_{k+1} t, at least log2 t hidden states at k = 1
    assert P.chen_recursive(1000, 1, 4, 3)["units"] >= 10
    for t in (100, 1000):
        assert P.chen_recursive(t, 3, 4, 3)["forwards"] >= P.cost(P.MSM, t, P.chen_recursive(t, 3, 4, 3)["units"], 4, 3)


# ---------------------------------------------------------------- sizes that are no whole hidden states
@pytest.mark.parametrize("sigma,alpha,beta", [(3, 10, 7), (3, 10, None), (2, 5, 3), (2, 7, None), (1, 4, 3)])
def test_sized_msm_matches_protocol_enumeration(sigma, alpha, beta):
    """The mixed recursion over a finer unit (a hidden state of sigma units, an internal state of
    alpha, beta without its input state -- e.g. 3 : 10 : 7 for bfloat16 h and gates with a float32
    cell state) against the exhaustive enumeration of protocol trees with a unit counter."""
    for t in range(1, 7):
        mm = alpha * t + sigma
        C = P.msm_tables(t, mm, alpha, beta, sigma)[0]
        for m in range(1, mm + 1):
            found = BF.msm_protocol(t, m, alpha, beta, sigma)
            if found is BF.INFEASIBLE:
                assert m < sigma and C[t, m] >= P.INF, (t, m)       # not even the start state fits
            else:
                assert found == C[t, m], (t, m)


def test_sized_msm_closed_forms_and_scaling():
    t_max = 40
    # sigma = 1 is Section 3.3 itself
    for alpha, beta in [(4, None), (4, 3), (5, None)]:
        a = P.msm_tables(t_max, 60, alpha, beta)[0]
        b = P.msm_tables(t_max, 60, alpha, beta, 1)[0]
        assert np.array_equal(a, b)
    # multiplying every size by k changes nothing but the unit: C(t, k m + r; k sigma, k alpha, k beta)
    # = C(t, m; sigma, alpha, beta) for 0 <= r < k
    base = P.msm_tables(t_max, 30, 4, 3)[0]
    k = 3
    scaled = P.msm_tables(t_max, 30 * k + k - 1, 4 * k, 3 * k, k)[0]
    for m in range(1, 31):
        for r in range(k):
            assert np.array_equal(scaled[:, k * m + r], base[:, m]), (m, r)
    assert np.all(scaled[1:, :k] >= P.INF)                 # no room for the start state
    # boundaries of Section 3.3 in the finer unit: only the start state fits -> t (t + 1) / 2;
    # every internal state fits -> t
    C = P.msm_tables(t_max, 10 * t_max + 3, 10, 7, 3)[0]
    for t in range(1, t_max + 1):
        assert C[t, 3] == t * (t + 1) // 2 and C[t, 5] == t * (t + 1) // 2
        assert C[t, 3 + 10 * (t - 1)] == t
    # a finer unit never costs more than rounding the sizes up to whole hidden states: with
    # sizes 3 : 10 : 7 a budget of 3 m units holds what m units hold at 1 : 4 : 3 (= 3 : 12 : 9)
    fine = P.msm_tables(t_max, 3 * 30, 10, 7, 3)[0]
    coarse = P.msm_tables(t_max, 30, 4, 3)[0]
    for m in range(1, 31):
        assert np.all(fine[:, 3 * m] <= coarse[:, m])
    assert np.any(fine[:, 3 * 8] < coarse[:, 8])


def test_sized_msm_protocol_runs_within_budget():
    for t, m in [(30, 20), (57, 41), (100, 100), (100, 33)]:
        tab = P.plan_tables(P.MSM, t, m, 10, 7, 3)
        r = P.simulate(P.MSM, t, m, tab)
        assert r["forwards"] == tab["C"][t, m] and r["peak_units"] <= m and r["backwards"] == t
