"""Host side of the library (no GPU): planner against the oracle, tape validity, exported symbols."""
import os
import re

import numpy as np
import pytest

from oracle import policy as P

B = pytest.importorskip("paper_1606_03401_b200.binding")

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

SMALL = [(t, m) for t in (1, 2, 3, 5, 8, 13, 31, 64) for m in (1, 2, 3, 4, 7, 8, 20, 70, 300)]


def _oracle_cost(mode, t, m, alpha=4, beta=None):
    m = min(m, P.saturation_budget(mode, t, alpha))
    return P.cost(mode, t, m, alpha, beta)


@pytest.mark.parametrize("mode", [P.HSM, P.ISM, P.MSM])
def test_costs_match_oracle_bit_exactly(mode):
    for t, m in SMALL:
        plan = B.mebptt_plan(t, m, mode)
        assert plan.cost == _oracle_cost(mode, t, m), (mode, t, m)
        assert plan.peak_units <= min(m, plan.m)
        assert plan.validate() == B.MEBPTT_OK


@pytest.mark.parametrize("alpha,beta", [(2, 0), (3, 0), (5, 0), (4, 3), (5, 4), (4, 1), (6, 6)])
def test_msm_alpha_beta_costs(alpha, beta):
    for t, m in [(1, 1), (7, 3), (20, 9), (40, 17), (64, 8), (33, 200)]:
        plan = B.mebptt_plan_ex(t, m, B.MEBPTT_MSM, alpha, beta)
        assert plan.cost == _oracle_cost(P.MSM, t, m, alpha, beta or None), (alpha, beta, t, m)


def test_whole_cost_tables_match_oracle():
    t, m = 90, 40
    for mode in (P.HSM, P.ISM, P.MSM):
        tabs = B.mebptt_plan_ex(t, m, mode, 4, 0).tables()
        ref = P.plan_tables(mode, t, m, 4)
        C = tabs["C"].astype(np.int64)
        Cref = ref["C"]
        if mode == P.HSM:      # row 0 / column 0 are unused there
            assert np.array_equal(C[1:, 1:], Cref[1:, 1:])
        else:
            assert np.array_equal(C[:, 1:], Cref[:, 1:])
    # section 3.4 variant
    tabs = B.mebptt_plan_ex(t, m, P.MSM, 4, 3).tables()
    ref = P.plan_tables(P.MSM, t, m, 4, 3)
    assert np.array_equal(tabs["C"][:, 1:], ref["C"][:, 1:])
    assert np.array_equal(tabs["H"][1:, 1:], ref["H"][1:, 1:])
    # the push position matters only for the kind of push that is chosen
    hid, itl = ref["H"] == 1, ref["H"] == 2
    assert np.array_equal(tabs["D"][hid], ref["D1"][hid])
    assert np.array_equal(tabs["D2"][itl], ref["D2"][itl])


@pytest.mark.parametrize("mode", [P.HSM, P.ISM, P.MSM])
def test_convexity_shortcut_changes_no_table_entry(mode, monkeypatch):
    """Where a cost column is convex in t the planner walks from the previous split point instead
    of scanning every y (Appendix A's remark), and the mixed mode's columns are filled by several
    threads; with MEBPTT_PLAN_SCAN=1 one thread scans everywhere.  Both must give the same C and
    the same D (smallest y on ties) in every cell."""
    # (the last size is large enough for the mixed mode's columns to be filled by several threads,
    # which MEBPTT_PLAN_SCAN=1 also turns off)
    for t, m in [(150, 150), (257, 31), (64, 200), (2, 1), (1, 5)] + ([(300, 800)] if mode == P.MSM else []):
        fast = B.mebptt_plan_ex(t, m, mode, 4, 0).tables()
        monkeypatch.setenv("MEBPTT_PLAN_SCAN", "1")
        slow = B.mebptt_plan_ex(t, m, mode, 4, 0).tables()
        monkeypatch.delenv("MEBPTT_PLAN_SCAN")
        for k in fast:
            assert np.array_equal(fast[k], slow[k]), (mode, t, m, k)


def test_long_sequence_plans_match_oracle_columns():
    """t = 4000 (config 4): the fast path's costs against the oracle's own DP at a few budgets."""
    for mode, m in [(P.ISM, 20), (P.ISM, 50), (P.HSM, 12)]:
        plan = B.mebptt_plan_ex(4000, m, mode, 4, 0)
        assert plan.cost == _oracle_cost(mode, 4000, m)
        assert plan.validate() == B.MEBPTT_OK


def test_benchmark_budgets_match_oracle():
    """The (t, m) points of the timed workloads; the oracle runs its own DP for each."""
    for mode, t, m, alpha, beta in [(P.HSM, 64, 8, 4, 0), (P.HSM, 256, 16, 4, 0), (P.ISM, 256, 64, 4, 0),
                                    (P.MSM, 1000, 10, 4, 0), (P.MSM, 1000, 32, 4, 0),
                                    (P.MSM, 1000, 100, 4, 0), (P.ISM, 1000, 50, 4, 0)]:
        plan = B.mebptt_plan_ex(t, m, mode, alpha, beta)
        assert plan.cost == _oracle_cost(mode, t, m, alpha, beta or None)


def _replay(plan):
    """Replays the tape with the oracle's abstract machine (integer bookkeeping only)."""
    tape = plan.tape()
    t = plan.t
    where = {B.MEBPTT_LOC_INIT: ("hidden", 0)}   # location -> (format, step)
    nxt, forwards = t, 0
    for op in tape:
        k = int(op["k"])
        if op["kind"] == B.MEBPTT_OP_FWD:
            src = where.get(int(op["src"]))
            assert src is not None and src[1] == k - 1, f"forward {k}: state {k - 1} not at src"
            forwards += 1
            # arena: anything at or above the written offset is gone
            dst = int(op["dst"])
            if dst >= 0:
                for loc in [l for l in where if l >= dst]:
                    del where[loc]
            where[dst] = ("hidden" if op["dst_fmt"] == B.MEBPTT_FMT_HIDDEN else "internal", k)
        else:
            assert k == nxt
            rec = where.get(int(op["src"]))
            assert rec == ("internal", k), f"backward {k}: no internal state at src"
            if op["dst_fmt"] == B.MEBPTT_FMT_INTERNAL_NOINPUT:
                aux = where.get(int(op["aux"]))
                assert aux is not None and aux[1] == k - 1
            nxt -= 1
    assert nxt == 0
    return forwards


@pytest.mark.parametrize("mode,t,m,alpha,beta", [
    (P.HSM, 64, 8, 4, 0), (P.HSM, 40, 1, 4, 0), (P.HSM, 50, 50, 4, 0), (P.HSM, 100, 3, 4, 0),
    (P.ISM, 64, 8, 4, 0), (P.ISM, 30, 30, 4, 0), (P.ISM, 30, 1, 4, 0),
    (P.MSM, 64, 8, 4, 0), (P.MSM, 64, 8, 4, 3), (P.MSM, 100, 37, 4, 3), (P.MSM, 50, 197, 4, 0),
    (P.MSM, 50, 1, 4, 0), (P.MSM, 256, 64, 5, 4)])
def test_tape_replay_counts_C_forwards(mode, t, m, alpha, beta):
    plan = B.mebptt_plan_ex(t, m, mode, alpha, beta)
    assert _replay(plan) == plan.cost == _oracle_cost(mode, t, m, alpha, beta or None)
    tape = plan.tape()
    assert plan.num_ops == len(tape) == plan.cost + t
    assert int(tape["units"].max()) == plan.peak_units <= plan.m
    # the oracle's own simulation of the protocol gives the same forward count and peak
    sim = P.simulate(mode, t, plan.m, alpha=alpha, beta=beta or None)
    assert sim["forwards"] == plan.cost
    assert sim["peak_units"] == plan.peak_units
    # and the same sequence of operations
    mine = [("F", int(o["k"])) if o["kind"] == B.MEBPTT_OP_FWD else ("B", int(o["k"])) for o in tape]
    assert mine == [(o[0], o[1]) for o in sim["ops"]]


def test_budget_clamping_and_errors():
    assert B.mebptt_plan(10, 10 ** 9, B.MEBPTT_HSM).m == 10
    assert B.mebptt_plan(10, 10 ** 9, B.MEBPTT_ISM).cost == 10
    p = B.mebptt_plan(10, 10 ** 9, B.MEBPTT_MSM)
    assert p.m == 4 * 9 + 1 and p.cost == 10
    for bad in (0, -3):
        with pytest.raises(B.MebpttError) as e:
            B.mebptt_plan(10, bad, B.MEBPTT_HSM)
        assert e.value.status == B.MEBPTT_ERR_BUDGET
    with pytest.raises(B.MebpttError) as e:
        B.mebptt_plan(0, 4, B.MEBPTT_HSM)
    assert e.value.status == B.MEBPTT_ERR_ARG
    with pytest.raises(B.MebpttError):
        B.mebptt_plan(10, 4, 7)
    with pytest.raises(B.MebpttError):
        B.mebptt_plan_ex(10, 4, B.MEBPTT_MSM, 1, 0)
    with pytest.raises(B.MebpttError):
        B.mebptt_plan_ex(10, 4, B.MEBPTT_MSM, 4, 5)


def test_plan_from_a_byte_budget():
    """Budgets in bytes (config 5's way of stating them): the mode's own unit, and, when the
    working memory is to be counted, the largest m whose whole workspace fits."""
    desc = B.make_desc(2, 1024, 2048, 1024, 128, 1000, "bf16")
    unit = B.mebptt_lstm_unit_bytes(desc)
    assert unit == 2 * 128 * 2048 * 6
    plan = B.mebptt_plan_for_bytes(desc, 1 << 30, B.MEBPTT_MSM)
    assert plan.m == 341 and plan.cost == _oracle_cost(P.MSM, 1000, 341)
    assert B.mebptt_plan_for_bytes(desc, 4 << 30, B.MEBPTT_MSM).m == 1365
    # 16 GiB is past the point where the cost stops falling: clamped, full memory
    assert B.mebptt_plan_for_bytes(desc, 16 << 30, B.MEBPTT_MSM).cost == 1000
    # internal states cost four units each
    assert B.mebptt_plan_for_bytes(desc, 1 << 30, B.MEBPTT_ISM).m == (1 << 30) // (4 * unit)
    # counting the working memory: the workspace fits, and one more unit would not
    small = B.make_desc(1, 256, 256, 256, 64, 300, "bf16")
    u = B.mebptt_lstm_unit_bytes(small)
    for mode in (B.MEBPTT_HSM, B.MEBPTT_ISM, B.MEBPTT_MSM):
        free = B.mebptt_plan_for_bytes(small, 64 << 20, mode)
        budget = B.mebptt_lstm_working_bytes(small, free) + 37 * u + 1000
        plan = B.mebptt_plan_for_bytes(small, budget, mode, include_working=True)
        assert B.mebptt_lstm_workspace_bytes(small, plan) <= budget
        nxt = B.mebptt_plan_ex(300, plan.m + 1, mode, 4, 0)
        assert nxt.m == plan.m or B.mebptt_lstm_workspace_bytes(small, nxt) > budget
        assert 1 <= plan.m <= 37
    with pytest.raises(B.MebpttError) as e:
        B.mebptt_plan_for_bytes(small, 4096, B.MEBPTT_MSM, include_working=True)
    assert e.value.status == B.MEBPTT_ERR_BUDGET
    with pytest.raises(B.MebpttError) as e:
        B.mebptt_plan_for_bytes(small, u - 1, B.MEBPTT_HSM)
    assert e.value.status == B.MEBPTT_ERR_BUDGET


def test_descriptor_queries():
    d = B.make_desc(1, 1024, 1024, 1024, 64, 1000, "bf16")
    unit = B.mebptt_lstm_unit_bytes(d)
    assert unit == 64 * 1024 * 6                       # h in bf16, c in fp32
    assert B.mebptt_budget_bytes_to_units(d, 10 * unit + 5) == 10
    d2 = B.make_desc(2, 1024, 2048, 1024, 128, 1000, "bf16")
    assert B.mebptt_lstm_unit_bytes(d2) == 2 * 128 * 2048 * 6
    assert B.mebptt_budget_bytes_to_units(d2, 1 << 30) == 341
    plan = B.mebptt_plan(1000, 32, B.MEBPTT_MSM)
    ws = B.mebptt_lstm_workspace_bytes(d, plan)
    working = B.mebptt_lstm_working_bytes(d, plan)
    assert ws - working == plan.arena_units * unit
    assert B.mebptt_lstm_host_workspace_bytes(d, plan) > ws
    # a plan for another sequence length is refused
    assert B.mebptt_lstm_workspace_bytes(d, B.mebptt_plan(999, 32, B.MEBPTT_MSM)) == 0
    # alpha too small for the LSTM's internal state
    assert B.mebptt_lstm_workspace_bytes(d, B.mebptt_plan_ex(1000, 32, B.MEBPTT_MSM, 3, 0)) == 0
    bad = B.make_desc(0, 4, 4, 4, 4, 4, "fp32")
    assert B.mebptt_lstm_unit_bytes(bad) == 0


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "mebptt.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(mebptt_[a-z0-9_]+)\s*\(", header))
    assert len(declared) >= 20
    for name in declared:
        assert hasattr(B.lib, name), f"{name} declared in mebptt.h but not exported"
    assert declared == set(B.EXPORTED)


def test_train_step_argument_errors_need_no_gpu():
    """Host-detectable errors return before any CUDA call."""
    import ctypes as C
    d = B.make_desc(1, 4, 4, 4, 2, 8, "fp32")
    plan = B.mebptt_plan(8, 3, B.MEBPTT_HSM)
    nul = [None] * 8
    st = B.lib.mebptt_lstm_train_step(C.byref(d), plan.handle, *nul, None, 0, None, *([None] * 7))
    assert st == B.MEBPTT_ERR_ARG
    st = B.lib.mebptt_slot_copy(None, None, 16, None)
    assert st == B.MEBPTT_ERR_ARG
    assert B.mebptt_strerror(B.MEBPTT_ERR_BUDGET).startswith("memory budget")


@pytest.mark.parametrize("beta", [0, 3])
def test_chen_sqrt_schedule(beta):
    """Chen's sqrt(t) schedule as a tape: cost and memory as the oracle derives them from the
    description of Section 2.2, and never cheaper than the DP at the same memory (Section 4.1)."""
    for t in (1, 2, 3, 7, 10, 17, 64, 100, 256, 1000):
        plan = B.mebptt_plan_chen_sqrt(t, 4, beta)
        ref = P.chen_sqrt(t, 4, beta or None)
        assert plan.mode == B.MEBPTT_CHEN_SQRT
        assert plan.cost == ref["forwards"] and plan.peak_units == ref["units"] == plan.m
        assert plan.validate() == B.MEBPTT_OK
        assert _replay(plan) == plan.cost
        assert P.cost(P.MSM, t, plan.peak_units, 4, beta or None) <= plan.cost
        assert "C" not in plan.tables()
    # two forward operations per step on average, at most (Section 2.2)
    assert B.mebptt_plan_chen_sqrt(1000, 4, 3).cost <= 2 * 1000


@pytest.mark.parametrize("beta", [0, 3])
def test_chen_recursive_schedule(beta):
    """Chen's recursive schedule as a tape: cost and memory as the oracle derives them from the
    description of Section 2.2; never cheaper than the DP at the same memory (Section 4.1); for
    k = 1 (bisection) the memory is about log2 t hidden states, and the cost grows like
    t log t (Section 2.2's figures)."""
    import math
    for t in (1, 2, 3, 7, 10, 17, 64, 100, 257, 1000):
        for k in (1, 2, 3, 8, 31):
            plan = B.mebptt_plan_chen_recursive(t, k, 4, beta)
            ref = P.chen_recursive(t, k, 4, beta or None)
            assert plan.mode == B.MEBPTT_CHEN_RECURSIVE
            assert plan.cost == ref["forwards"] and plan.peak_units == ref["units"] == plan.m, (t, k)
            assert plan.validate() == B.MEBPTT_OK
            assert _replay(plan) == plan.cost
            assert P.cost(P.MSM, t, plan.peak_units, 4, beta or None) <= plan.cost
    per = 3
    bis = B.mebptt_plan_chen_recursive(1024, 1, 4, per)
    # ten levels of one cut each, the start state, and one internal state at the bottom
    assert bis.peak_units == 1 + 10 + per
    assert bis.cost == 1024 + 10 * 512
    # with t <= k there is nothing to cut: standard BPTT
    assert B.mebptt_plan_chen_recursive(20, 20, 4, 0).cost == 20
    with pytest.raises(B.MebpttError):
        B.mebptt_plan_chen_recursive(10, 0, 4, 3)


@pytest.mark.parametrize("sigma,alpha,beta", [(3, 10, 7), (3, 10, 0), (2, 5, 3), (1, 4, 3), (5, 17, 12)])
def test_sized_mixed_planner_matches_oracle_tables_and_replays(sigma, alpha, beta):
    """mebptt_plan_sized (a hidden state of sigma units, internal states of alpha / beta) against
    the oracle's recursion over the same sizes: every cost of the table, and a tape that replays
    within the budget with exactly C(t, m) forward operations."""
    from oracle import policy as P
    t = 45
    for m in [sigma, sigma + 1, alpha + sigma - 1, alpha + sigma, 3 * alpha, 7 * alpha + 2, alpha * t + sigma + 5]:
        plan = B.mebptt_plan_sized(t, m, sigma, alpha, beta)
        ref = P.msm_tables(t, plan.m, alpha, beta or None, sigma)[0]
        C = plan.tables()["C"]
        assert np.array_equal(np.minimum(C, P.INF), np.minimum(ref, P.INF)), (m,)
        assert plan.cost == ref[t, plan.m] and plan.sigma == sigma
        assert plan.peak_units <= plan.m and B.lib.mebptt_plan_validate(plan.handle) == 0
        fwd = int((plan.tape()["kind"] == B.MEBPTT_OP_FWD).sum())
        assert fwd == plan.cost
    with pytest.raises(B.MebpttError):
        B.mebptt_plan_sized(t, sigma - 1 if sigma > 1 else 0, sigma, alpha, beta)   # not even the start state fits


def test_plan_bytes_exact_uses_the_layout_sizes():
    """Config 5's layout (two layers, bfloat16 h and gates, float32 c): hidden : internal : without
    input state = 3 : 10 : 7 units of 1 MiB.  At 1 GiB the exact sizes save forward operations
    against internal states rounded up to 4 (3) hidden states, and never cost more."""
    from oracle import policy as P
    desc = B.make_desc(2, 1024, 2048, 1024, 128, 1000, "bf16")
    exact = B.mebptt_plan_bytes_exact(desc, 1 << 30)
    assert (exact.sigma, exact.alpha, exact.beta, exact.m) == (3, 10, 7, 1024)
    assert exact.cost == P.cost(P.MSM, 1000, 1024, 10, 7, 3)
    rounded = B.mebptt_plan_ex(1000, B.mebptt_budget_bytes_to_units(desc, 1 << 30), B.MEBPTT_MSM, 4, 3)
    assert exact.cost < rounded.cost
    assert B.mebptt_lstm_workspace_bytes(desc, exact) > 0
    # a float32 layout is 1 : 4 : 3 already
    d32 = B.make_desc(1, 32, 64, 32, 4, 64, "fp32")
    p32 = B.mebptt_plan_bytes_exact(d32, 20 * B.mebptt_lstm_unit_bytes(d32))
    assert (p32.sigma, p32.alpha, p32.beta, p32.m) == (1, 4, 3, 20)
    # the whole workspace inside the budget
    inside = B.mebptt_plan_bytes_exact(desc, 2 << 30, True, True)
    assert B.mebptt_lstm_workspace_bytes(desc, inside) <= 2 << 30
    # a plan over sizes the layout does not fit is refused at execution time (here: at sizing time)
    tight = B.mebptt_plan_sized(1000, 300, 3, 9, 7)      # internal states one unit too small for this layout
    assert B.mebptt_lstm_workspace_bytes(desc, tight) == 0
