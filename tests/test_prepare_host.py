"""Host logic of the executor's cache of prepared steps (no GPU needed).

What a training step derives from the descriptor and the plan -- work items, input-projection
windows, the tape in the kernels' format -- is made once per (problem, plan, workspace) and
looked up afterwards; freeing a plan drops what was made for it.
"""
import gc

from paper_1606_03401_b200 import binding as B


def _stats():
    return B.mebptt_lstm_prepare_stats()


def test_a_set_is_built_once_and_then_reused():
    desc = B.make_desc(1, 128, 256, 128, 64, 150, "bf16")
    plan = B.mebptt_plan(150, 9, B.MEBPTT_MSM)
    s0 = _stats()
    B.mebptt_lstm_prepare(desc, plan)
    s1 = _stats()
    assert s1["built"] == s0["built"] + 1 and s1["reused"] == s0["reused"] and s1["held"] == s0["held"] + 1
    for _ in range(3):
        B.mebptt_lstm_prepare(desc, plan)
    s2 = _stats()
    assert s2["built"] == s1["built"] and s2["reused"] == s1["reused"] + 3 and s2["held"] == s1["held"]
    # counting launches goes through the same set
    n = B.mebptt_lstm_launch_count(desc, plan)
    assert n > 0 and _stats()["built"] == s2["built"]


def test_another_problem_or_plan_gets_its_own_set_and_freeing_a_plan_drops_its_sets():
    desc = B.make_desc(1, 128, 256, 128, 64, 150, "bf16")
    desc_dx = B.make_desc(1, 128, 256, 128, 64, 150, "bf16", want_dx=1)
    desc_b = B.make_desc(1, 128, 256, 128, 32, 150, "bf16")
    p1 = B.mebptt_plan(150, 9, B.MEBPTT_MSM)
    p2 = B.mebptt_plan(150, 9, B.MEBPTT_MSM)          # same policy, another plan object
    s0 = _stats()
    for d, p in ((desc, p1), (desc_dx, p1), (desc_b, p1), (desc, p2)):
        B.mebptt_lstm_prepare(d, p)
    del d, p
    s1 = _stats()
    assert s1["built"] == s0["built"] + 4 and s1["held"] == s0["held"] + 4
    del p1
    gc.collect()
    s2 = _stats()
    assert s2["held"] == s1["held"] - 3               # the three sets of p1 went with it
    B.mebptt_lstm_prepare(desc, p2)
    assert _stats()["reused"] == s2["reused"] + 1
    del p2
    gc.collect()
    assert _stats()["held"] == s2["held"] - 1


def test_the_cache_holds_eight_sets_and_evicts_the_least_recently_used():
    plans = [B.mebptt_plan(60, m, B.MEBPTT_HSM) for m in range(2, 12)]
    desc = B.make_desc(1, 64, 64, 64, 16, 60, "bf16")
    for p in plans:
        B.mebptt_lstm_prepare(desc, p)
    del p
    s = _stats()
    assert s["held"] == 8
    B.mebptt_lstm_prepare(desc, plans[-1])            # most recent: still there
    assert _stats()["built"] == s["built"]
    B.mebptt_lstm_prepare(desc, plans[0])             # the oldest was evicted: built again
    assert _stats()["built"] == s["built"] + 1
    del plans
    gc.collect()
    assert _stats()["held"] == 0


def test_paths_without_a_device_tape_need_no_preparation():
    desc = B.make_desc(1, 32, 64, 32, 4, 64, "fp32")
    plan = B.mebptt_plan(64, 8, B.MEBPTT_HSM)
    s0 = _stats()
    B.mebptt_lstm_prepare(desc, plan)
    assert _stats() == s0
