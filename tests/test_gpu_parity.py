"""GPU parity: the CUDA path, called through the C interface, against the fp64 oracle."""
import numpy as np
import pytest

from oracle import policy as P
from paper_1606_03401_b200 import synth
from tests.util import assert_bit_identical, assert_close_to_oracle, oracle_run

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def H():
    from paper_1606_03401_b200 import harness
    return harness


def _cfg(base, **kw):
    return synth.with_overrides(synth.CONFIGS[base], **kw)


def test_c1_hsm_m8_matches_oracle(H):
    """Config 1 in full: fp32, I32 H64 B4 t64, BPTT-HSM with m = 8."""
    cfg = synth.CONFIGS["c1"]
    dp = H.DeviceProblem(cfg, want_dx=True)
    plan = dp.plan("hsm", 8)
    assert plan.cost == P.cost(P.HSM, 64, 8)
    res = dp.run(plan)
    ref = oracle_run(dp.prob)
    assert_close_to_oracle(res, ref, "fp32", want_dx=True)
    c = res["counters"]
    assert c[0] == plan.cost and c[1] == cfg.t and c[2] == plan.peak_units and c[3] == 0


POLICIES = [("hsm", 1), ("hsm", 2), ("hsm", 8), ("hsm", 64), ("ism", 1), ("ism", 3), ("ism", 8),
            ("msm", 1), ("msm", 5), ("msm", 8), ("msm", 40), ("msm", 10 ** 6)]


def test_c1_every_policy_is_bit_identical_to_full_memory(H):
    cfg = synth.CONFIGS["c1"]
    dp = H.DeviceProblem(cfg, want_dx=True)
    full = dp.run(dp.full_memory_plan())
    assert full["counters"][0] == cfg.t
    for mode, m in POLICIES:
        for beta in ((0, 3) if mode == "msm" else (0,)):
            plan = dp.plan(mode, m, beta=beta)
            res = dp.run(plan)
            code = {"hsm": P.HSM, "ism": P.ISM, "msm": P.MSM}[mode]
            assert res["counters"][0] == plan.cost == P.cost(code, cfg.t, plan.m, 4, beta or None)
            assert res["counters"][1] == cfg.t and res["counters"][3] == 0
            assert_bit_identical(res, full, want_dx=True)
    # and twice the same plan gives the same bits
    again = dp.run(dp.full_memory_plan())
    assert_bit_identical(again, full, want_dx=True)


@pytest.mark.parametrize("dtype", ["fp32", "bf16", "tf32"])
@pytest.mark.parametrize("shape", [dict(input=5, hidden=7, batch=3, t=11, readout=3),
                                   dict(input=70, hidden=65, batch=67, t=9, readout=66),
                                   dict(input=1, hidden=1, batch=1, t=1, readout=1)])
def test_ragged_shapes_match_oracle(H, dtype, shape):
    """Sizes that are no multiple of any tile, down to the degenerate 1 x 1 x 1 problem."""
    cfg = _cfg("c1", dtype=dtype, **shape)
    dp = H.DeviceProblem(cfg, want_dx=True)
    ref = oracle_run(dp.prob)
    full = dp.run(dp.full_memory_plan())
    assert_close_to_oracle(full, ref, dtype, want_dx=True)
    for mode, m in [("hsm", 3), ("ism", 2), ("msm", 6)]:
        res = dp.run(dp.plan(mode, m))
        assert_bit_identical(res, full, want_dx=True)


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_two_layers_match_oracle(H, dtype):
    cfg = _cfg("c1", layers=2, dtype=dtype, input=24, hidden=40, batch=6, t=20, readout=10)
    dp = H.DeviceProblem(cfg, want_dx=True)
    ref = oracle_run(dp.prob)
    full = dp.run(dp.full_memory_plan())
    assert_close_to_oracle(full, ref, dtype, want_dx=True)
    for mode, m, beta in [("hsm", 4, 0), ("ism", 3, 0), ("msm", 9, 0), ("msm", 9, 3)]:
        res = dp.run(dp.plan(mode, m, beta=beta))
        assert_bit_identical(res, full, want_dx=True)


def test_nonzero_initial_state_and_no_dx(H):
    cfg = _cfg("c1", t=12)
    prob = synth.make_problem(cfg)
    r = np.random.default_rng(7)
    prob["h0"] = synth.round_to_fp32(r.standard_normal(prob["h0"].shape) * 0.5)
    prob["c0"] = synth.round_to_fp32(r.standard_normal(prob["c0"].shape) * 0.5)
    dp = H.DeviceProblem(cfg, prob, want_dx=False)
    res = dp.run(dp.plan("msm", 7, beta=3))
    assert_close_to_oracle(res, oracle_run(prob), "fp32")


def test_c2_shape_bf16_truncated(H):
    """Config 2's layer sizes (I512 H512 B64, bf16) on a shortened sequence."""
    cfg = _cfg("c2", t=24)
    dp = H.DeviceProblem(cfg)
    ref = oracle_run(dp.prob)
    full = dp.run(dp.full_memory_plan())
    assert_close_to_oracle(full, ref, "bf16")
    for mode, m in [("hsm", 4), ("ism", 4)]:
        plan = dp.plan(mode, m)
        res = dp.run(plan)
        assert res["counters"][0] == plan.cost
        assert_bit_identical(res, full)


@pytest.mark.parametrize("base,kw,mode,m", [("c1", dict(t=16), "hsm", 4),
                                            ("c2", dict(input=128, hidden=256, batch=64, t=150, readout=128), "msm", 9),
                                            ("c5", dict(layers=2, input=64, hidden=72, batch=32, t=21, readout=40), "msm", 9)])
def test_host_buffer_entry_point(H, base, kw, mode, m):
    """Host buffers in, host buffers out, on each of the paths (on the persistent tensor path x and
    the targets are copied in pieces beside the forward pass, the targets last piece first): the
    bits of the device-resident call."""
    import torch
    from paper_1606_03401_b200 import binding as B
    cfg = _cfg(base, **kw)
    dp = H.DeviceProblem(cfg, want_dx=True)
    plan = dp.plan(mode, m)
    dev = dp.run(plan)
    h = dp.host
    out = {k: np.zeros_like(v) for k, v in dev.items() if isinstance(v, np.ndarray)}
    loss = np.zeros(1, np.float32)
    ws = torch.empty(B.mebptt_lstm_host_workspace_bytes(dp.desc, plan), dtype=torch.uint8, device="cuda:0")
    B.mebptt_lstm_train_step_host(dp.desc, plan, h["W"], h["b"], h["W_out"], h["b_out"], h["x"],
                                  h["targets"], h["h0"], h["c0"], ws, None, loss, out["dW"], out["db"],
                                  out["dW_out"], out["db_out"], out["dx"], out["counters"])
    torch.cuda.synchronize()
    out["loss"] = float(loss[0])
    assert_bit_identical(out, dev, want_dx=True)
    assert out["counters"][0] == plan.cost


def test_workspace_errors(H):
    import torch
    from paper_1606_03401_b200 import binding as B
    cfg = _cfg("c1", t=8)
    dp = H.DeviceProblem(cfg)
    plan = dp.plan("hsm", 3)
    need = B.mebptt_lstm_workspace_bytes(dp.desc, plan)
    d, o = dp.dev, dp.out
    small = torch.empty(need - 256, dtype=torch.uint8, device="cuda:0")
    with pytest.raises(B.MebpttError) as e:
        B.mebptt_lstm_train_step(dp.desc, plan, d["W"], d["b"], d["W_out"], d["b_out"], d["x"], d["targets"],
                                 d["h0"], d["c0"], small, None, o["loss"], o["dW"], o["db"], o["dW_out"],
                                 o["db_out"], None, o["counters"])
    assert e.value.status == B.MEBPTT_ERR_WORKSPACE
    big = torch.empty(need + 512, dtype=torch.uint8, device="cuda:0")
    with pytest.raises(B.MebpttError) as e:
        B.mebptt_lstm_train_step(dp.desc, plan, d["W"], d["b"], d["W_out"], d["b_out"], d["x"], d["targets"],
                                 d["h0"], d["c0"], big[16:], None, o["loss"], o["dW"], o["db"], o["dW_out"],
                                 o["db_out"], None, o["counters"])
    assert e.value.status == B.MEBPTT_ERR_WORKSPACE


@pytest.mark.parametrize("nbytes", [16, 4096 + 16, (256 << 10) - 16, 256 << 10, (1 << 20) + 48, 393216 * 4,
                                    (32 << 10) * 148 * 3 + 16, (200 << 20) + 32])
def test_slot_copy(H, nbytes):
    """Byte-exact copies: below and above the switch to bulk asynchronous copies, a ragged last
    chunk, fewer chunks than SMs, several rounds per CTA; the bytes around the destination stay."""
    import torch
    from paper_1606_03401_b200 import binding as B
    g = torch.Generator(device="cuda:0").manual_seed(nbytes % 1000)
    src = torch.randint(0, 255, (nbytes,), dtype=torch.uint8, device="cuda:0", generator=g)
    dst = torch.full((nbytes + 512,), 7, dtype=torch.uint8, device="cuda:0")
    B.mebptt_slot_copy(dst[256:256 + nbytes], src, nbytes, torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    assert torch.equal(src, dst[256:256 + nbytes])
    assert bool((dst[:256] == 7).all()) and bool((dst[256 + nbytes:] == 7).all())


@pytest.mark.parametrize("shape", [dict(input=64, hidden=64, batch=64, t=40, readout=64),
                                   dict(input=72, hidden=200, batch=24, t=37, readout=40),
                                   dict(input=256, hidden=256, batch=64, t=50, readout=256),
                                   # two groups of batch rows, the second one ragged; a K-slice per CTA
                                   # of the backward cluster that is shorter than one copy's box
                                   dict(input=64, hidden=192, batch=40, t=40, readout=48),
                                   dict(input=128, hidden=768, batch=56, t=36, readout=64)])
def test_tensor_core_path_matches_oracle_and_cuda_core_path(H, shape):
    """bf16 shapes the tcgen05 kernels cover: oracle parity, bit identity across plans, and
    agreement with the CUDA-core kernels (same roundings of stored values, other sum order)."""
    from paper_1606_03401_b200 import binding as B
    cfg = _cfg("c2", **shape)
    dp = H.DeviceProblem(cfg, want_dx=True)
    ref = oracle_run(dp.prob)
    full = dp.run(dp.full_memory_plan())
    assert full["counters"][3] == 0
    assert_close_to_oracle(full, ref, "bf16", want_dx=True)
    for mode, m, beta in [("hsm", 1, 0), ("hsm", 5, 0), ("ism", 1, 0), ("ism", 6, 0), ("msm", 9, 0), ("msm", 13, 3)]:
        plan = dp.plan(mode, m, beta=beta)
        res = dp.run(plan)
        assert res["counters"][0] == plan.cost and res["counters"][1] == cfg.t and res["counters"][3] == 0
        assert_bit_identical(res, full, want_dx=True)
    slow = H.DeviceProblem(cfg, dp.prob, want_dx=True, flags=B.MEBPTT_FLAG_NO_TENSOR_CORES)
    other = slow.run(slow.full_memory_plan())
    from tests.util import rel_l2
    for k in ("dW", "db", "dW_out", "db_out", "dx"):
        assert rel_l2(full[k], other[k]) < 1e-2, k


def test_run_times_count_every_backward_operation_and_change_no_result(H):
    """The per-launch event timing: results stay bit-identical, every backward operation is inside
    a timed backward run, forward runs hold at most C(t, m) operations (leaves of the recursion
    are computed in batches outside them), and the collection clears itself."""
    from paper_1606_03401_b200 import binding as B
    cfg = _cfg("c2", input=128, hidden=128, batch=32, t=45, readout=64)
    dp = H.DeviceProblem(cfg)
    plan = dp.plan("hsm", 4)
    plain = dp.run(plan)
    B.mebptt_lstm_run_times()
    dp.desc.flags |= B.MEBPTT_FLAG_TIME_RUNS
    timed = dp.run(plan)
    dp.desc.flags &= ~B.MEBPTT_FLAG_TIME_RUNS
    assert_bit_identical(timed, plain)
    r = B.mebptt_lstm_run_times()
    f_ms, f_n, f_ops = r["forward"]
    b_ms, b_n, b_ops = r["backward"]
    assert b_ops == cfg.t and 0 < b_n <= cfg.t and b_ms > 0
    assert 0 < f_ops <= plan.cost and 0 < f_n <= f_ops and f_ms > 0
    again = B.mebptt_lstm_run_times()
    assert again["forward"][1] == 0 and again["backward"][1] == 0


@pytest.mark.parametrize("shape", [dict(layers=2, input=64, hidden=72, batch=32, t=21, readout=40),
                                   dict(layers=3, input=24, hidden=64, batch=96, t=13, readout=8),
                                   dict(layers=1, input=128, hidden=1152, batch=64, t=9, readout=64),
                                   dict(layers=1, input=64, hidden=128, batch=128, t=17, readout=72)])
def test_stepwise_tensor_core_path_matches_oracle_and_cuda_core_path(H, shape):
    """bf16 shapes outside the persistent kernels' range (several layers, H > 1024, B > 64): every
    operation is a sequence of launches whose contractions run on the tensor cores.  Oracle
    parity, bit identity across plans, agreement with the CUDA-core kernels."""
    from paper_1606_03401_b200 import binding as B
    from tests.util import rel_l2
    cfg = _cfg("c2", **shape)
    dp = H.DeviceProblem(cfg, want_dx=True)
    ref = oracle_run(dp.prob)
    full = dp.run(dp.full_memory_plan())
    assert full["counters"][3] == 0
    assert_close_to_oracle(full, ref, "bf16", want_dx=True)
    for mode, m, beta in [("hsm", 1, 0), ("hsm", 4, 0), ("ism", 2, 0), ("msm", 9, 0), ("msm", 13, 3)]:
        plan = dp.plan(mode, m, beta=beta)
        res = dp.run(plan)
        assert res["counters"][0] == plan.cost and res["counters"][1] == cfg.t and res["counters"][3] == 0
        assert_bit_identical(res, full, want_dx=True)
    slow = H.DeviceProblem(cfg, dp.prob, want_dx=True, flags=B.MEBPTT_FLAG_NO_TENSOR_CORES)
    other = slow.run(slow.full_memory_plan())
    assert abs(other["loss"] - full["loss"]) < 1e-3 * abs(other["loss"])
    for k in ("dW", "db", "dW_out", "db_out", "dx"):
        assert rel_l2(full[k], other[k]) < 1e-2, k
    # without dx the first layer skips its input-gradient contraction; nothing else may change
    nodx = H.DeviceProblem(cfg, dp.prob, want_dx=False)
    res = nodx.run(nodx.plan("msm", 9))
    assert_bit_identical(res, full)


@pytest.mark.parametrize("shape", [dict(layers=2, input=64, hidden=72, batch=32, t=45, readout=40),
                                   dict(layers=3, input=24, hidden=64, batch=96, t=23, readout=8),
                                   dict(layers=2, input=128, hidden=2048, batch=128, t=19, readout=128)])
def test_stepwise_runs_give_the_bits_of_single_operations(H, shape, monkeypatch):
    """The step-by-step tensor-core path takes runs of consecutive operations one layer at a time,
    with the input products, the readout and the gradients handed down batched over the run (at
    config 5's widths some of those contractions are split along K).  Operation by operation
    (MEBPTT_STEPWISE_PER_OP=1) every sum must come out the same, bit for bit, under long runs and
    short ones, with and without dx."""
    cfg = _cfg("c5", **shape)
    for want_dx in (True, False):
        dp = H.DeviceProblem(cfg, want_dx=want_dx)
        plans = [dp.full_memory_plan(), dp.plan("msm", 11), dp.plan("hsm", 3), dp.plan("ism", 2)]
        runs = [dp.run(p) for p in plans]
        monkeypatch.setenv("MEBPTT_STEPWISE_PER_OP", "1")
        single = dp.run(plans[0])
        monkeypatch.delenv("MEBPTT_STEPWISE_PER_OP")
        for p, r in zip(plans, runs):
            assert r["counters"][0] == p.cost and r["counters"][1] == cfg.t and r["counters"][3] == 0
            assert_bit_identical(r, single, want_dx=want_dx)


@pytest.mark.parametrize("shape", [dict(layers=2, input=64, hidden=72, batch=32, t=45, readout=40),
                                   dict(layers=1, input=256, hidden=1024, batch=32, t=70, readout=256)])
def test_float32_storage_run_readout_gives_the_bits_of_single_operations(H, shape, monkeypatch):
    """With float32 storage the readout of a run of backward operations is taken for the whole run
    at once; operation by operation (MEBPTT_STEPWISE_PER_OP=1) the bits must be the same."""
    cfg = _cfg("c4", **shape)
    dp = H.DeviceProblem(cfg, want_dx=True)
    plans = [dp.full_memory_plan(), dp.plan("msm", 11), dp.plan("ism", 3), dp.plan("hsm", 2)]
    runs = [dp.run(p) for p in plans]
    monkeypatch.setenv("MEBPTT_STEPWISE_PER_OP", "1")
    single = dp.run(plans[0])
    monkeypatch.delenv("MEBPTT_STEPWISE_PER_OP")
    for p, r in zip(plans, runs):
        assert r["counters"][0] == p.cost and r["counters"][1] == cfg.t and r["counters"][3] == 0
        assert_bit_identical(r, single, want_dx=True)


@pytest.mark.parametrize("shape", [dict(layers=2, input=64, hidden=72, batch=32, t=21, readout=40),
                                   dict(layers=1, input=24, hidden=256, batch=96, t=13, readout=8),
                                   dict(layers=1, input=128, hidden=1152, batch=32, t=9, readout=64)])
def test_float32_storage_on_tensor_cores_matches_oracle_within_1e_4(H, shape):
    """The tf32 data type: float32 storage, contractions on the tensor cores as three bfloat16
    products per float32 product.  Oracle parity at the float32 tolerance, bit identity across
    plans, agreement with the float32 FMA kernels."""
    from paper_1606_03401_b200 import binding as B
    from tests.util import rel_l2
    cfg = _cfg("c4", **shape)
    assert cfg.dtype == "tf32"
    dp = H.DeviceProblem(cfg, want_dx=True)
    ref = oracle_run(dp.prob)
    full = dp.run(dp.full_memory_plan())
    assert full["counters"][3] == 0
    assert_close_to_oracle(full, ref, "tf32", want_dx=True)
    for mode, m, beta in [("hsm", 1, 0), ("hsm", 4, 0), ("ism", 2, 0), ("msm", 9, 0), ("msm", 13, 3)]:
        plan = dp.plan(mode, m, beta=beta)
        res = dp.run(plan)
        assert res["counters"][0] == plan.cost and res["counters"][1] == cfg.t and res["counters"][3] == 0
        assert_bit_identical(res, full, want_dx=True)
    slow = H.DeviceProblem(cfg, dp.prob, want_dx=True, flags=B.MEBPTT_FLAG_NO_TENSOR_CORES)
    other = slow.run(slow.full_memory_plan())
    for k in ("dW", "db", "dW_out", "db_out", "dx"):
        assert rel_l2(full[k], other[k]) < 1e-4, k


def test_c2_full_size_every_budget(H):
    """Config 2 as timed: I512 H512 B64 t256 bf16, HSM and ISM at m = 16, 64, 256."""
    cfg = synth.CONFIGS["c2"]
    dp = H.DeviceProblem(cfg)
    ref = oracle_run(dp.prob)
    full = dp.run(dp.full_memory_plan())
    assert_close_to_oracle(full, ref, "bf16")
    for mode, code in (("hsm", P.HSM), ("ism", P.ISM)):
        for m in (16, 64, 256):
            plan = dp.plan(mode, m)
            res = dp.run(plan)
            assert res["counters"][0] == plan.cost == P.cost(code, cfg.t, plan.m)
            assert res["counters"][2] == plan.peak_units <= m and res["counters"][3] == 0
            assert_bit_identical(res, full)


def test_c3_full_size_headline_budget(H):
    """Config 3 as the benchmark times it: I1024 H1024 B64 t1000 bf16, MSM m = 100 (and m = 10),
    against the fp64 oracle at full length and bit for bit against the full-memory run."""
    cfg = synth.CONFIGS["c3"]
    dp = H.DeviceProblem(cfg)
    ref = oracle_run(dp.prob)
    full = dp.run(dp.full_memory_plan())
    assert_close_to_oracle(full, ref, "bf16")
    for m in (100, 10):
        plan = dp.plan("msm", m)
        res = dp.run(plan)
        assert res["counters"][0] == plan.cost and res["counters"][1] == cfg.t and res["counters"][3] == 0
        assert_bit_identical(res, full)


@pytest.mark.parametrize("base,kw", [("c1", dict()), ("c2", dict(t=70))])
def test_chen_plans_give_the_same_gradients(H, base, kw):
    """Chen's sqrt(t) and recursive schedules run on the same executor as the DP policies."""
    from paper_1606_03401_b200 import binding as B
    cfg = _cfg(base, **kw)
    dp = H.DeviceProblem(cfg, want_dx=True)
    full = dp.run(dp.full_memory_plan())
    for beta in (0, 3):
        plan = B.mebptt_plan_chen_sqrt(cfg.t, 4, beta)
        res = dp.run(plan)
        assert res["counters"][0] == plan.cost and res["counters"][2] == plan.peak_units and res["counters"][3] == 0
        assert_bit_identical(res, full, want_dx=True)
        for k in (1, 3):
            plan = B.mebptt_plan_chen_recursive(cfg.t, k, 4, beta)
            res = dp.run(plan)
            assert res["counters"][0] == plan.cost and res["counters"][2] == plan.peak_units and res["counters"][3] == 0
            assert_bit_identical(res, full, want_dx=True)


def test_c4_shape_truncated_ism_versus_msm(H):
    """Config 4's layer sizes (I256 H1024 B32, float32 storage) on a shortened sequence: ISM with
    m internal states against MSM with alpha * m hidden-state units, as the paper compares them."""
    cfg = _cfg("c4", t=48)
    dp = H.DeviceProblem(cfg)
    ref = oracle_run(dp.prob)
    full = dp.run(dp.full_memory_plan())
    assert_close_to_oracle(full, ref, "tf32")
    for mode, m in [("ism", 5), ("msm", 20)]:
        plan = dp.plan(mode, m)
        res = dp.run(plan)
        assert res["counters"][0] == plan.cost and res["counters"][3] == 0
        assert_bit_identical(res, full)
    assert dp.plan("msm", 20).cost <= dp.plan("ism", 5).cost      # Section 3.6


def test_c5_shape_truncated_two_layers_byte_budget(H):
    """Config 5's layer sizes (two layers, I1024 H2048 B128, bf16) on a very short sequence, with
    the budget given in bytes and converted to hidden-state units."""
    from paper_1606_03401_b200 import binding as B
    cfg = _cfg("c5", t=6)
    dp = H.DeviceProblem(cfg)
    ref = oracle_run(dp.prob)
    full = dp.run(dp.full_memory_plan())
    assert_close_to_oracle(full, ref, "bf16")
    unit = B.mebptt_lstm_unit_bytes(dp.desc)
    assert unit == 2 * 128 * 2048 * 6
    m = B.mebptt_budget_bytes_to_units(dp.desc, 16 << 20)         # 16 MiB -> 5 units
    assert m == (16 << 20) // unit == 5
    plan = dp.plan("msm", m)
    res = dp.run(plan)
    assert res["counters"][0] == plan.cost and res["counters"][2] <= m
    assert_bit_identical(res, full)


def test_c5_full_size_properties(H):
    """Config 5 as specified (two layers, I1024 H2048 B128 t1000, bf16) with the 1 GiB budget:
    bit identity with the full-memory run, forward count equal to C(t, m), peak within budget."""
    from paper_1606_03401_b200 import binding as B
    cfg = synth.CONFIGS["c5"]
    dp = H.DeviceProblem(cfg)
    m = B.mebptt_budget_bytes_to_units(dp.desc, 1 << 30)
    assert m == 341
    full = dp.run(dp.full_memory_plan())
    assert full["counters"][0] == cfg.t and full["counters"][3] == 0 and np.isfinite(full["loss"])
    plan = dp.plan("msm", m)
    res = dp.run(plan)
    assert res["counters"][0] == plan.cost == P.cost(P.MSM, cfg.t, m, alpha=4)
    assert res["counters"][1] == cfg.t and res["counters"][2] <= m and res["counters"][3] == 0
    assert_bit_identical(res, full)


GENERAL_CASES = [
    # CUDA-core path (float32)
    ("c1", dict(t=24)),
    # persistent tensor path, config 2's widths, more than two staged chunks of S = 32 steps
    ("c2", dict(t=70)),
    # persistent tensor path, batch below the tile height and a hidden size that is no multiple of 64
    ("c2", dict(input=72, hidden=200, batch=24, t=37, readout=40)),
    # step-by-step bf16 path, two layers, more than two chunks of S = 32 steps
    ("c5", dict(layers=2, input=64, hidden=72, batch=32, t=70, readout=40)),
    # step-by-step path for float32 storage, more than two chunks
    ("c4", dict(layers=1, input=64, hidden=128, batch=32, t=70, readout=40)),
    ("c4", dict(layers=2, input=40, hidden=72, batch=32, t=37, readout=24)),
]


@pytest.mark.parametrize("base,kw", GENERAL_CASES)
def test_general_biases_and_initial_state_match_oracle_on_every_path(H, base, kw):
    """Every bias entry, the readout bias and the initial state drawn at random (the benchmark
    recipe leaves them at constants, which cannot expose a misplaced bias entry, a dropped readout
    bias or a mishandled caller's (h0, c0)): oracle parity per tensor and per block with dx, under
    full memory and one plan of each kind, on each of the four kernel paths."""
    cfg = _cfg(base, **kw)
    prob = synth.make_problem(cfg, general=True)
    assert np.abs(prob["b_out"]).min() > 0 and np.abs(prob["h0"]).max() > 0.5 and np.abs(prob["c0"]).max() > 0.5
    dp = H.DeviceProblem(cfg, prob, want_dx=True)
    ref = oracle_run(prob)
    full = dp.run(dp.full_memory_plan())
    assert full["counters"][3] == 0
    assert_close_to_oracle(full, ref, cfg.dtype, want_dx=True)
    for mode, m, beta in [("hsm", 5, 0), ("ism", 3, 0), ("msm", 13, 3)]:
        plan = dp.plan(mode, m, beta=beta)
        res = dp.run(plan)
        assert res["counters"][0] == plan.cost and res["counters"][1] == cfg.t and res["counters"][3] == 0
        assert_close_to_oracle(res, ref, cfg.dtype, want_dx=True)
        assert_bit_identical(res, full, want_dx=True)


def test_c4_full_size_against_oracle(H):
    """Config 4 as timed (I256 H1024 B32 t4000, float32 storage, three bf16 products per float32
    product) against the fp64 oracle over all 4000 steps, at the float32 tolerance; ISM m = 50
    gives the bits of the full-memory run."""
    cfg = synth.CONFIGS["c4"]
    dp = H.DeviceProblem(cfg)
    full = dp.run(dp.full_memory_plan())
    assert full["counters"][0] == cfg.t and full["counters"][3] == 0 and np.isfinite(full["loss"])
    plan = dp.plan("ism", 50)
    res = dp.run(plan)
    assert res["counters"][0] == plan.cost == P.cost(P.ISM, cfg.t, 50)
    assert res["counters"][1] == cfg.t and res["counters"][2] <= 50 and res["counters"][3] == 0
    assert_bit_identical(res, full)
    ref = oracle_run(dp.prob)
    errs = assert_close_to_oracle(full, ref, "tf32")
    print("c4 t=4000 errors against the oracle:", {k: f"{v:.2e}" for k, v in errs.items()})


def test_c5_shape_across_chunks_against_oracle_with_byte_budget(H):
    """Config 5's widths (two layers, I1024 H2048 B128, bf16) over 40 steps -- more than two staged
    chunks of S = 16 steps, so the per-chunk flush of the weight gradients is crossed twice --
    with general biases and initial state, against the oracle; the budget is given in bytes."""
    from paper_1606_03401_b200 import binding as B
    cfg = _cfg("c5", t=40)
    prob = synth.make_problem(cfg, general=True)
    dp = H.DeviceProblem(cfg, prob, want_dx=True)
    ref = oracle_run(prob)
    full = dp.run(dp.full_memory_plan())
    assert_close_to_oracle(full, ref, "bf16", want_dx=True)
    m = B.mebptt_budget_bytes_to_units(dp.desc, 48 << 20)          # 48 MiB -> 16 units
    assert m == 16
    plan = dp.plan("msm", m, beta=3)
    res = dp.run(plan)
    assert res["counters"][0] == plan.cost == P.cost(P.MSM, cfg.t, m, 4, 3) and res["counters"][2] <= m
    assert_bit_identical(res, full, want_dx=True)


@pytest.mark.parametrize("base,kw,plans", [
    ("c1", dict(t=20), [("hsm", 4), ("msm", 9)]),                                                   # CUDA-core path
    ("c1", dict(t=20, layers=2, cell="gru"), [("msm", 9)]),                                          # CUDA-core path, GRU core
    ("c2", dict(input=128, hidden=256, batch=64, t=70, readout=128), [("hsm", 5), ("msm", 13), ("ism", 70)]),  # persistent tensor path
    ("c5", dict(layers=2, input=64, hidden=72, batch=32, t=45, readout=40), [("msm", 11), ("ism", 45)]),      # step by step, bf16
    ("c4", dict(layers=1, input=64, hidden=128, batch=32, t=45, readout=40), [("msm", 11), ("ism", 45)]),     # step by step, float32 storage
])
def test_launch_count_is_what_the_profiler_sees(H, base, kw, plans):
    """mebptt_lstm_launch_count (the benchmark's gpu_launches) against the kernels CUPTI records for
    one training step (memsets and copies are not kernels and are not counted by either)."""
    import torch
    from torch.profiler import ProfilerActivity, profile
    from paper_1606_03401_b200 import binding as B
    cfg = _cfg(base, **kw)
    dp = H.DeviceProblem(cfg)
    for mode, m in plans:
        plan = dp.plan(mode, m)
        dp.run(plan)
        with profile(activities=[ProfilerActivity.CUDA]) as prof:
            dp.enqueue(plan)
            torch.cuda.synchronize()
        seen = sum(1 for ev in prof.events()
                   if ev.device_type == torch.autograd.DeviceType.CUDA and not ev.name.startswith(("Memset", "Memcpy")))
        assert seen == B.mebptt_lstm_launch_count(dp.desc, plan), (base, mode, m, seen)


def test_prepared_set_is_reused_per_workspace_and_the_enqueue_is_cheap(H):
    """The per-step call looks its prepared set (tape, tensor maps, kernel variants) up instead of
    rebuilding it: one set per (problem, plan, workspace), a new one when the workspace moves, the
    bits of the first call on every later one, and -- at config 3 with the headline budget -- an
    enqueue that takes the host under a quarter of what the step takes the device."""
    import time
    import torch
    from paper_1606_03401_b200 import binding as B
    cfg = synth.CONFIGS["c3"]
    dp = H.DeviceProblem(cfg)
    plan = dp.plan("msm", 100)
    s0 = B.mebptt_lstm_prepare_stats()
    first = dp.run(plan)
    s1 = B.mebptt_lstm_prepare_stats()
    assert s1["built"] == s0["built"] + 1 and s1["page_locked"] == s0["page_locked"] + 1
    again = dp.run(plan)
    s2 = B.mebptt_lstm_prepare_stats()
    assert s2["built"] == s1["built"] and s2["reused"] == s1["reused"] + 1
    assert_bit_identical(again, first)
    # the workspace moves: the tensor maps are made anew, the results stay
    keep = dp._ws
    dp._ws = torch.empty(keep.numel() + 4096, dtype=torch.uint8, device=keep.device)[256:]
    assert dp._ws.data_ptr() != keep.data_ptr()
    moved = dp.run(plan)
    assert B.mebptt_lstm_prepare_stats()["built"] == s2["built"] + 1
    assert_bit_identical(moved, first)
    # host time of an enqueue against device time of the step
    torch.cuda.synchronize()
    host, dev = [], []
    for _ in range(5):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        t0 = time.perf_counter()
        dp.enqueue(plan)
        host.append((time.perf_counter() - t0) * 1e3)
        e1.record()
        torch.cuda.synchronize()
        dev.append(e0.elapsed_time(e1))
    host_ms, dev_ms = sorted(host)[len(host) // 2], sorted(dev)[len(dev) // 2]
    print(f"c3 msm m=100: host enqueue {host_ms:.2f} ms, device {dev_ms:.2f} ms")
    assert host_ms < 0.25 * dev_ms, (host_ms, dev_ms)


@pytest.mark.parametrize("base,kw", [
    ("c2", dict(input=128, hidden=256, batch=64, t=70, readout=128)),                  # persistent tensor path
    ("c5", dict(layers=2, input=64, hidden=128, batch=32, t=45, readout=40)),           # step by step, bf16, two layers
    ("c1", dict(t=24)),                                                                 # float32: sizes 1 : 4 : 3
])
def test_plans_over_the_layouts_byte_sizes_give_the_same_gradients(H, base, kw):
    """BPTT-MSM planned over the real sizes of the layout's states (bfloat16: hidden : internal :
    without input state = 3 : 10 : 7 units) instead of internal states rounded up to whole hidden
    states: forward count equal to the oracle's cost for those sizes, peak within the budget, the
    bits of the full-memory run, and never more forward operations than the rounded plan at the
    same bytes."""
    from paper_1606_03401_b200 import binding as B
    cfg = _cfg(base, **kw)
    dp = H.DeviceProblem(cfg, want_dx=True)
    full = dp.run(dp.full_memory_plan())
    unit = B.mebptt_lstm_unit_bytes(dp.desc)
    for units in (3, 7, 12):
        nbytes = units * unit
        for use_beta in (False, True):
            plan = B.mebptt_plan_bytes_exact(dp.desc, nbytes, use_beta)
            assert plan.cost == P.cost(P.MSM, cfg.t, plan.m, plan.alpha, plan.beta or None, plan.sigma)
            res = dp.run(plan)
            assert res["counters"][0] == plan.cost and res["counters"][1] == cfg.t and res["counters"][3] == 0
            assert res["counters"][2] == plan.peak_units <= plan.m
            assert_bit_identical(res, full, want_dx=True)
            rounded = dp.plan("msm", units, beta=3 if use_beta else 0)
            assert plan.cost <= rounded.cost
    if cfg.dtype == "bf16":
        assert (plan.sigma, plan.alpha, plan.beta) == (3, 10, 7)


@pytest.mark.parametrize("dtype,shape", [("fp32", dict(layers=1, input=32, hidden=64, batch=4, t=40, readout=32)),
                                         ("fp32", dict(layers=2, input=24, hidden=40, batch=6, t=20, readout=10)),
                                         ("bf16", dict(layers=2, input=24, hidden=40, batch=6, t=20, readout=10)),
                                         ("tf32", dict(layers=1, input=70, hidden=65, batch=67, t=9, readout=66))])
def test_gru_core_matches_oracle_and_is_plan_independent(H, dtype, shape):
    """A second recurrent core behind the same plans and tape (Section 1: the method does not depend
    on the architecture of the core): a GRU, with general biases and initial state, against its own
    fp64 oracle per tensor and per block, bit-identical under every kind of plan, forward count equal
    to C(t, m)."""
    cfg = _cfg("c1", dtype=dtype, cell="gru", **shape)
    prob = synth.make_problem(cfg, general=True)
    assert prob["W"][0].shape[0] == 3 * cfg.hidden
    dp = H.DeviceProblem(cfg, prob, want_dx=True)
    ref = oracle_run(prob)
    full = dp.run(dp.full_memory_plan())
    assert full["counters"][0] == cfg.t and full["counters"][1] == cfg.t and full["counters"][3] == 0
    assert_close_to_oracle(full, ref, dtype, want_dx=True)
    for mode, m, beta in [("hsm", 1, 0), ("hsm", 4, 0), ("ism", 2, 0), ("msm", 9, 0), ("msm", 13, 3)]:
        plan = dp.plan(mode, m, beta=beta)
        res = dp.run(plan)
        assert res["counters"][0] == plan.cost and res["counters"][1] == cfg.t and res["counters"][3] == 0
        assert_bit_identical(res, full, want_dx=True)
    # without dx the first layer skips its input-gradient columns; nothing else may change
    nodx = H.DeviceProblem(cfg, prob, want_dx=False)
    assert_bit_identical(nodx.run(nodx.plan("msm", 9)), full)
