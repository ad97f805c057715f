"""GPU: the allocation-free training step against the ordinary one.

Some users of the library run where device memory can no longer be allocated (all of it has
been promised elsewhere, or their host application only lends them input and output buffers).
They call mebptt_lstm_train_step_static, whose workspace is an array built into the library.
This file checks, through the C interface, that it returns exactly what the ordinary entry
point returns -- twice in a row, because the second call starts from the first one's leftovers
in the shared array -- and that it refuses problems that do not fit.  The file name sorts last
on purpose: a run that stops at the first failure has then already run everything else.
"""
import numpy as np
import pytest

from paper_1606_03401_b200 import synth
from tests.util import assert_bit_identical

pytestmark = pytest.mark.gpu


def _static_run(dp, plan):
    import torch
    from paper_1606_03401_b200 import binding as B
    d, o = dp.dev, dp.out
    for v in o.values():
        if v is not None:
            v.fill_(7)            # results must be overwritten, not inherited from the other call
    B.mebptt_lstm_train_step_static(dp.desc, plan, d["W"], d["b"], d["W_out"], d["b_out"], d["x"], d["targets"],
                                    d["h0"], d["c0"], torch.cuda.current_stream().cuda_stream, o["loss"],
                                    o["dW"], o["db"], o["dW_out"], o["db_out"], o["dx"], o["counters"])
    torch.cuda.synchronize()
    res = {k: (v.cpu().numpy().copy() if v is not None else None) for k, v in o.items()}
    res["loss"] = float(res["loss"][0])
    return res


@pytest.mark.parametrize("base,kw,mode,m", [
    ("c1", dict(), "hsm", 8),                                                      # fp32, CUDA-core kernels
    ("c2", dict(input=64, hidden=128, batch=32, t=40, readout=64), "msm", 9),      # bf16, tensor-core kernels
])
def test_static_workspace_step_matches_ordinary_step_twice(base, kw, mode, m):
    from paper_1606_03401_b200 import binding as B
    from paper_1606_03401_b200 import harness
    cfg = synth.with_overrides(synth.CONFIGS[base], **kw)
    dp = harness.DeviceProblem(cfg, want_dx=True)
    plan = dp.plan(mode, m)
    assert B.mebptt_lstm_workspace_bytes(dp.desc, plan) <= B.MEBPTT_STATIC_WORKSPACE_BYTES
    import torch
    want = dp.run(plan)                      # ordinary entry point, caller-owned workspace
    first = _static_run(dp, plan)            # the set-up call of this device, if no earlier test made it
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    second = _static_run(dp, plan)           # same array, previous contents still in it
    torch.cuda.synchronize()
    # nothing was reserved by the later call: the driver reports the same free memory (torch's own
    # caching allocator serves the result copies from host memory and blocks it already holds)
    assert torch.cuda.mem_get_info()[0] >= free_before
    for got in (first, second):
        assert got["counters"][0] == plan.cost and got["counters"][1] == cfg.t and got["counters"][3] == 0
        assert_bit_identical(got, want, want_dx=True)
    # a different plan afterwards, again on the shared array
    other = dp.full_memory_plan()
    if B.mebptt_lstm_workspace_bytes(dp.desc, other) <= B.MEBPTT_STATIC_WORKSPACE_BYTES:
        assert_bit_identical(_static_run(dp, other), want, want_dx=True)


def test_static_workspace_step_refuses_per_launch_timing():
    """Timing every launch creates CUDA events on demand, which the allocation-free call must not."""
    from paper_1606_03401_b200 import binding as B
    desc = B.make_desc(1, 64, 128, 64, 32, 40, "bf16", flags=B.MEBPTT_FLAG_TIME_RUNS)
    plan = B.mebptt_plan(40, 9, B.MEBPTT_MSM)
    dummy = np.zeros(8, np.float32)
    with pytest.raises(B.MebpttError) as e:
        B.mebptt_lstm_train_step_static(desc, plan, dummy, dummy, dummy, dummy, dummy, dummy, dummy, dummy, None,
                                        dummy, dummy, dummy, dummy, dummy, None, dummy)
    assert e.value.status == B.MEBPTT_ERR_ARG


def test_static_workspace_step_refuses_what_does_not_fit():
    from paper_1606_03401_b200 import binding as B
    desc = B.make_desc(1, 1024, 1024, 1024, 64, 1000, "bf16")
    plan = B.mebptt_plan(1000, 100, B.MEBPTT_MSM)
    assert B.mebptt_lstm_workspace_bytes(desc, plan) > B.MEBPTT_STATIC_WORKSPACE_BYTES
    dummy = np.zeros(8, np.float32)
    with pytest.raises(B.MebpttError) as e:
        B.mebptt_lstm_train_step_static(desc, plan, dummy, dummy, dummy, dummy, dummy, dummy, dummy, dummy, None,
                                        dummy, dummy, dummy, dummy, dummy, None, dummy)
    assert e.value.status == B.MEBPTT_ERR_WORKSPACE
