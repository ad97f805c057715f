"""GPU: the bounded waits of the tensor-core kernels, made to run out on purpose.

Every wait of those kernels (on a grid-wide step counter, on a barrier that TMA copies complete)
gives up after a bounded number of polls, writes MEBPTT_ERR_TIMEOUT to the status word and lets
the kernel end through its ordinary exit path.  Nothing faults or hangs here: the testing aid
mebptt_test_wait_fault only makes a wait expect something that never comes (one signal more than
there are CTAs, 16 bytes more than the copies bring), with a poll limit of a few thousand.  After
each case the same process runs an ordinary step, which must come out clean.
"""
import numpy as np
import pytest

from paper_1606_03401_b200 import synth
from tests.util import assert_bit_identical

pytestmark = pytest.mark.gpu


@pytest.fixture()
def fault():
    from paper_1606_03401_b200 import binding as B
    yield B.mebptt_test_wait_fault
    B.mebptt_test_wait_fault(0)


@pytest.mark.parametrize("bit,what", [(1, "forward run kernel"), (2, "backward run kernel")])
def test_step_counter_wait_runs_out_and_reports_timeout(fault, bit, what):
    from paper_1606_03401_b200 import binding as B
    from paper_1606_03401_b200 import harness
    cfg = synth.with_overrides(synth.CONFIGS["c2"], t=12)
    dp = harness.DeviceProblem(cfg)
    plan = dp.full_memory_plan()
    clean = dp.run(plan)
    assert clean["counters"][3] == 0
    fault(bit)
    res = dp.run(plan)                       # returns: the waits give up, the kernels end
    assert res["counters"][3] == B.MEBPTT_ERR_TIMEOUT, what
    fault(0)
    again = dp.run(plan)
    assert again["counters"][3] == 0 and again["counters"][0] == cfg.t and again["counters"][1] == cfg.t
    assert_bit_identical(again, clean)


def test_gemm_pipeline_wait_runs_out_and_reports_timeout(fault):
    import torch
    from paper_1606_03401_b200 import binding as B
    M, N, K = 128, 128, 256
    g = torch.Generator(device="cuda:0").manual_seed(3)
    A = torch.randn(M, K, device="cuda:0", generator=g).to(torch.bfloat16)
    Bm = torch.randn(N, K, device="cuda:0", generator=g).to(torch.bfloat16)
    C = torch.zeros(M, N, device="cuda:0")
    status = torch.zeros(1, dtype=torch.int32, device="cuda:0")
    s = torch.cuda.current_stream().cuda_stream
    fault(4)
    B.mebptt_gemm_bf16(A, K, 0, Bm, K, 0, C, N, 0, None, M, N, K, status, s)
    torch.cuda.synchronize()
    assert int(status.item()) == B.MEBPTT_ERR_TIMEOUT
    fault(0)
    status.zero_()
    B.mebptt_gemm_bf16(A, K, 0, Bm, K, 0, C, N, 0, None, M, N, K, status, s)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    want = A.float() @ Bm.float().T
    assert torch.allclose(C, want, rtol=1e-3, atol=1e-2)
