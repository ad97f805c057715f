"""GPU: the tensor-core contraction against its plain definition in float64."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu


def _bf16(a):
    from paper_1606_03401_b200 import synth
    return synth.round_to_bf16(a)


def _run(M, N, K, a_mn, b_mn, accumulate=False, bias=False, seed=0, pad=0):
    import torch
    from paper_1606_03401_b200 import binding as B
    from paper_1606_03401_b200.harness import _upload
    from paper_1606_03401_b200 import synth
    r = np.random.default_rng(seed)
    A = _bf16(r.standard_normal((M, K)))
    Bm = _bf16(r.standard_normal((N, K)))
    C0 = r.standard_normal((M, N)).astype(np.float32)
    bv = r.standard_normal(N).astype(np.float32)
    # storage: [m][k] with row stride lda, or [k][m]
    def store(X, mn):
        Y = X.T if mn else X
        rows, cols = Y.shape
        ld = (cols + 7) // 8 * 8 + pad
        buf = np.zeros((rows, ld))
        buf[:, :cols] = Y
        return synth.bf16_bits(buf), ld
    Ab, lda = store(A, a_mn)
    Bb, ldb = store(Bm, b_mn)
    dA, dB = _upload(Ab, "cuda:0"), _upload(Bb, "cuda:0")
    dC = torch.from_numpy(C0.copy()).cuda()
    dbias = torch.from_numpy(bv).cuda() if bias else None
    status = torch.zeros(1, dtype=torch.int32, device="cuda:0")
    B.mebptt_gemm_bf16(dA, lda, int(a_mn), dB, ldb, int(b_mn), dC, N, accumulate, dbias, M, N, K, status,
                       torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ref = A @ Bm.T + (bv if bias else 0.0) + (C0 if accumulate else 0.0)
    got = dC.cpu().numpy().astype(np.float64)
    err = np.abs(got - ref).max() / max(1.0, np.abs(ref).max())
    return err


@pytest.mark.parametrize("a_mn,b_mn", [(False, False), (True, True), (True, False), (False, True)])
@pytest.mark.parametrize("M,N,K", [(128, 128, 64), (256, 384, 512), (100, 72, 40), (1, 8, 8), (333, 129, 1000)])
def test_gemm_matches_definition(M, N, K, a_mn, b_mn):
    assert _run(M, N, K, a_mn, b_mn) < 2e-6 * np.sqrt(K) + 1e-6


def test_gemm_accumulate_bias_and_strides():
    assert _run(200, 136, 192, False, False, accumulate=True, bias=True, pad=8) < 1e-4
    assert _run(200, 136, 192, True, True, accumulate=True, pad=16) < 1e-4


def test_gemm_training_shapes():
    # input projection of 16 steps at config 3, and a weight-gradient chunk
    assert _run(1024, 4096, 1024, False, False, bias=True) < 1e-4
    assert _run(4096, 2048, 1024, True, True, accumulate=True) < 1e-4


def test_gemm_short_and_wide_shapes():
    # a short backward run at config 3: readout of one and two steps, pre-activations of two leaves
    # (these take the 32-wide tiles)
    assert _run(64, 1024, 1024, False, False, bias=True) < 1e-4
    assert _run(128, 1024, 1024, False, False) < 1e-4
    assert _run(128, 4096, 1024, False, False, accumulate=True) < 1e-4
    assert _run(40, 264, 200, False, False, accumulate=True, bias=True, pad=8) < 1e-4
