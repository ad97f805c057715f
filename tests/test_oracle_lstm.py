"""Pins for oracle.lstm_bptt: finite differences, closed forms, decoupling, autograd."""
import numpy as np
import pytest

from oracle import lstm_bptt as O


def _problem(L, I, H, B, t, Oo, seed=0, scale=0.7):
    r = np.random.default_rng(seed)
    W = [r.uniform(-scale, scale, (4 * H, (I if l == 0 else H) + H)) for l in range(L)]
    b = [r.uniform(-0.3, 0.3, 4 * H) for _ in range(L)]
    return dict(W=W, b=b, W_out=r.uniform(-scale, scale, (Oo, H)), b_out=r.uniform(-0.2, 0.2, Oo),
                x=r.standard_normal((t, B, I)), targets=r.standard_normal((t, B, Oo)),
                h0=r.standard_normal((L, B, H)) * 0.3, c0=r.standard_normal((L, B, H)) * 0.3)


def _fd(p, name, idx, eps=1e-6, layer=None):
    def loss_with(delta):
        q = {k: ([a.copy() for a in v] if isinstance(v, list) else v.copy()) for k, v in p.items()}
        arr = q[name][layer] if layer is not None else q[name]
        arr[idx] += delta
        return O.lstm_loss(**q)
    return (loss_with(eps) - loss_with(-eps)) / (2 * eps)


@pytest.mark.parametrize("L", [1, 2])
def test_finite_differences_every_parameter(L):
    p = _problem(L, 3, 4, 2, 5, 3, seed=L)
    g = O.lstm_bptt(**p)
    assert abs(g["loss"] - O.lstm_loss(**p)) < 1e-12
    checks = 0
    for l in range(L):
        for idx in np.ndindex(p["W"][l].shape):
            fd = _fd(p, "W", idx, layer=l)
            assert abs(fd - g["dW"][l][idx]) <= 1e-6 * max(1.0, abs(fd)), ("W", l, idx)
            checks += 1
        for idx in np.ndindex(p["b"][l].shape):
            fd = _fd(p, "b", idx, layer=l)
            assert abs(fd - g["db"][l][idx]) <= 1e-6 * max(1.0, abs(fd)), ("b", l, idx)
    for name, key in (("W_out", "dW_out"), ("b_out", "db_out"), ("x", "dx")):
        for idx in np.ndindex(p[name].shape):
            fd = _fd(p, name, idx)
            assert abs(fd - g[key][idx]) <= 1e-6 * max(1.0, abs(fd)), (name, idx)
    assert checks > 100


def test_single_step_is_a_feed_forward_net():
    """t = 1: gradient of a one-layer gated unit, written out by hand for one sample."""
    p = _problem(1, 2, 1, 1, 1, 1, seed=3)
    g = O.lstm_bptt(**p)
    W, b = p["W"][0], p["b"][0]
    v = np.concatenate([p["x"][0, 0], p["h0"][0, 0]])
    z = W @ v + b
    s = lambda a: 1 / (1 + np.exp(-a))
    i, f, gg, o = s(z[0]), s(z[1]), np.tanh(z[2]), s(z[3])
    c = f * p["c0"][0, 0, 0] + i * gg
    h = o * np.tanh(c)
    y = p["W_out"][0, 0] * h + p["b_out"][0]
    r = y - p["targets"][0, 0, 0]
    assert np.isclose(g["loss"], r * r)
    dh = 2 * r * p["W_out"][0, 0]
    dc = dh * o * (1 - np.tanh(c) ** 2)
    dz = np.array([dc * gg * i * (1 - i), dc * p["c0"][0, 0, 0] * f * (1 - f),
                   dc * i * (1 - gg ** 2), dh * np.tanh(c) * o * (1 - o)])
    assert np.allclose(g["dW"][0], np.outer(dz, v), rtol=1e-12, atol=1e-15)
    assert np.allclose(g["db"][0], dz, rtol=1e-12)
    assert np.allclose(g["dW_out"], 2 * r * h)
    assert np.allclose(g["db_out"], 2 * r)
    assert np.allclose(g["dx"][0, 0], W[:, :2].T @ dz)


def test_zero_recurrent_weights_decouple_the_steps():
    """With W_hh = 0 and the forget path cut, the gradient is a sum of one-step gradients."""
    I, H, B, t, Oo = 3, 4, 2, 6, 2
    p = _problem(1, I, H, B, t, Oo, seed=5)
    p["W"][0][:, I:] = 0.0
    p["b"][0][H:2 * H] = -800.0           # f = 0 exactly in float64: c_{t-1} has no effect
    p["h0"][:] = 0
    p["c0"][:] = 0
    np.seterr(over="ignore")               # exp(800) -> inf -> sigmoid = 0, as intended
    g = O.lstm_bptt(**p)
    dW = np.zeros_like(p["W"][0]); db = np.zeros_like(p["b"][0])
    dWo = np.zeros_like(p["W_out"]); loss = 0.0
    for k in range(t):
        q = dict(p, x=p["x"][k:k + 1], targets=p["targets"][k:k + 1])
        gk = O.lstm_bptt(**q)
        dW += gk["dW"][0]; db += gk["db"][0]; dWo += gk["dW_out"]; loss += gk["loss"]
    assert np.isclose(g["loss"], loss, rtol=1e-13)
    assert np.allclose(g["dW"][0][:, :I], dW[:, :I], rtol=1e-12, atol=1e-15)
    assert np.allclose(g["db"][0], db, rtol=1e-12, atol=1e-15)
    assert np.allclose(g["dW_out"], dWo, rtol=1e-12, atol=1e-15)


@pytest.mark.parametrize("L", [1, 2])
def test_against_torch_autograd_float64(L):
    torch = pytest.importorskip("torch")
    I, H, B, t, Oo = 5, 7, 3, 9, 4
    p = _problem(L, I, H, B, t, Oo, seed=11 + L)
    g = O.lstm_bptt(**p)
    lstm = torch.nn.LSTM(I, H, num_layers=L).double()
    with torch.no_grad():
        for l in range(L):
            I_l = I if l == 0 else H
            getattr(lstm, f"weight_ih_l{l}").copy_(torch.from_numpy(p["W"][l][:, :I_l]))
            getattr(lstm, f"weight_hh_l{l}").copy_(torch.from_numpy(p["W"][l][:, I_l:]))
            getattr(lstm, f"bias_ih_l{l}").copy_(torch.from_numpy(p["b"][l]))
            getattr(lstm, f"bias_hh_l{l}").zero_()
    W_out = torch.from_numpy(p["W_out"]).requires_grad_()
    b_out = torch.from_numpy(p["b_out"]).requires_grad_()
    x = torch.from_numpy(p["x"]).requires_grad_()
    out, _ = lstm(x, (torch.from_numpy(p["h0"]), torch.from_numpy(p["c0"])))
    y = out @ W_out.T + b_out
    loss = ((y - torch.from_numpy(p["targets"])) ** 2).sum() / (B * Oo)
    loss.backward()
    assert np.isclose(g["loss"], loss.item(), rtol=1e-12)
    for l in range(L):
        I_l = I if l == 0 else H
        assert np.allclose(g["dW"][l][:, :I_l], getattr(lstm, f"weight_ih_l{l}").grad.numpy(), rtol=1e-9, atol=1e-12)
        assert np.allclose(g["dW"][l][:, I_l:], getattr(lstm, f"weight_hh_l{l}").grad.numpy(), rtol=1e-9, atol=1e-12)
        assert np.allclose(g["db"][l], getattr(lstm, f"bias_ih_l{l}").grad.numpy(), rtol=1e-9, atol=1e-12)
    assert np.allclose(g["dW_out"], W_out.grad.numpy(), rtol=1e-9, atol=1e-12)
    assert np.allclose(g["db_out"], b_out.grad.numpy(), rtol=1e-9, atol=1e-12)
    assert np.allclose(g["dx"], x.grad.numpy(), rtol=1e-9, atol=1e-12)


def test_synthetic_problem_is_seeded_and_representable():
    from paper_1606_03401_b200 import synth
    cfg = synth.with_overrides(synth.CONFIGS["c2"], t=3, batch=2, hidden=8, input=8, readout=8)
    a, b = synth.make_problem(cfg), synth.make_problem(cfg)
    assert all(np.array_equal(a["W"][0], b["W"][0]) for _ in [0])
    assert np.array_equal(a["x"], b["x"])
    assert np.array_equal(synth.round_to_bf16(a["x"]), a["x"])
    assert np.array_equal(synth.round_to_bf16(a["W"][0]), a["W"][0])
    assert np.all(a["b"][0][8:16] == 1.0) and a["b"][0].sum() == 8.0
    assert np.all(np.abs(a["W"][0]) <= 1 / np.sqrt(8))
    # bf16 round-to-nearest-even on a hand-made case: 1 + 2^-8 is a tie -> rounds to 1.0
    assert synth.round_to_bf16(np.array([1.0 + 2.0 ** -8]))[0] == 1.0
    assert synth.round_to_bf16(np.array([1.0 + 3 * 2.0 ** -8]))[0] == 1.0 + 2.0 ** -6
    d = synth.to_device_arrays(cfg, a)
    assert d["W"].dtype == np.uint16 and d["targets"].dtype == np.float32


def test_general_problem_keeps_the_plain_draws_and_adds_distinguishing_values():
    from paper_1606_03401_b200 import synth
    cfg = synth.with_overrides(synth.CONFIGS["c2"], t=3, batch=2, hidden=8, input=8, readout=8, layers=2)
    a, g = synth.make_problem(cfg), synth.make_problem(cfg, general=True)
    for k in ("W_out", "x", "targets"):
        assert np.array_equal(a[k], g[k])
    assert all(np.array_equal(u, v) for u, v in zip(a["W"], g["W"]))
    for l in range(2):
        d = g["b"][l] - a["b"][l]
        assert np.all(np.abs(d) <= 0.3 + 1e-6) and len(np.unique(g["b"][l])) == 32
    assert len(np.unique(g["b_out"])) == 8 and np.all(np.abs(g["b_out"]) <= 0.3 + 1e-6)
    assert np.array_equal(synth.round_to_bf16(g["h0"]), g["h0"]) and np.abs(g["h0"]).max() > 0
    assert np.array_equal(synth.round_to_fp32(g["c0"]), g["c0"]) and np.abs(g["c0"]).max() > 0


def test_block_check_catches_what_the_whole_tensor_norm_lets_through():
    """The parity helper compares block by block: one wrong 128 x 128 tile, one wrong gate row
    block entry or one wrong group of bias entries, planted in a copy of the oracle's result, stays
    far below the whole-tensor tolerance and must still be refused."""
    import pytest
    from tests.util import assert_close_to_oracle, flat_oracle
    r = np.random.default_rng(5)
    H, K, O, t, B, I = 256, 768, 128, 6, 4, 128
    ref = {"loss": 1.0, "dW": [r.standard_normal((4 * H, K))], "db": [r.standard_normal(4 * H)],
           "dW_out": r.standard_normal((O, H)), "db_out": r.standard_normal(O), "dx": r.standard_normal((t, B, I))}

    def result():
        fo = flat_oracle(ref)
        return {"loss": 1.0, **{k: v.copy() for k, v in fo.items()}}

    assert_close_to_oracle(result(), ref, "bf16", want_dx=True)
    for key, plant in [
        ("dW", lambda a: a.reshape(4 * H, K).__setitem__((slice(128, 256), slice(256, 384)), 0.0)),       # a lost tile
        ("db", lambda a: a.__setitem__(slice(512, 544), a[512:544] * 1.5)),                              # 32 entries off
        ("dW_out", lambda a: a.reshape(O, H).__setitem__((slice(0, 128), slice(128, 256)),
                                                         a.reshape(O, H)[0:128, 0:128])),                # a misplaced tile
        ("db_out", lambda a: a.__setitem__(slice(96, 128), 0.0)),                                        # dropped entries
        ("dx", lambda a: a.reshape(t, B, I).__setitem__(0, 0.0)),                                        # a missing step
    ]:
        res = result()
        plant(res[key])
        with pytest.raises(AssertionError):
            assert_close_to_oracle(res, ref, "bf16", want_dx=True)
    # a dW tile that is 12 % off is under the whole-tensor tolerance at this size: only the block check sees it
    res = result()
    res["dW"].reshape(4 * H, K)[128:256, 256:384] *= 0.88
    from tests.util import rel_l2
    assert rel_l2(res["dW"], flat_oracle(ref)["dW"]) < 2e-2
    with pytest.raises(AssertionError):
        assert_close_to_oracle(res, ref, "bf16", want_dx=True)
