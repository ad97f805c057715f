"""Pins of the GRU oracle (oracle/gru_bptt.py): finite differences on every parameter, torch
autograd in float64, a hand-written single step, and the saturated update gate, where the state
never changes and the gradient has a closed form."""
import numpy as np
import pytest

from oracle import gru_bptt as G


def _problem(L, I, H, B, t, O, seed=0):
    r = np.random.default_rng(seed)
    lim = 1 / np.sqrt(H)
    W = [r.uniform(-lim, lim, size=(3 * H, (I if l == 0 else H) + H)) for l in range(L)]
    b = [r.uniform(-0.3, 0.3, size=3 * H) for _ in range(L)]
    return dict(W=W, b=b, W_out=r.uniform(-lim, lim, size=(O, H)), b_out=r.uniform(-0.3, 0.3, size=O),
                x=r.standard_normal((t, B, I)), targets=r.standard_normal((t, B, O)),
                h0=0.5 * r.standard_normal((L, B, H)))


def _args(p):
    return (p["W"], p["b"], p["W_out"], p["b_out"], p["x"], p["targets"], p["h0"])


@pytest.mark.parametrize("L", [1, 2])
def test_finite_differences_on_every_parameter(L):
    p = _problem(L, 3, 4, 2, 5, 3, seed=L)
    g = G.gru_bptt(*_args(p))
    eps = 1e-6

    def check(arr, grad):
        flat, gflat = arr.reshape(-1), np.asarray(grad).reshape(-1)
        for i in range(flat.size):
            old = flat[i]
            flat[i] = old + eps
            up = G.gru_loss(*_args(p))
            flat[i] = old - eps
            dn = G.gru_loss(*_args(p))
            flat[i] = old
            num = (up - dn) / (2 * eps)
            assert abs(num - gflat[i]) <= 1e-6 * max(1.0, abs(num)), (i, num, gflat[i])

    for l in range(L):
        check(p["W"][l], g["dW"][l])
        check(p["b"][l], g["db"][l])
    check(p["W_out"], g["dW_out"])
    check(p["b_out"], g["db_out"])
    check(p["x"], g["dx"])
    assert np.isclose(g["loss"], G.gru_loss(*_args(p)), rtol=1e-13)


def test_matches_torch_autograd_in_float64():
    import torch
    L, I, H, B, t, O = 2, 5, 6, 3, 7, 4
    p = _problem(L, I, H, B, t, O, seed=7)
    g = G.gru_bptt(*_args(p))
    gru = torch.nn.GRU(I, H, num_layers=L).double()
    with torch.no_grad():
        for l in range(L):
            I_l = I if l == 0 else H
            getattr(gru, f"weight_ih_l{l}").copy_(torch.from_numpy(p["W"][l][:, :I_l]))
            getattr(gru, f"weight_hh_l{l}").copy_(torch.from_numpy(p["W"][l][:, I_l:]))
            getattr(gru, f"bias_ih_l{l}").copy_(torch.from_numpy(p["b"][l]))
            getattr(gru, f"bias_hh_l{l}").zero_()      # one bias per gate row: the recurrent one is zero
    W_out = torch.from_numpy(p["W_out"]).requires_grad_()
    b_out = torch.from_numpy(p["b_out"]).requires_grad_()
    x = torch.from_numpy(p["x"]).requires_grad_()
    out, _ = gru(x, torch.from_numpy(p["h0"]))
    y = out @ W_out.T + b_out
    loss = ((y - torch.from_numpy(p["targets"])) ** 2).sum() / (B * O)
    loss.backward()
    assert np.isclose(g["loss"], loss.item(), rtol=1e-12)
    for l in range(L):
        I_l = I if l == 0 else H
        assert np.allclose(g["dW"][l][:, :I_l], getattr(gru, f"weight_ih_l{l}").grad.numpy(), rtol=1e-9, atol=1e-12)
        assert np.allclose(g["dW"][l][:, I_l:], getattr(gru, f"weight_hh_l{l}").grad.numpy(), rtol=1e-9, atol=1e-12)
        assert np.allclose(g["db"][l], getattr(gru, f"bias_ih_l{l}").grad.numpy(), rtol=1e-9, atol=1e-12)
    assert np.allclose(g["dW_out"], W_out.grad.numpy(), rtol=1e-9, atol=1e-12)
    assert np.allclose(g["db_out"], b_out.grad.numpy(), rtol=1e-9, atol=1e-12)
    assert np.allclose(g["dx"], x.grad.numpy(), rtol=1e-9, atol=1e-12)


def test_single_step_by_hand():
    """t = 1, B = 1, H = 1, I = 1: the chain rule written out by hand."""
    wxr, whr, wxz, whz, wxn, whn = 0.3, -0.2, 0.5, 0.1, -0.4, 0.7
    br, bz, bn = 0.05, -0.1, 0.2
    wo, bo, x, h0, tau = 1.5, 0.1, 0.8, -0.6, 0.25
    sig = lambda a: 1 / (1 + np.exp(-a))
    r, z = sig(wxr * x + whr * h0 + br), sig(wxz * x + whz * h0 + bz)
    q = whn * h0
    n = np.tanh(wxn * x + bn + r * q)
    h = (1 - z) * n + z * h0
    y = wo * h + bo
    dy = 2 * (y - tau)
    dh = dy * wo
    dn_pre = dh * (1 - z) * (1 - n * n)
    dz_pre = dh * (h0 - n) * z * (1 - z)
    dr_pre = dn_pre * q * r * (1 - r)
    W = [np.array([[wxr, whr], [wxz, whz], [wxn, whn]])]
    g = G.gru_bptt(W, [np.array([br, bz, bn])], np.array([[wo]]), np.array([bo]), np.array([[[x]]]),
                   np.array([[[tau]]]), np.array([[[h0]]]))
    assert np.isclose(g["loss"], (y - tau) ** 2)
    want = np.array([[dr_pre * x, dr_pre * h0], [dz_pre * x, dz_pre * h0], [dn_pre * x, dn_pre * r * h0]])
    assert np.allclose(g["dW"][0], want, rtol=1e-12)
    assert np.allclose(g["db"][0], [dr_pre, dz_pre, dn_pre], rtol=1e-12)
    assert np.isclose(g["dx"][0, 0, 0], dr_pre * wxr + dz_pre * wxz + dn_pre * wxn)
    assert np.isclose(g["dW_out"][0, 0], dy * h) and np.isclose(g["db_out"][0], dy)


def test_saturated_update_gate_copies_the_state():
    """With the update gate's bias at +40, z is 1 to the last bit in float64: h_t = h_0 for every t,
    the loss is that of a constant readout, nothing reaches the recurrent parameters, and
    dW_out = sum_t dy_t^T h_0."""
    L, I, H, B, t, O = 1, 3, 4, 2, 6, 3
    p = _problem(L, I, H, B, t, O, seed=3)
    p["b"][0][H:2 * H] = 40.0
    g = G.gru_bptt(*_args(p))
    y = p["h0"][0] @ p["W_out"].T + p["b_out"]
    diffs = y[None] - p["targets"]
    assert np.isclose(g["loss"], np.sum(diffs ** 2) / (B * O), rtol=1e-13)
    dy = 2 * diffs / (B * O)
    assert np.allclose(g["dW_out"], np.einsum("tbo,bh->oh", dy, p["h0"][0]), rtol=1e-12)
    assert np.all(g["dW"][0] == 0) and np.all(g["db"][0] == 0) and np.all(g["dx"] == 0)
