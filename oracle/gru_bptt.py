"""Oracle: standard full-memory BPTT (Section 2.1) of a stacked GRU, in float64.

Test infrastructure only.  Section 1 of the paper calls its method largely independent of the
architecture of the recurrent core; the second core this repository runs behind the same plans
is the gated recurrent unit in the form in which the reset gate multiplies the product with the
recurrent weights.  With W = [W_r ; W_z ; W_n] (three blocks of H rows over the columns
[x_t ; h_{t-1}], the first I of them W_x., the other H of them W_h.) and one bias per gate row:

    r = sigmoid(W_xr x_t + W_hr h_{t-1} + b_r)
    z = sigmoid(W_xz x_t + W_hz h_{t-1} + b_z)
    q = W_hn h_{t-1}
    n = tanh(W_xn x_t + b_n + r * q)
    h_t = (1 - z) * n + z * h_{t-1}

The hidden state in the sense of Definition 2 is h_t alone.  Layers are stacked by feeding h_t of
layer l as the input of layer l + 1 at the same time step; the readout and the loss are those of
``oracle.lstm_bptt``:  y_t = W_out h_t + b_out,  L = sum_t mean_{b,o} (y_t - target_t)^2.

Shapes: x [t, B, I], targets [t, B, O], W[l] [3H, I_l + H] (I_0 = I, I_l = H), b[l] [3H],
W_out [O, H], b_out [O], h0 [L, B, H].  Matrix products use numpy's ``@``; nothing is blocked,
fused or reordered.
"""
from __future__ import annotations

import numpy as np


def _sigmoid(a):
    return 1.0 / (1.0 + np.exp(-a))


def gru_forward(W, b, x, h0):
    """All forward steps; returns hs [L, t + 1, B, H] and the stored r, z, n, q [L, t + 1, 4, B, H]."""
    L = len(W)
    t, B, _ = x.shape
    H = W[0].shape[0] // 3
    hs = np.zeros((L, t + 1, B, H), np.float64)
    gates = np.zeros((L, t + 1, 4, B, H), np.float64)
    hs[:, 0] = h0
    for k in range(1, t + 1):
        inp = x[k - 1]
        for l in range(L):
            I_l = inp.shape[1]
            Wx, Wh = W[l][:, :I_l], W[l][:, I_l:]
            hp = hs[l, k - 1]
            ax = inp @ Wx.T + b[l]                  # [B, 3H]: input part and bias of every gate
            ah = hp @ Wh.T                          # [B, 3H]: recurrent part of every gate
            r = _sigmoid(ax[:, 0:H] + ah[:, 0:H])
            z = _sigmoid(ax[:, H:2 * H] + ah[:, H:2 * H])
            q = ah[:, 2 * H:3 * H]
            n = np.tanh(ax[:, 2 * H:3 * H] + r * q)
            h = (1.0 - z) * n + z * hp
            gates[l, k] = (r, z, n, q)
            hs[l, k] = h
            inp = h
    return hs, gates


def gru_bptt(W, b, W_out, b_out, x, targets, h0):
    """Loss and gradients by full-memory BPTT.

    Returns a dict: loss, loss_t [t], dW (list), db (list), dW_out, db_out, dx [t, B, I].
    """
    f64 = np.float64
    W = [np.asarray(w, f64) for w in W]
    b = [np.asarray(v, f64) for v in b]
    W_out = np.asarray(W_out, f64)
    b_out = np.asarray(b_out, f64)
    x = np.asarray(x, f64)
    targets = np.asarray(targets, f64)
    L = len(W)
    t, B, I = x.shape
    H = W[0].shape[0] // 3
    O = W_out.shape[0]
    h0 = np.asarray(h0, f64).reshape(L, B, H)

    hs, gates = gru_forward(W, b, x, h0)

    dW = [np.zeros_like(w) for w in W]
    db = [np.zeros_like(v) for v in b]
    dW_out = np.zeros_like(W_out)
    db_out = np.zeros_like(b_out)
    dx = np.zeros_like(x)
    loss_t = np.zeros(t, f64)

    dh_next = np.zeros((L, B, H), f64)   # gradient w.r.t. h_k arriving from step k + 1
    for k in range(t, 0, -1):
        y = hs[L - 1, k] @ W_out.T + b_out
        diff = y - targets[k - 1]
        loss_t[k - 1] = np.sum(diff * diff) / (B * O)
        dy = 2.0 * diff / (B * O)
        dW_out += dy.T @ hs[L - 1, k]
        db_out += dy.sum(axis=0)
        d_from_above = dy @ W_out
        for l in range(L - 1, -1, -1):
            r, z, n, q = gates[l, k]
            hp = hs[l, k - 1]
            inp = x[k - 1] if l == 0 else hs[l - 1, k]
            I_l = inp.shape[1]
            dh = d_from_above + dh_next[l]
            dn = dh * (1.0 - z)
            dz = dh * (hp - n)
            dn_pre = dn * (1.0 - n * n)
            dr = dn_pre * q
            dq = dn_pre * r
            dr_pre = dr * r * (1.0 - r)
            dz_pre = dz * z * (1.0 - z)
            d_ax = np.concatenate([dr_pre, dz_pre, dn_pre], axis=1)   # w.r.t. the input parts (and the biases)
            d_ah = np.concatenate([dr_pre, dz_pre, dq], axis=1)       # w.r.t. the recurrent parts
            dW[l][:, :I_l] += d_ax.T @ inp
            dW[l][:, I_l:] += d_ah.T @ hp
            db[l] += d_ax.sum(axis=0)
            d_inp = d_ax @ W[l][:, :I_l]
            dh_next[l] = d_ah @ W[l][:, I_l:] + dh * z
            if l == 0:
                dx[k - 1] = d_inp
            else:
                d_from_above = d_inp
    return {"loss": float(loss_t.sum()), "loss_t": loss_t, "dW": dW, "db": db, "dW_out": dW_out,
            "db_out": db_out, "dx": dx}


def gru_loss(W, b, W_out, b_out, x, targets, h0) -> float:
    """Forward pass and loss only (used by finite-difference checks)."""
    f64 = np.float64
    W = [np.asarray(w, f64) for w in W]
    b = [np.asarray(v, f64) for v in b]
    x = np.asarray(x, f64)
    L = len(W)
    t, B, _ = x.shape
    H = W[0].shape[0] // 3
    O = np.asarray(W_out).shape[0]
    hs, _ = gru_forward(W, b, x, np.asarray(h0, f64).reshape(L, B, H))
    total = 0.0
    for k in range(1, t + 1):
        y = hs[L - 1, k] @ np.asarray(W_out, f64).T + np.asarray(b_out, f64)
        diff = y - np.asarray(targets, f64)[k - 1]
        total += np.sum(diff * diff) / (B * O)
    return float(total)
