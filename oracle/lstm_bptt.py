"""Oracle: standard full-memory BPTT (Section 2.1) of a stacked LSTM, in float64.

Test infrastructure only.  Every memory-saving policy of the paper reorders and repeats forward
operations but reaches the gradient of ordinary BPTT, so the gradient oracle is ordinary BPTT
written out: run all ``t`` forward steps keeping every internal state, then walk back from
step ``t`` to step 1.

The paper uses "an LSTM" (Section 4) without printing its equations; the standard cell
without peepholes is taken.  With ``z = W [x_t ; h_{t-1}] + b`` split into four blocks of H
rows in the order i, f, g, o:

    i = sigmoid(z_i)  f = sigmoid(z_f)  g = tanh(z_g)  o = sigmoid(z_o)
    c_t = f * c_{t-1} + i * g          h_t = o * tanh(c_t)

The hidden state in the sense of Definition 2 is the pair (h_t, c_t).  Layers are stacked by
feeding h_t of layer l as the input of layer l + 1 at the same time step; the RNN core of
Definition 1 is the whole stack at one time step.  On top sits a linear readout of the last
layer, ``y_t = W_out h_t + b_out``, and the loss is a sum of per-step terms

    L = sum_t  (1 / (B * O)) * sum_{b, o} (y_t[b, o] - target_t[b, o])^2 .

Shapes: x [t, B, I], targets [t, B, O], W[l] [4H, I_l + H] (I_0 = I, I_l = H), b[l] [4H],
W_out [O, H], b_out [O], h0 / c0 [L, B, H].  Matrix products use numpy's ``@``; nothing is
blocked, fused or reordered.
"""
from __future__ import annotations

import numpy as np


def _sigmoid(a):
    return 1.0 / (1.0 + np.exp(-a))


def lstm_forward(W, b, x, h0, c0):
    """All forward steps; returns per-layer lists of the stored internal states."""
    L = len(W)
    t, B, _ = x.shape
    H = W[0].shape[0] // 4
    f64 = np.float64
    hs = np.zeros((L, t + 1, B, H), f64)
    cs = np.zeros((L, t + 1, B, H), f64)
    gates = np.zeros((L, t + 1, 4, B, H), f64)
    hs[:, 0] = h0
    cs[:, 0] = c0
    for k in range(1, t + 1):
        inp = x[k - 1]
        for l in range(L):
            z = np.concatenate([inp, hs[l, k - 1]], axis=1) @ W[l].T + b[l]
            i = _sigmoid(z[:, 0 * H:1 * H])
            f = _sigmoid(z[:, 1 * H:2 * H])
            g = np.tanh(z[:, 2 * H:3 * H])
            o = _sigmoid(z[:, 3 * H:4 * H])
            c = f * cs[l, k - 1] + i * g
            h = o * np.tanh(c)
            gates[l, k] = (i, f, g, o)
            cs[l, k] = c
            hs[l, k] = h
            inp = h
    return hs, cs, gates


def lstm_bptt(W, b, W_out, b_out, x, targets, h0, c0):
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
    H = W[0].shape[0] // 4
    O = W_out.shape[0]
    h0 = np.asarray(h0, f64).reshape(L, B, H)
    c0 = np.asarray(c0, f64).reshape(L, B, H)

    hs, cs, gates = lstm_forward(W, b, x, h0, c0)

    dW = [np.zeros_like(w) for w in W]
    db = [np.zeros_like(v) for v in b]
    dW_out = np.zeros_like(W_out)
    db_out = np.zeros_like(b_out)
    dx = np.zeros_like(x)
    loss_t = np.zeros(t, f64)

    dh_next = np.zeros((L, B, H), f64)   # gradient w.r.t. h_k arriving from step k + 1
    dc_next = np.zeros((L, B, H), f64)
    for k in range(t, 0, -1):
        # readout and its loss term at step k
        y = hs[L - 1, k] @ W_out.T + b_out
        diff = y - targets[k - 1]
        loss_t[k - 1] = np.sum(diff * diff) / (B * O)
        dy = 2.0 * diff / (B * O)
        dW_out += dy.T @ hs[L - 1, k]
        db_out += dy.sum(axis=0)
        d_from_above = dy @ W_out        # gradient entering the top layer's h_k
        for l in range(L - 1, -1, -1):
            i, f, g, o = gates[l, k]
            c_prev = cs[l, k - 1]
            tanh_c = np.tanh(cs[l, k])
            dh = d_from_above + dh_next[l]
            do = dh * tanh_c
            dc = dh * o * (1.0 - tanh_c * tanh_c) + dc_next[l]
            di = dc * g
            df = dc * c_prev
            dg = dc * i
            dz = np.concatenate([
                di * i * (1.0 - i),
                df * f * (1.0 - f),
                dg * (1.0 - g * g),
                do * o * (1.0 - o),
            ], axis=1)                   # [B, 4H]
            inp = x[k - 1] if l == 0 else hs[l - 1, k]
            dW[l] += dz.T @ np.concatenate([inp, hs[l, k - 1]], axis=1)
            db[l] += dz.sum(axis=0)
            d_in = dz @ W[l]             # [B, I_l + H]
            I_l = inp.shape[1]
            dh_next[l] = d_in[:, I_l:]
            dc_next[l] = dc * f
            if l == 0:
                dx[k - 1] = d_in[:, :I_l]
            else:
                d_from_above = d_in[:, :I_l]
    return {
        "loss": float(loss_t.sum()),
        "loss_t": loss_t,
        "dW": dW,
        "db": db,
        "dW_out": dW_out,
        "db_out": db_out,
        "dx": dx,
    }


def lstm_loss(W, b, W_out, b_out, x, targets, h0, c0) -> float:
    """Forward pass and loss only (used by finite-difference checks)."""
    f64 = np.float64
    W = [np.asarray(w, f64) for w in W]
    b = [np.asarray(v, f64) for v in b]
    x = np.asarray(x, f64)
    L = len(W)
    t, B, _ = x.shape
    H = W[0].shape[0] // 4
    O = np.asarray(W_out).shape[0]
    hs, _, _ = lstm_forward(W, b, x, np.asarray(h0, f64).reshape(L, B, H),
                            np.asarray(c0, f64).reshape(L, B, H))
    total = 0.0
    for k in range(1, t + 1):
        y = hs[L - 1, k] @ np.asarray(W_out, f64).T + np.asarray(b_out, f64)
        diff = y - np.asarray(targets, f64)[k - 1]
        total += np.sum(diff * diff) / (B * O)
    return float(total)
