"""Helpers shared by the GPU parity tests."""
import numpy as np

from oracle import gru_bptt as OG
from oracle import lstm_bptt as O

TOL = {"fp32": 1e-4, "tf32": 1e-4, "bf16": 2e-2}   # relative L2 error against the fp64 oracle


def oracle_run(prob):
    if prob["W"][0].shape[0] % 3 == 0 and prob["W"][0].shape[0] // 3 == prob["h0"].shape[-1]:   # three gate blocks: a GRU
        return OG.gru_bptt(prob["W"], prob["b"], prob["W_out"], prob["b_out"], prob["x"], prob["targets"], prob["h0"])
    return O.lstm_bptt(prob["W"], prob["b"], prob["W_out"], prob["b_out"], prob["x"], prob["targets"],
                       prob["h0"], prob["c0"])


def flat_oracle(ref):
    """Oracle gradients flattened the way the C interface lays them out."""
    return {
        "dW": np.concatenate([a.ravel() for a in ref["dW"]]),
        "db": np.concatenate([a.ravel() for a in ref["db"]]),
        "dW_out": ref["dW_out"].ravel(),
        "db_out": ref["db_out"].ravel(),
        "dx": ref["dx"].ravel(),
    }


def rel_l2(a, b):
    a = np.asarray(a, np.float64).ravel()
    b = np.asarray(b, np.float64).ravel()
    den = np.linalg.norm(b)
    return float(np.linalg.norm(a - b) / (den if den > 0 else 1.0))


BLOCK_FACTOR = 4.0   # a block may be this many times further off than the whole tensor is allowed to be


def _blocks(name, arr, gates=4):
    """(label, index) pairs cutting an oracle array into the blocks a kernel mistake would hit:
    gate blocks and 128 x 128 tiles of a weight gradient, 32 entries of a bias gradient, one
    time step of dx."""
    if name == "dW":          # [4H, K] (LSTM) or [3H, K] (GRU): K - I = H columns are recurrent
        G, K = arr.shape
        ng = 4 if gates == 4 else 3
        H = G // ng
        for q in range(ng):
            yield f"gate block {q}", (slice(q * H, (q + 1) * H), slice(None))
        for r in range(0, G, 128):
            for c in range(0, K, 128):
                yield f"tile ({r},{c})", (slice(r, r + 128), slice(c, c + 128))
    elif name == "dW_out":    # [O, H]
        R, C = arr.shape
        for r in range(0, R, 128):
            for c in range(0, C, 128):
                yield f"tile ({r},{c})", (slice(r, r + 128), slice(c, c + 128))
    elif name in ("db", "db_out"):
        for r in range(0, arr.shape[0], 32):
            yield f"entries {r}..", (slice(r, r + 32),)
    elif name == "dx":        # [t, B, I]
        for k in range(arr.shape[0]):
            yield f"step {k + 1}", (k,)


def _assert_blocks_close(name, got, ref, tol, gates=4):
    """Relative L2 per block.  The denominator is the block's own norm, floored at a tenth of
    what an average block of the tensor carries, so that a block that happens to be near zero is
    held to the tensor's scale instead of its own."""
    got = np.asarray(got, np.float64).reshape(ref.shape)
    labels, num, den = [], [], []
    for label, idx in _blocks(name, ref, gates):
        labels.append(label)
        num.append(np.linalg.norm(got[idx] - ref[idx]))
        den.append(np.linalg.norm(ref[idx]))
    if not labels:
        return 0.0
    num, den = np.array(num), np.array(den)
    floor = 0.1 * np.sqrt(np.mean(den ** 2))
    err = num / np.maximum(np.maximum(den, floor), 1e-300)
    worst = int(np.argmax(err))
    assert err[worst] <= BLOCK_FACTOR * tol, (name, labels[worst], float(err[worst]))
    return float(err[worst])


def assert_close_to_oracle(res, ref, dtype, want_dx=False):
    """Loss and every gradient against the oracle: relative L2 over each whole tensor within the
    tolerance, and over each block of it (``_blocks``) within BLOCK_FACTOR times the tolerance --
    a wrong tile edge, gate row or bias entry is a small part of the whole tensor's norm but all
    of its block's."""
    tol = TOL[dtype]
    fo = flat_oracle(ref)
    assert abs(res["loss"] - ref["loss"]) <= tol * abs(ref["loss"]), (res["loss"], ref["loss"])
    keys = ["dW", "db", "dW_out", "db_out"] + (["dx"] if want_dx else [])
    errs = {k: rel_l2(res[k], fo[k]) for k in keys}
    for k, e in errs.items():
        assert e <= tol, (k, e, errs)
    off_w = off_b = 0
    H = ref["dW_out"].shape[1]
    for l, (w, v) in enumerate(zip(ref["dW"], ref["db"])):
        errs[f"dW[{l}] worst block"] = _assert_blocks_close("dW", res["dW"][off_w:off_w + w.size], w, tol, w.shape[0] // H)
        errs[f"db[{l}] worst block"] = _assert_blocks_close("db", res["db"][off_b:off_b + v.size], v, tol)
        off_w += w.size
        off_b += v.size
    errs["dW_out worst block"] = _assert_blocks_close("dW_out", res["dW_out"], ref["dW_out"], tol)
    errs["db_out worst block"] = _assert_blocks_close("db_out", res["db_out"], ref["db_out"], tol)
    if want_dx:
        errs["dx worst step"] = _assert_blocks_close("dx", res["dx"], ref["dx"], tol)
    return errs


def assert_bit_identical(a, b, want_dx=False):
    keys = ["dW", "db", "dW_out", "db_out"] + (["dx"] if want_dx else [])
    assert np.float32(a["loss"]).tobytes() == np.float32(b["loss"]).tobytes()
    for k in keys:
        assert a[k].tobytes() == b[k].tobytes(), k
