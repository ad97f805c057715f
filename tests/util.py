"""Helpers shared by the GPU parity tests."""
import numpy as np

from oracle import lstm_bptt as O

TOL = {"fp32": 1e-4, "tf32": 1e-4, "bf16": 2e-2}   # relative L2 error against the fp64 oracle


def oracle_run(prob):
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


def assert_close_to_oracle(res, ref, dtype, want_dx=False):
    tol = TOL[dtype]
    fo = flat_oracle(ref)
    assert abs(res["loss"] - ref["loss"]) <= tol * abs(ref["loss"]), (res["loss"], ref["loss"])
    keys = ["dW", "db", "dW_out", "db_out"] + (["dx"] if want_dx else [])
    errs = {k: rel_l2(res[k], fo[k]) for k in keys}
    for k, e in errs.items():
        assert e <= tol, (k, e, errs)
    return errs


def assert_bit_identical(a, b, want_dx=False):
    keys = ["dW", "db", "dW_out", "db_out"] + (["dx"] if want_dx else [])
    assert np.float32(a["loss"]).tobytes() == np.float32(b["loss"]).tobytes()
    for k in keys:
        assert a[k].tobytes() == b[k].tobytes(), k
