"""Seeded synthetic LSTM training problems (inputs only; none of the method's arithmetic).

The paper's one timed workload is itself synthetic: an LSTM of a given size run over random
sequences of growing length (Section 4).  The problems made here have that shape.  Values are
drawn with a counter-based generator (Philox) in float64 and then rounded to the storage type
of the chosen precision, so every consumer sees exactly the same numbers:

* x, targets ~ N(0, 1) i.i.d.
* W (all layers), W_out ~ U(-1/sqrt(H), 1/sqrt(H)); biases 0 except the forget-gate block,
  which is 1; h0 = c0 = 0.
* ``make_problem(cfg, general=True)`` keeps x, targets and the weights and draws what the
  benchmark recipe leaves at a constant: every bias entry of every layer and of the readout
  ~ U(-0.3, 0.3) (the forget-gate block keeps its offset of 1), h0, c0 ~ 0.5 N(0, 1).  A
  consumer that mislaid a bias entry, dropped the readout bias or mishandled the caller's
  initial state cannot pass on such a problem.

Arrays are returned as float64 holding values that are exactly representable in the storage
type ("bf16": x, W, W_out, h0 in bfloat16 and the rest in float32; "fp32"/"tf32": float32).
``to_device_arrays`` turns them into the raw buffers a consumer uploads.
"""
from __future__ import annotations

from dataclasses import dataclass, asdict

import numpy as np

BASE_SEED = 160603401


@dataclass(frozen=True)
class LstmConfig:
    name: str
    layers: int
    input: int
    hidden: int
    batch: int
    t: int
    readout: int
    dtype: str          # "fp32" | "tf32" | "bf16"
    seed: int
    cell: str = "lstm"  # "lstm" | "gru": the recurrent core (a GRU has three gate blocks and no cell state)

    def asdict(self):
        return asdict(self)


# The five workloads, plus the shape of the paper's own timing experiment (Section 4).
CONFIGS = {
    "c1": LstmConfig("c1", 1, 32, 64, 4, 64, 32, "fp32", BASE_SEED + 0),
    "c2": LstmConfig("c2", 1, 512, 512, 64, 256, 512, "bf16", BASE_SEED + 1),
    "c3": LstmConfig("c3", 1, 1024, 1024, 64, 1000, 1024, "bf16", BASE_SEED + 2),
    "c4": LstmConfig("c4", 1, 256, 1024, 32, 4000, 256, "tf32", BASE_SEED + 3),
    "c5": LstmConfig("c5", 2, 1024, 2048, 128, 1000, 1024, "bf16", BASE_SEED + 4),
    "p0": LstmConfig("p0", 1, 256, 256, 64, 1000, 256, "bf16", BASE_SEED + 5),
}


def with_overrides(cfg: LstmConfig, **kw) -> LstmConfig:
    d = cfg.asdict()
    d.update(kw)
    return LstmConfig(**d)


def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """Round float64 values to the nearest bfloat16 (ties to even); result as float64."""
    f = np.asarray(a, np.float64).astype(np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).astype(np.float64)


def bf16_bits(a: np.ndarray) -> np.ndarray:
    """Raw uint16 patterns of values that are already bfloat16-representable."""
    f = np.ascontiguousarray(np.asarray(a, np.float64).astype(np.float32))
    return (f.view(np.uint32) >> 16).astype(np.uint16)


def round_to_fp32(a: np.ndarray) -> np.ndarray:
    return np.asarray(a, np.float64).astype(np.float32).astype(np.float64)


def make_problem(cfg: LstmConfig, general: bool = False) -> dict:
    """Draw one problem.  Keys: W (list per layer), b (list), W_out, b_out, x, targets, h0, c0.

    general: also draw the biases, the readout bias and the initial state (after everything else,
    so that x, targets and the weights are those of the plain problem with the same seed).
    """
    rng = np.random.Generator(np.random.Philox(key=cfg.seed))
    L, I, H, B, t, O = cfg.layers, cfg.input, cfg.hidden, cfg.batch, cfg.t, cfg.readout
    lim = 1.0 / np.sqrt(H)
    opnd = round_to_bf16 if cfg.dtype == "bf16" else round_to_fp32
    W, b = [], []
    for l in range(L):
        I_l = I if l == 0 else H
        ng = 3 if cfg.cell == "gru" else 4
        W.append(opnd(rng.uniform(-lim, lim, size=(ng * H, I_l + H))))
        bias = np.zeros(ng * H)
        if cfg.cell != "gru":
            bias[H:2 * H] = 1.0        # forget gate
        b.append(bias)
    W_out = opnd(rng.uniform(-lim, lim, size=(O, H)))
    b_out = np.zeros(O)
    x = opnd(rng.standard_normal(size=(t, B, I)))
    targets = round_to_fp32(rng.standard_normal(size=(t, B, O)))
    h0 = np.zeros((L, B, H))
    c0 = np.zeros((L, B, H))
    if general:
        b = [round_to_fp32(v + rng.uniform(-0.3, 0.3, size=v.size)) for v in b]
        b_out = round_to_fp32(rng.uniform(-0.3, 0.3, size=O))
        h0 = opnd(0.5 * rng.standard_normal(size=(L, B, H)))
        c0 = round_to_fp32(0.5 * rng.standard_normal(size=(L, B, H)))
    return {"W": W, "b": b, "W_out": W_out, "b_out": b_out, "x": x, "targets": targets,
            "h0": h0, "c0": c0}


def to_device_arrays(cfg: LstmConfig, prob: dict) -> dict:
    """Host arrays in the storage types of the library's C interface.

    Weights of all layers are concatenated row-major, layer after layer.  Operands (W, W_out,
    x, h0) are uint16 bfloat16 patterns in "bf16" precision and float32 otherwise; biases,
    targets and c0 are float32.
    """
    if cfg.dtype == "bf16":
        conv = bf16_bits
    else:
        conv = lambda a: np.ascontiguousarray(np.asarray(a, np.float64).astype(np.float32))
    f32 = lambda a: np.ascontiguousarray(np.asarray(a, np.float64).astype(np.float32))
    return {
        "W": np.concatenate([conv(w).ravel() for w in prob["W"]]),
        "b": np.concatenate([f32(v).ravel() for v in prob["b"]]),
        "W_out": conv(prob["W_out"]).ravel(),
        "b_out": f32(prob["b_out"]).ravel(),
        "x": conv(prob["x"]).ravel(),
        "targets": f32(prob["targets"]).ravel(),
        "h0": conv(prob["h0"]).ravel(),
        "c0": f32(prob["c0"]).ravel(),
    }
