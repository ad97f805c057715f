"""Device-memory plumbing around the C interface: upload a problem, run steps, fetch results.

Nothing here computes anything; it allocates torch tensors, hands their addresses to
``binding`` and copies results back.  Used by the tests, the smoke check and the benchmark.
"""
from __future__ import annotations

import numpy as np
import torch

from . import binding as B
from . import synth


def _torch_dtype(cfg_dtype: str):
    return torch.bfloat16 if cfg_dtype == "bf16" else torch.float32


def _upload(arr: np.ndarray, device) -> torch.Tensor:
    """Raw upload; uint16 arrays are bfloat16 bit patterns."""
    if arr.dtype == np.uint16:
        return torch.from_numpy(arr.view(np.int16)).to(device).view(torch.bfloat16)
    return torch.from_numpy(arr).to(device)


class DeviceProblem:
    """One synthetic problem resident on a GPU, with output buffers and a workspace."""

    def __init__(self, cfg: synth.LstmConfig, prob: dict | None = None, device="cuda:0", want_dx=False,
                 flags=0):
        self.cfg = cfg
        self.device = torch.device(device)
        self.prob = prob if prob is not None else synth.make_problem(cfg)
        self.host = synth.to_device_arrays(cfg, self.prob)
        self.want_dx = bool(want_dx)
        if getattr(cfg, "cell", "lstm") == "gru":
            flags |= B.MEBPTT_FLAG_GRU
        self.desc = B.make_desc(cfg.layers, cfg.input, cfg.hidden, cfg.readout, cfg.batch, cfg.t,
                                cfg.dtype, want_dx=int(self.want_dx), flags=flags)
        self.dev = {k: _upload(v, self.device) for k, v in self.host.items()}
        f32 = dict(dtype=torch.float32, device=self.device)
        nW = self.host["W"].size
        self.out = {
            "loss": torch.zeros(1, **f32),
            "dW": torch.zeros(nW, **f32),
            "db": torch.zeros(self.host["b"].size, **f32),
            "dW_out": torch.zeros(self.host["W_out"].size, **f32),
            "db_out": torch.zeros(self.host["b_out"].size, **f32),
            "dx": torch.zeros(self.host["x"].size, **f32) if self.want_dx else None,
            "counters": torch.zeros(8, dtype=torch.int64, device=self.device),
        }
        self._ws = None

    def plan(self, mode, m, alpha=4, beta=0) -> B.Plan:
        if isinstance(mode, str):
            mode = B.MODES[mode]
        return B.mebptt_plan_ex(self.cfg.t, m, mode, alpha, beta)

    def full_memory_plan(self) -> B.Plan:
        """Standard BPTT: ISM with as many internal states as steps (Section 3.2)."""
        return B.mebptt_plan_ex(self.cfg.t, self.cfg.t, B.MEBPTT_ISM, 4, 0)

    def workspace(self, nbytes: int) -> torch.Tensor:
        if self._ws is None or self._ws.numel() < nbytes:
            self._ws = None
            self._ws = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
        return self._ws

    def enqueue(self, plan: B.Plan, stream=None):
        """Enqueue one training step; returns immediately."""
        ws = self.workspace(B.mebptt_lstm_workspace_bytes(self.desc, plan))
        d, o = self.dev, self.out
        s = stream if stream is not None else torch.cuda.current_stream(self.device).cuda_stream
        B.mebptt_lstm_train_step(self.desc, plan, d["W"], d["b"], d["W_out"], d["b_out"], d["x"],
                                 d["targets"], d["h0"], d["c0"], ws, s, o["loss"], o["dW"], o["db"],
                                 o["dW_out"], o["db_out"], o["dx"], o["counters"])

    def run(self, plan: B.Plan) -> dict:
        """One step, synchronised, results as numpy arrays (exact copies of the device bits)."""
        self.enqueue(plan)
        torch.cuda.synchronize(self.device)
        res = {k: (v.cpu().numpy().copy() if v is not None else None) for k, v in self.out.items()}
        res["loss"] = float(res["loss"][0])
        return res

    def split_dW(self, flat: np.ndarray):
        """Flat dW -> list of per-layer [4H, I_l + H] arrays."""
        c, out, off = self.cfg, [], 0
        for l in range(c.layers):
            K = (c.input if l == 0 else c.hidden) + c.hidden
            ng = 3 if getattr(c, "cell", "lstm") == "gru" else 4
            n = ng * c.hidden * K
            out.append(flat[off:off + n].reshape(ng * c.hidden, K))
            off += n
        return out


def rel_l2(a, b) -> float:
    """|| a - b || / || b || over flattened float64 copies."""
    a = np.asarray(a, np.float64).ravel()
    b = np.asarray(b, np.float64).ravel()
    den = np.linalg.norm(b)
    return float(np.linalg.norm(a - b) / (den if den > 0 else 1.0))
