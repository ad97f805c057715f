"""ctypes binding of libmebptt: same names as the C interface, argument marshalling only.

Device buffers are torch CUDA tensors (PyTorch is used for memory and streams, nothing else);
every step of the computation runs inside the library.  Importing this module loads the shared
library and fails loudly when it has not been built -- there is no fallback.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("MEBPTT_LIB") or os.path.join(_PKG, "libmebptt.so")   # MEBPTT_LIB: another build of the library

MEBPTT_HSM, MEBPTT_ISM, MEBPTT_MSM, MEBPTT_CHEN_SQRT, MEBPTT_CHEN_RECURSIVE = 0, 1, 2, 3, 4
MEBPTT_FP32, MEBPTT_TF32, MEBPTT_BF16 = 0, 1, 2
MEBPTT_OK = 0
MEBPTT_ERR_ARG, MEBPTT_ERR_BUDGET, MEBPTT_ERR_WORKSPACE, MEBPTT_ERR_UNSUPPORTED = -1, -2, -3, -4
MEBPTT_ERR_CUDA, MEBPTT_ERR_TIMEOUT, MEBPTT_ERR_OOM, MEBPTT_ERR_PLAN = -5, -6, -7, -8
MEBPTT_OP_FWD, MEBPTT_OP_BWD = 1, 2
MEBPTT_FMT_HIDDEN, MEBPTT_FMT_INTERNAL, MEBPTT_FMT_INTERNAL_NOINPUT = 0, 1, 2
MEBPTT_LOC_INIT, MEBPTT_LOC_PING, MEBPTT_LOC_PONG, MEBPTT_LOC_CORE = -1, -2, -3, -4
MEBPTT_INF = 1 << 60
MODES = {"hsm": MEBPTT_HSM, "ism": MEBPTT_ISM, "msm": MEBPTT_MSM}
DTYPES = {"fp32": MEBPTT_FP32, "tf32": MEBPTT_TF32, "bf16": MEBPTT_BF16}

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python -m paper_1606_03401_b200.build` "
        "(there is no fallback implementation)")
lib = C.CDLL(LIB_PATH)


class mebptt_op(C.Structure):
    _fields_ = [("kind", C.c_int32), ("k", C.c_int32), ("src", C.c_int32), ("dst", C.c_int32),
                ("dst_fmt", C.c_int32), ("aux", C.c_int32), ("units", C.c_int32),
                ("reserved", C.c_int32)]


OP_DTYPE = np.dtype([("kind", "<i4"), ("k", "<i4"), ("src", "<i4"), ("dst", "<i4"),
                     ("dst_fmt", "<i4"), ("aux", "<i4"), ("units", "<i4"), ("reserved", "<i4")])


class mebptt_lstm_desc(C.Structure):
    _fields_ = [("layers", C.c_int32), ("input", C.c_int32), ("hidden", C.c_int32),
                ("readout", C.c_int32), ("batch", C.c_int32), ("dtype", C.c_int32),
                ("want_dx", C.c_int32), ("flags", C.c_int32), ("t", C.c_int64)]


_vp, _i64, _i32, _sz = C.c_void_p, C.c_int64, C.c_int, C.c_size_t
_descp = C.POINTER(mebptt_lstm_desc)
_STEP_ARGS = [_descp, _vp] + [_vp] * 8 + [_vp, _sz, _vp] + [_vp] * 7

_SIGS = {
    "mebptt_plan": (_i32, [_i64, _i64, _i32, C.POINTER(_vp)]),
    "mebptt_plan_ex": (_i32, [_i64, _i64, _i32, _i32, _i32, C.POINTER(_vp)]),
    "mebptt_plan_chen_sqrt": (_i32, [_i64, _i32, _i32, C.POINTER(_vp)]),
    "mebptt_plan_chen_recursive": (_i32, [_i64, _i32, _i32, _i32, C.POINTER(_vp)]),
    "mebptt_plan_free": (None, [_vp]),
    "mebptt_plan_cost": (_i64, [_vp]),
    "mebptt_plan_num_ops": (_i64, [_vp]),
    "mebptt_plan_tape": (C.POINTER(mebptt_op), [_vp]),
    "mebptt_plan_peak_units": (_i64, [_vp]),
    "mebptt_plan_arena_units": (_i64, [_vp]),
    "mebptt_plan_t_len": (_i64, [_vp]),
    "mebptt_plan_m": (_i64, [_vp]),
    "mebptt_plan_mode": (_i32, [_vp]),
    "mebptt_plan_sized": (_i32, [_i64, _i64, _i32, _i32, _i32, C.POINTER(_vp)]),
    "mebptt_plan_bytes_exact": (_i32, [_descp, _sz, _i32, _i32, C.POINTER(_vp)]),
    "mebptt_plan_sigma": (_i32, [_vp]),
    "mebptt_plan_alpha": (_i32, [_vp]),
    "mebptt_plan_beta": (_i32, [_vp]),
    "mebptt_plan_tables": (_i32, [_vp, C.POINTER(C.POINTER(C.c_int64)), C.POINTER(C.POINTER(C.c_int32)),
                                  C.POINTER(C.POINTER(C.c_int32)), C.POINTER(C.POINTER(C.c_uint8)),
                                  C.POINTER(_i64), C.POINTER(_i64)]),
    "mebptt_plan_validate": (_i32, [_vp]),
    "mebptt_lstm_unit_bytes": (_sz, [_descp]),
    "mebptt_budget_bytes_to_units": (_i64, [_descp, _sz]),
    "mebptt_plan_for_bytes": (_i32, [_descp, _sz, _i32, _i32, C.POINTER(_vp)]),
    "mebptt_lstm_workspace_bytes": (_sz, [_descp, _vp]),
    "mebptt_lstm_working_bytes": (_sz, [_descp, _vp]),
    "mebptt_lstm_host_workspace_bytes": (_sz, [_descp, _vp]),
    "mebptt_lstm_launch_count": (_i64, [_descp, _vp]),
    "mebptt_lstm_train_step": (_i32, _STEP_ARGS),
    "mebptt_lstm_train_step_host": (_i32, _STEP_ARGS),
    "mebptt_lstm_train_step_static": (_i32, [_descp, _vp] + [_vp] * 8 + [_vp] + [_vp] * 7),
    "mebptt_lstm_run_times": (_i32, [C.POINTER(C.c_double), C.POINTER(_i64), C.POINTER(_i64)]),
    "mebptt_lstm_prepare": (_i32, [_descp, _vp]),
    "mebptt_lstm_prepare_stats": (_i32, [C.POINTER(_i64)]),
    "mebptt_test_wait_fault": (_i32, [_i32]),
    "mebptt_slot_copy": (_i32, [_vp, _vp, _sz, _vp]),
    "mebptt_gemm_bf16": (_i32, [_vp, _i64, _i32, _vp, _i64, _i32, _vp, _i64, _i32, _vp, _i64, _i64, _i64, _vp, _vp]),
    "mebptt_strerror": (C.c_char_p, [_i32]),
}
for _name, (_res, _args) in _SIGS.items():
    _fn = getattr(lib, _name)       # AttributeError here = the library does not export it
    _fn.restype = _res
    _fn.argtypes = _args

EXPORTED = tuple(_SIGS)


class MebpttError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {mebptt_strerror(status)} ({status})")


def mebptt_strerror(status: int) -> str:
    return lib.mebptt_strerror(status).decode()


def _check(status: int, where: str):
    if status != MEBPTT_OK:
        raise MebpttError(status, where)


class Plan:
    """Owner of a mebptt_plan_t."""

    def __init__(self, handle):
        self._h = handle

    def __del__(self):
        h, self._h = getattr(self, "_h", None), None
        if h:
            lib.mebptt_plan_free(h)

    handle = property(lambda self: self._h)
    cost = property(lambda self: lib.mebptt_plan_cost(self._h))
    num_ops = property(lambda self: lib.mebptt_plan_num_ops(self._h))
    peak_units = property(lambda self: lib.mebptt_plan_peak_units(self._h))
    arena_units = property(lambda self: lib.mebptt_plan_arena_units(self._h))
    t = property(lambda self: lib.mebptt_plan_t_len(self._h))
    m = property(lambda self: lib.mebptt_plan_m(self._h))
    mode = property(lambda self: lib.mebptt_plan_mode(self._h))
    sigma = property(lambda self: lib.mebptt_plan_sigma(self._h))
    alpha = property(lambda self: lib.mebptt_plan_alpha(self._h))
    beta = property(lambda self: lib.mebptt_plan_beta(self._h))

    def tape(self) -> np.ndarray:
        """Copy of the tape as a structured array."""
        n = self.num_ops
        ptr = lib.mebptt_plan_tape(self._h)
        buf = C.string_at(ptr, n * C.sizeof(mebptt_op))
        return np.frombuffer(buf, dtype=OP_DTYPE).copy()

    def tables(self) -> dict:
        """Copies of the DP tables, each [t + 1, m + 1]."""
        pc, pd, pd2, ph = (C.POINTER(C.c_int64)(), C.POINTER(C.c_int32)(), C.POINTER(C.c_int32)(),
                           C.POINTER(C.c_uint8)())
        td, md = _i64(), _i64()
        _check(lib.mebptt_plan_tables(self._h, C.byref(pc), C.byref(pd), C.byref(pd2), C.byref(ph),
                                      C.byref(td), C.byref(md)), "mebptt_plan_tables")
        shape = (td.value, md.value)
        n = shape[0] * shape[1]
        out = {}
        if pc:
            out["C"] = np.ctypeslib.as_array(pc, shape=(n,)).reshape(shape).copy()
        if pd:
            out["D"] = np.ctypeslib.as_array(pd, shape=(n,)).reshape(shape).copy()
        if pd2:
            out["D2"] = np.ctypeslib.as_array(pd2, shape=(n,)).reshape(shape).copy()
        if ph:
            out["H"] = np.ctypeslib.as_array(ph, shape=(n,)).reshape(shape).copy()
        return out

    def validate(self) -> int:
        return lib.mebptt_plan_validate(self._h)


def mebptt_plan(t: int, m: int, mode: int) -> Plan:
    h = _vp()
    _check(lib.mebptt_plan(t, m, mode, C.byref(h)), "mebptt_plan")
    return Plan(h)


def mebptt_plan_ex(t: int, m: int, mode: int, alpha: int = 4, beta: int = 0) -> Plan:
    h = _vp()
    _check(lib.mebptt_plan_ex(t, m, mode, alpha, beta, C.byref(h)), "mebptt_plan_ex")
    return Plan(h)


MEBPTT_FLAG_NO_TENSOR_CORES = 1
MEBPTT_FLAG_TIME_RUNS = 2
MEBPTT_FLAG_GRU = 4


def mebptt_plan_chen_sqrt(t: int, alpha: int = 4, beta: int = 3) -> Plan:
    h = _vp()
    _check(lib.mebptt_plan_chen_sqrt(t, alpha, beta, C.byref(h)), "mebptt_plan_chen_sqrt")
    return Plan(h)


def mebptt_plan_chen_recursive(t: int, k: int, alpha: int = 4, beta: int = 3) -> Plan:
    h = _vp()
    _check(lib.mebptt_plan_chen_recursive(t, k, alpha, beta, C.byref(h)), "mebptt_plan_chen_recursive")
    return Plan(h)


def make_desc(layers, input, hidden, readout, batch, t, dtype, want_dx=0, flags=0) -> mebptt_lstm_desc:
    if isinstance(dtype, str):
        dtype = DTYPES[dtype]
    return mebptt_lstm_desc(layers, input, hidden, readout, batch, dtype, int(want_dx), int(flags), t)


def mebptt_lstm_unit_bytes(desc) -> int:
    return lib.mebptt_lstm_unit_bytes(C.byref(desc))


def mebptt_budget_bytes_to_units(desc, nbytes: int) -> int:
    return lib.mebptt_budget_bytes_to_units(C.byref(desc), nbytes)


def mebptt_plan_for_bytes(desc, nbytes: int, mode: int, include_working: bool = False) -> Plan:
    h = _vp()
    _check(lib.mebptt_plan_for_bytes(C.byref(desc), nbytes, mode, int(include_working), C.byref(h)),
           "mebptt_plan_for_bytes")
    return Plan(h)


def mebptt_plan_sized(t: int, m: int, sigma: int, alpha: int, beta: int = 0) -> Plan:
    h = _vp()
    _check(lib.mebptt_plan_sized(t, m, sigma, alpha, beta, C.byref(h)), "mebptt_plan_sized")
    return Plan(h)


def mebptt_plan_bytes_exact(desc, nbytes: int, use_beta: bool = True, include_working: bool = False) -> Plan:
    h = _vp()
    _check(lib.mebptt_plan_bytes_exact(C.byref(desc), nbytes, int(use_beta), int(include_working), C.byref(h)),
           "mebptt_plan_bytes_exact")
    return Plan(h)


def mebptt_lstm_workspace_bytes(desc, plan: Plan) -> int:
    return lib.mebptt_lstm_workspace_bytes(C.byref(desc), plan.handle)


def mebptt_lstm_working_bytes(desc, plan: Plan) -> int:
    return lib.mebptt_lstm_working_bytes(C.byref(desc), plan.handle)


def mebptt_lstm_host_workspace_bytes(desc, plan: Plan) -> int:
    return lib.mebptt_lstm_host_workspace_bytes(C.byref(desc), plan.handle)


def mebptt_lstm_launch_count(desc, plan: Plan) -> int:
    return lib.mebptt_lstm_launch_count(C.byref(desc), plan.handle)


def _ptr(a):
    """Address of a torch tensor, a numpy array, or None."""
    if a is None:
        return None
    if isinstance(a, np.ndarray):
        return a.ctypes.data
    return a.data_ptr()


def _nbytes(a):
    return a.nbytes if isinstance(a, np.ndarray) else a.numel() * a.element_size()


def _step(fn, name, desc, plan, W, b, W_out, b_out, x, targets, h0, c0, workspace, stream,
          loss, dW, db, dW_out, db_out, dx, counters):
    st = fn(C.byref(desc), plan.handle, _ptr(W), _ptr(b), _ptr(W_out), _ptr(b_out), _ptr(x),
            _ptr(targets), _ptr(h0), _ptr(c0), _ptr(workspace), _nbytes(workspace),
            stream, _ptr(loss), _ptr(dW), _ptr(db), _ptr(dW_out), _ptr(db_out), _ptr(dx),
            _ptr(counters))
    _check(st, name)


def mebptt_lstm_train_step(desc, plan, W, b, W_out, b_out, x, targets, h0, c0, workspace, stream,
                           loss, dW, db, dW_out, db_out, dx, counters):
    """All tensors on the device; `stream` is a raw cudaStream_t (int) or None."""
    _step(lib.mebptt_lstm_train_step, "mebptt_lstm_train_step", desc, plan, W, b, W_out, b_out, x,
          targets, h0, c0, workspace, stream, loss, dW, db, dW_out, db_out, dx, counters)


def mebptt_lstm_train_step_host(desc, plan, W, b, W_out, b_out, x, targets, h0, c0, workspace,
                                stream, loss, dW, db, dW_out, db_out, dx, counters):
    """Inputs and outputs in host memory (numpy arrays or pinned torch tensors); the workspace
    is a device tensor of at least mebptt_lstm_host_workspace_bytes()."""
    _step(lib.mebptt_lstm_train_step_host, "mebptt_lstm_train_step_host", desc, plan, W, b, W_out,
          b_out, x, targets, h0, c0, workspace, stream, loss, dW, db, dW_out, db_out, dx, counters)


MEBPTT_STATIC_WORKSPACE_BYTES = 32 << 20


def mebptt_lstm_train_step_static(desc, plan, W, b, W_out, b_out, x, targets, h0, c0, stream,
                                  loss, dW, db, dW_out, db_out, dx, counters):
    """The training step without a caller-supplied workspace: for code that may not allocate
    device memory.  Uses the library's built-in MEBPTT_STATIC_WORKSPACE_BYTES array; problems
    that need more raise MebpttError(MEBPTT_ERR_WORKSPACE).  Calls share the array: keep them on
    one stream."""
    st = lib.mebptt_lstm_train_step_static(
        C.byref(desc), plan.handle, _ptr(W), _ptr(b), _ptr(W_out), _ptr(b_out), _ptr(x), _ptr(targets),
        _ptr(h0), _ptr(c0), stream, _ptr(loss), _ptr(dW), _ptr(db), _ptr(dW_out), _ptr(db_out), _ptr(dx),
        _ptr(counters))
    _check(st, "mebptt_lstm_train_step_static")


def mebptt_lstm_prepare(desc, plan) -> None:
    _check(lib.mebptt_lstm_prepare(C.byref(desc), plan._h), "mebptt_lstm_prepare")


def mebptt_lstm_prepare_stats() -> dict:
    out = (_i64 * 4)()
    _check(lib.mebptt_lstm_prepare_stats(out), "mebptt_lstm_prepare_stats")
    return {"built": out[0], "reused": out[1], "page_locked": out[2], "held": out[3]}


def mebptt_test_wait_fault(mask: int) -> None:
    _check(lib.mebptt_test_wait_fault(int(mask)), "mebptt_test_wait_fault")


def mebptt_lstm_run_times() -> dict:
    """{"forward": (ms, launches, ops), "backward": (...)} of the steps run with MEBPTT_FLAG_TIME_RUNS."""
    ms, n, ops = (C.c_double * 2)(), (_i64 * 2)(), (_i64 * 2)()
    _check(lib.mebptt_lstm_run_times(ms, n, ops), "mebptt_lstm_run_times")
    return {"forward": (ms[0], n[0], ops[0]), "backward": (ms[1], n[1], ops[1])}


def mebptt_gemm_bf16(A, lda, a_major, Bm, ldb, b_major, Cm, ldc, accumulate, bias, M, N, K, status=None,
                     stream=None):
    _check(lib.mebptt_gemm_bf16(_ptr(A), lda, a_major, _ptr(Bm), ldb, b_major, _ptr(Cm), ldc, int(accumulate),
                                _ptr(bias), M, N, K, _ptr(status), stream), "mebptt_gemm_bf16")


def mebptt_slot_copy(dst, src, nbytes: int, stream=None):
    _check(lib.mebptt_slot_copy(_ptr(dst), _ptr(src), nbytes, stream), "mebptt_slot_copy")
