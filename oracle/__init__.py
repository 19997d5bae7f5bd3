"""Double-precision CPU oracle for the nested Forward-AD activation pass.

TEST INFRASTRUCTURE.  Only the test-suite, the smoke check and the benchmark's
``cpu_baseline`` / ``--impl reference`` legs may import this package; the CUDA
library never does, and this package imports nothing of the CUDA library.

The arithmetic lives in ``nfad_oracle.c`` (plain C, fp64, one expression per
quantity: Table I for the activations, Table II / Eq. 3 for the derivatives,
Eq. 4 for the backward product), ``nfad_seq_oracle.c`` (run-time FAD sequences)
and ``nfad_bias_oracle.c`` (the pass with its producer's bias-add and the bias
gradient).  This module compiles those files with gcc on first use and marshals numpy arrays into it.  Stored tensors cross the boundary
as raw bit patterns: ``float32`` arrays for fp32, ``uint16`` arrays for bf16 and
fp16.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

KINDS = {"gelu_erf": 0, "gelu_tanh": 1, "swish": 2, "mish": 3}
DTYPES = {"f32": 0, "bf16": 1, "f16": 2}

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "nfad_oracle.c")
_SRC_SEQ = os.path.join(_HERE, "nfad_seq_oracle.c")
_SRC_BIAS = os.path.join(_HERE, "nfad_bias_oracle.c")
_LIB = os.path.join(_HERE, "libnfad_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (IEEE semantics: no fast-math, no contraction)."""
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < max(os.path.getmtime(f) for f in (_SRC, _SRC_SEQ, _SRC_BIAS))
        if force or stale:
            cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp",
                   "-ffp-contract=off", "-fno-fast-math", "-o", _LIB, _SRC, _SRC_SEQ, _SRC_BIAS, "-lm"]
            subprocess.run(cmd, check=True, capture_output=True)
    return _LIB


class _Point(ctypes.Structure):
    _fields_ = [("f", ctypes.c_double), ("fprime", ctypes.c_double),
                ("term_h", ctypes.c_double), ("term_xh", ctypes.c_double)]


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        vp, sz, ci = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int
        lib.nfad_oracle_eval_point.argtypes = [ci, ctypes.c_double, ctypes.POINTER(_Point)]
        lib.nfad_oracle_forward.argtypes = [ci, ci, vp, sz, vp, vp, vp]
        lib.nfad_oracle_round.argtypes = [ci, vp, sz, vp]
        lib.nfad_oracle_widen.argtypes = [ci, vp, sz, vp]
        lib.nfad_oracle_backward.argtypes = [ci, vp, vp, sz, vp]
        lib.nfad_oracle_forward_backward.argtypes = [ci, ci, vp, vp, sz, vp, vp, vp]
        lib.nfad_oracle_set_threads.argtypes = [ci]
        for name in ("nfad_oracle_eval_point", "nfad_oracle_forward", "nfad_oracle_round",
                     "nfad_oracle_widen", "nfad_oracle_backward", "nfad_oracle_forward_backward",
                     "nfad_oracle_get_threads", "nfad_oracle_max_threads"):
            getattr(lib, name).restype = ci
        lib.nfad_oracle_set_threads.restype = None
        ip, dp = ctypes.POINTER(ctypes.c_int), ctypes.POINTER(ctypes.c_double)
        lib.nfad_seq_oracle_forward.argtypes = [ci, ip, ip, ip, ip, dp, vp, sz, ci, vp, vp]
        lib.nfad_seq_oracle_forward.restype = ci
        lib.nfad_seq_oracle_backward.argtypes = [vp, vp, sz, ci, vp, vp]
        lib.nfad_seq_oracle_backward.restype = ci
        lib.nfad_bias_oracle_forward.argtypes = [ci, ci, vp, vp, sz, sz, vp, vp, vp, vp]
        lib.nfad_bias_oracle_forward.restype = ci
        lib.nfad_bias_oracle_backward.argtypes = [ci, vp, vp, sz, sz, vp, vp, vp]
        lib.nfad_bias_oracle_backward.restype = ci
        _lib = lib
    return _lib


def _code(table, key):
    return table[key] if isinstance(key, str) else int(key)


def _storage_np(dtype) -> np.dtype:
    return np.dtype(np.float32) if _code(DTYPES, dtype) == 0 else np.dtype(np.uint16)


def _check_storage(a: np.ndarray, dtype) -> np.ndarray:
    want = _storage_np(dtype)
    if a.dtype != want:
        raise TypeError(f"stored tensor for dtype {dtype!r} must be a {want} array of raw values, got {a.dtype}")
    return np.ascontiguousarray(a).reshape(-1)


def _ptr(a: np.ndarray):
    return ctypes.c_void_p(a.ctypes.data)


def _ok(rc: int, what: str):
    if rc != 0:
        raise ValueError(f"{what}: oracle status {rc}")


def set_threads(t: int) -> None:
    _load().nfad_oracle_set_threads(int(t))


def get_threads() -> int:
    return _load().nfad_oracle_get_threads()


def max_threads() -> int:
    """Cores the process may run on (what an all-core timing uses)."""
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return _load().nfad_oracle_max_threads()


def eval_point(kind, x: float):
    """(f, f', h, x h') at one double x; f' = h + x h' (product rule, Eq. 3)."""
    p = _Point()
    _ok(_load().nfad_oracle_eval_point(_code(KINDS, kind), float(x), ctypes.byref(p)), "eval_point")
    return p.f, p.fprime, p.term_h, p.term_xh


def forward(kind, dtype, x: np.ndarray, want_cond: bool = False):
    """Unrounded f(x), f'(x) in fp64 for a stored tensor x; optionally |h| + |x h'|."""
    x = _check_storage(x, dtype)
    n = x.size
    f = np.empty(n, np.float64)
    fp = np.empty(n, np.float64)
    cond = np.empty(n, np.float64) if want_cond else None
    _ok(_load().nfad_oracle_forward(_code(KINDS, kind), _code(DTYPES, dtype), _ptr(x), n,
                                    _ptr(f), _ptr(fp), _ptr(cond) if want_cond else None), "forward")
    return (f, fp, cond) if want_cond else (f, fp)


def round_to(dtype, v: np.ndarray) -> np.ndarray:
    """One round-to-nearest-even from fp64 to the storage type (raw bit patterns)."""
    v = np.ascontiguousarray(v, np.float64).reshape(-1)
    out = np.empty(v.size, _storage_np(dtype))
    _ok(_load().nfad_oracle_round(_code(DTYPES, dtype), _ptr(v), v.size, _ptr(out)), "round_to")
    return out


def widen(dtype, a: np.ndarray) -> np.ndarray:
    """Stored values to fp64 (exact)."""
    a = _check_storage(a, dtype)
    out = np.empty(a.size, np.float64)
    _ok(_load().nfad_oracle_widen(_code(DTYPES, dtype), _ptr(a), a.size, _ptr(out)), "widen")
    return out


def backward(dtype, grad_out: np.ndarray, fprime_saved: np.ndarray) -> np.ndarray:
    """grad_in = RN(grad_out * f'_saved), the product formed exactly in fp64 (Eq. 4)."""
    g = _check_storage(grad_out, dtype)
    d = _check_storage(fprime_saved, dtype)
    if g.size != d.size:
        raise ValueError("size mismatch")
    out = np.empty(g.size, _storage_np(dtype))
    _ok(_load().nfad_oracle_backward(_code(DTYPES, dtype), _ptr(g), _ptr(d), g.size, _ptr(out)), "backward")
    return out


def forward_backward(kind, dtype, x: np.ndarray, grad_out: np.ndarray):
    """The whole path on the CPU: (y, f'_saved, grad_in) as stored tensors. Used for timing."""
    x = _check_storage(x, dtype)
    g = _check_storage(grad_out, dtype)
    if g.size != x.size:
        raise ValueError("size mismatch")
    st = _storage_np(dtype)
    y, d, gin = (np.empty(x.size, st) for _ in range(3))
    _ok(_load().nfad_oracle_forward_backward(_code(KINDS, kind), _code(DTYPES, dtype), _ptr(x), _ptr(g),
                                             x.size, _ptr(y), _ptr(d), _ptr(gin)), "forward_backward")
    return y, d, gin


SEQ_OPCODES = {"add": 0, "mul": 1, "scale": 2, "add_const": 3, "exp": 4, "log1p": 5, "tanh": 6, "erf": 7, "softplus": 8,
               "sigmoid": 9, "half_one_plus_tanh": 10, "half_one_plus_erf": 11, "out": 12}


def seq_forward(program, x: np.ndarray, m: int):
    """A FAD sequence in fp64.  program: list of (op name, a, b, dst, c); x: fp64 array.
    Returns (y, dydx), each of shape (m, n)."""
    n_ops = len(program)
    IntArr, DblArr = ctypes.c_int * n_ops, ctypes.c_double * n_ops
    op = IntArr(*[SEQ_OPCODES[o[0]] for o in program])
    a = IntArr(*[int(o[1]) for o in program])
    b = IntArr(*[int(o[2]) for o in program])
    dst = IntArr(*[int(o[3]) for o in program])
    c = DblArr(*[float(o[4]) for o in program])
    x = np.ascontiguousarray(x, np.float64).reshape(-1)
    y = np.empty((m, x.size), np.float64)
    d = np.empty((m, x.size), np.float64)
    _ok(_load().nfad_seq_oracle_forward(n_ops, op, a, b, dst, c, _ptr(x), x.size, m, _ptr(y), _ptr(d)), "seq_forward")
    return y, d


def seq_backward(g: np.ndarray, d: np.ndarray):
    """(sum_k g_k d_k, sum_k |g_k d_k|) in fp64 for operands of shape (m, n)."""
    g = np.ascontiguousarray(g, np.float64)
    d = np.ascontiguousarray(d, np.float64)
    m, n = g.shape
    out = np.empty(n, np.float64)
    out_abs = np.empty(n, np.float64)
    _ok(_load().nfad_seq_oracle_backward(_ptr(g), _ptr(d), n, m, _ptr(out), _ptr(out_abs)), "seq_backward")
    return out, out_abs


def bias_forward(kind, dtype, x: np.ndarray, bias: np.ndarray, rows: int, cols: int, want_cond: bool = False):
    """Unrounded f(z), f'(z) in fp64 at z = fl32(x[r, c] + bias[c]) for a row-major [rows, cols] stored tensor x
    and a stored bias of cols elements.  Returns (f, f', z) or (f, f', z, |h| + |z h'|), flat."""
    x = _check_storage(x, dtype)
    bias = _check_storage(bias, dtype)
    if x.size != rows * cols or bias.size != cols:
        raise ValueError("size mismatch")
    f, fp, z = (np.empty(x.size, np.float64) for _ in range(3))
    cond = np.empty(x.size, np.float64) if want_cond else None
    _ok(_load().nfad_bias_oracle_forward(_code(KINDS, kind), _code(DTYPES, dtype), _ptr(x), _ptr(bias), rows, cols,
                                         _ptr(f), _ptr(fp), _ptr(cond) if want_cond else None, _ptr(z)), "bias_forward")
    return (f, fp, z, cond) if want_cond else (f, fp, z)


def bias_backward(dtype, grad_out: np.ndarray, fprime_saved: np.ndarray, rows: int, cols: int):
    """(grad_in stored, grad_bias fp64, sum of |grad_in| per column fp64): grad_in = RN(grad_out * f'_saved) and
    grad_bias[c] = sum over rows of the rounded grad_in[r, c] (Eq. 4 for x; dz/db = 1 for the bias)."""
    g = _check_storage(grad_out, dtype)
    d = _check_storage(fprime_saved, dtype)
    if g.size != rows * cols or d.size != rows * cols:
        raise ValueError("size mismatch")
    gin = np.empty(g.size, _storage_np(dtype))
    gb = np.empty(cols, np.float64)
    gb_abs = np.empty(cols, np.float64)
    _ok(_load().nfad_bias_oracle_backward(_code(DTYPES, dtype), _ptr(g), _ptr(d), rows, cols, _ptr(gin), _ptr(gb),
                                          _ptr(gb_abs)), "bias_backward")
    return gin, gb, gb_abs
