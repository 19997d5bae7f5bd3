"""The library's dual-number algebra compiled for the host (tests/host_algebra.cpp) against the oracle: constants,
signs, clamps and the order of operations of the four chains, checked without a GPU.  The hardware's approximate
units are replaced by exact C functions, so the tolerances of the GPU parity tests apply unchanged (tests/parity.py);
the real instructions are covered by the GPU tests."""
import ctypes
import os
import shutil
import subprocess

import numpy as np
import pytest
import torch

import oracle
import parity
import ulp
from paper_2209_10778_b200 import workloads as W

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(os.path.dirname(HERE), "paper_2209_10778_b200", "csrc")
KINDS = list(W.KINDS)


@pytest.fixture(scope="module")
def host(tmp_path_factory):
    cxx = shutil.which("g++")
    if cxx is None:
        pytest.skip("no g++")
    so = str(tmp_path_factory.mktemp("host_algebra") / "libhost_algebra.so")
    subprocess.run([cxx, "-O2", "-std=c++17", "-ffp-contract=off", "-shared", "-fPIC", "-I", CSRC,
                    os.path.join(HERE, "host_algebra.cpp"), "-o", so], check=True)
    lib = ctypes.CDLL(so)
    lib.host_algebra.argtypes = [ctypes.c_int, ctypes.c_int] + [ctypes.c_void_p] * 5 + [ctypes.c_size_t]
    lib.host_algebra.restype = None
    lib.host_primitive.argtypes = [ctypes.c_int, ctypes.c_int] + [ctypes.c_void_p] * 3 + [ctypes.c_size_t]
    lib.host_primitive.restype = None

    def run(kind: str, width: int, x: np.ndarray):
        x = np.ascontiguousarray(x, np.float32)
        out = [np.empty_like(x) for _ in range(4)]
        lib.host_algebra(KINDS.index(kind), width, x.ctypes.data, *[o.ctypes.data for o in out], x.size)
        return out                                   # y, f', value-only y, gate

    def primitive(op: int, wide: bool, x: np.ndarray):
        x = np.ascontiguousarray(x, np.float64)
        v, t = np.empty_like(x), np.empty_like(x)
        lib.host_primitive(op, int(wide), x.ctypes.data, v.ctypes.data, t.ctypes.data, x.size)
        return v, t

    run.primitive = primitive
    return run


def _all_16bit_as_f32(dtype: str, limit: float = None):
    t = W.all_finite_16bit(dtype)
    if limit is not None:
        t = t[t.to(torch.float32).abs() <= limit].contiguous()
    return t, t.to(torch.float32).numpy().copy()


@pytest.mark.parametrize("kind", KINDS)
def test_one_and_two_elements_per_call_agree(host, kind):
    """The chains are one template for both widths: every lane of a pair must see the scalar operation sequence."""
    xs = np.concatenate([_all_16bit_as_f32("bf16")[1], _all_16bit_as_f32("f16")[1],
                         np.array([np.inf, -np.inf, np.nan, 3.0e38, -3.0e38, 1e-40], np.float32)])
    if xs.size % 2:
        xs = xs[:-1]
    one, two = host(kind, 0, xs), host(kind, 1, xs)
    for a, b, name in zip(one, two, ("y", "f'", "value-only y", "gate")):
        assert ulp.same_bits_or_both_nan(a, b, "f32").all(), name


@pytest.mark.parametrize("dtype", ["bf16", "f16"])
@pytest.mark.parametrize("kind", KINDS)
def test_fp32_chain_on_every_16bit_input(host, kind, dtype):
    """16-bit storage: results rounded once to the type are within 1 ulp of the oracle's, for every finite input
    with |x| <= 80.5 (the GPU test's range), in the training and in the value-only form."""
    t, x32 = _all_16bit_as_f32(dtype, 80.5)
    x_raw = W.raw_numpy(t)
    y, d, v, _ = host(kind, 0, x32)
    y_bits = oracle.round_to(dtype, y.astype(np.float64))
    d_bits = oracle.round_to(dtype, d.astype(np.float64))
    parity.check_forward_16(kind, dtype, x_raw, y_bits, d_bits)
    f, _ = oracle.forward(kind, dtype, x_raw)
    dv = ulp.ulp_distance16(oracle.round_to(dtype, v.astype(np.float64)), oracle.round_to(dtype, f))
    assert dv.max() <= 1, f"value-only {kind} {dtype}: {int(dv.max())} ulp at x = {x32[int(dv.argmax())]!r}"


@pytest.mark.parametrize("dist", ["normal", "uniform20", "mix"])
@pytest.mark.parametrize("kind", KINDS)
def test_fp64_chain_on_fp32_inputs(host, kind, dist):
    """fp32 storage: y and f' inside the fp32 gate of the GPU tests, with the margin the design states (a rounding of
    the exact value for the three logistic kinds, 2.6 ulp for GELU-erf); the value-only form gives the same y."""
    x = W.draw(dist, (1 << 16) + 37, "f32", 5).numpy().copy()
    y, d, v, _ = host(kind, 2, x)
    stats = {}
    parity.check_forward_fp32(kind, x, y, d, stats)
    bound = 2.6 if kind == "gelu_erf" else 0.6
    assert stats["y_max_ulp"] <= bound and stats["d_gate_max"] <= bound, stats
    assert ulp.same_bits_or_both_nan(v, y, "f32").all()


@pytest.mark.parametrize("kind", KINDS)
def test_non_finite_and_saturated_inputs(host, kind):
    """What the boundary promises where the paper is silent: NaN -> NaN; +inf -> (+inf, 1); -inf -> (-0, 0);
    far beyond saturation f = x and f' = 1 on the right, both 0 on the left."""
    x = np.array([np.nan, np.inf, -np.inf, 1000.0, -1000.0], np.float32)
    for width in (0, 2):
        y, d, v, _ = host(kind, width, x)
        # the fp32 chain feeds a 16-bit store: one fp32 ulp of slack, which that store's rounding removes
        tol = 2.0 ** -22 if width == 0 else 0.0
        assert np.isnan(y[0]) and np.isnan(d[0]) and np.isnan(v[0])
        assert y[1] >= np.float32(3.0e38) and abs(d[1] - 1.0) <= tol                # 3.4e38 becomes inf in a 16-bit store
        assert y[2] == 0.0 and np.signbit(y[2]) and d[2] == 0.0
        assert abs(y[3] - 1000.0) <= 1000.0 * tol and abs(d[3] - 1.0) <= tol and abs(v[3] - 1000.0) <= 1000.0 * tol
        assert y[4] == 0.0 and d[4] == 0.0 and v[4] == 0.0


def _reference_primitives():
    """(name, value, derivative, domain) of each general-purpose primitive, from mpmath at 50 digits."""
    mp = pytest.importorskip("mpmath")
    mp.mp.dps = 50
    sig = lambda a: 1 / (1 + mp.exp(-a))
    return mp, [
        ("exp", mp.exp, mp.exp, (-80.0, 80.0)),
        ("log1p", mp.log1p, lambda a: 1 / (1 + a), (-0.99, 1.0e6)),
        ("tanh", mp.tanh, lambda a: mp.sech(a) ** 2, (-12.0, 12.0)),
        ("erf", mp.erf, lambda a: 2 / mp.sqrt(mp.pi) * mp.exp(-a * a), (-5.0, 5.0)),
        ("softplus", lambda a: mp.log1p(mp.exp(a)), sig, (-80.0, 80.0)),
        ("sigmoid", sig, lambda a: sig(a) * sig(-a), (-80.0, 80.0)),
        ("(1+tanh)/2", lambda a: sig(2 * a), lambda a: 2 * sig(2 * a) * sig(-2 * a), (-40.0, 40.0)),
        ("(1+erf)/2", lambda a: mp.erfc(-a) / 2, lambda a: mp.exp(-a * a) / mp.sqrt(mp.pi), (-9.0, 9.0)),
    ]


@pytest.mark.parametrize("wide", [False, True])
def test_general_purpose_primitives(host, wide):
    """Section III-A's primitive set as the sequences use it: value and tangent of each primitive at (x, 1) against
    50-digit arithmetic, relative to the result (these points avoid the zero of tanh and erf, where the value itself
    is tiny and the absolute error is what stays small).  fp32 arithmetic: 2^-18 with exact stand-ins for the
    approximate units; double: 2^-40."""
    mp, prims = _reference_primitives()
    rng = np.random.default_rng(7)
    tol = 2.0 ** -40 if wide else 2.0 ** -18
    # fp32 arithmetic forms exp(a) from one rounding of a log2(e): its relative error grows like |a| 2^-24, so the
    # fp32 primitives are compared where |a| is moderate
    narrow = {"exp": 8.0, "tanh": 8.0, "erf": 3.0, "softplus": 8.0, "sigmoid": 8.0, "(1+tanh)/2": 4.0, "(1+erf)/2": 3.0}
    for op, (name, f, df, (lo, hi)) in enumerate(prims):
        if not wide:
            lo, hi = (-narrow[name], narrow[name]) if name in narrow else (lo, 1.0e4)
        x = rng.uniform(lo, hi, 400)
        if not wide:
            x = x.astype(np.float32).astype(np.float64)
        x = x[np.abs(x) > 1e-3]
        v, t = host.primitive(op, wide, x)
        for xi, vi, ti in zip(x, v, t):
            fv, ft = f(mp.mpf(float(xi))), df(mp.mpf(float(xi)))
            # the fp32 erfc fit is built for 16-bit results: 2^-16 of erfc itself, i.e. 2^-15 with the operations around it
            tl = 2.0 ** -15 if (not wide and "erf" in name) else tol
            assert abs(mp.mpf(float(vi)) - fv) <= tl * abs(fv), (name, "value", xi, vi, float(fv))
            assert abs(mp.mpf(float(ti)) - ft) <= tl * abs(ft), (name, "tangent", xi, ti, float(ft))
