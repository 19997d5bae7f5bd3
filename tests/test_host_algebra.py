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

    def run(kind: str, width: int, x: np.ndarray):
        x = np.ascontiguousarray(x, np.float32)
        out = [np.empty_like(x) for _ in range(4)]
        lib.host_algebra(KINDS.index(kind), width, x.ctypes.data, *[o.ctypes.data for o in out], x.size)
        return out                                   # y, f', value-only y, gate

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
