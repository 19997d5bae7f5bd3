"""Pins for the bias-fused part of the CPU oracle (``oracle/nfad_bias_oracle.c``): every check compares it with
something other than itself -- double-precision library routines (scipy, torch CPU) or 50-digit arithmetic evaluated
at a pre-activation formed independently with numpy's fp32 addition, on NON-square grids so that a transposed or
dropped index fails; a tie case that tells one fp32 rounding of the sum from none; exact rational column sums.
No GPU.
"""
import math
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle

KINDS = ["gelu_erf", "gelu_tanh", "swish", "mish"]
ROWS, COLS = 7, 5


def _bf16_bits(a32: np.ndarray) -> np.ndarray:
    return torch.from_numpy(np.asarray(a32, np.float32)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)


def _f16_bits(a32: np.ndarray) -> np.ndarray:
    return np.asarray(a32, np.float32).astype(np.float16).view(np.uint16)


def _bits_to_f64(bits: np.ndarray, dtype: str) -> np.ndarray:
    if dtype == "f32":
        return bits.astype(np.float64)
    if dtype == "f16":
        return bits.view(np.float16).astype(np.float64)
    return torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16).to(torch.float64).numpy()


def _stored(a32: np.ndarray, dtype: str) -> np.ndarray:
    return {"f32": lambda a: np.asarray(a, np.float32), "bf16": _bf16_bits, "f16": _f16_bits}[dtype](a32)


def _grid(dtype: str):
    rng = np.random.default_rng(11)
    x = _stored(rng.normal(0.0, 2.0, ROWS * COLS), dtype)
    b = _stored(np.array([-3.0, -0.5, 0.0, 0.25, 4.0]) + rng.normal(0.0, 0.01, COLS), dtype)
    z = (_bits_to_f64(x, dtype).astype(np.float32).reshape(ROWS, COLS)
         + _bits_to_f64(b, dtype).astype(np.float32)[None, :]).astype(np.float64)   # numpy's own fp32 addition
    return x, b, z.reshape(-1)


# --------------------------------------------------------------------------- forward

@pytest.mark.parametrize("dtype", ["f32", "bf16", "f16"])
def test_forward_gelu_erf_against_scipy_at_the_fp32_sum(dtype):
    from scipy.special import ndtr
    x, b, z = _grid(dtype)
    f, fp, zz = oracle.bias_forward("gelu_erf", dtype, x, b, ROWS, COLS)
    assert np.array_equal(zz, z)
    assert f == pytest.approx(z * ndtr(z), rel=4e-15, abs=1e-300)
    phi = np.exp(-0.5 * z * z) / math.sqrt(2.0 * math.pi)
    assert fp == pytest.approx(ndtr(z) + z * phi, rel=1e-13, abs=1e-16)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_forward_swish_against_torch_double(dtype):
    x, b, z = _grid(dtype)
    zt = torch.from_numpy(z).requires_grad_(True)
    y = zt * torch.sigmoid(zt)
    y.sum().backward()
    f, fp, _ = oracle.bias_forward("swish", dtype, x, b, ROWS, COLS)
    assert f == pytest.approx(y.detach().numpy(), rel=1e-14, abs=1e-300)
    assert fp == pytest.approx(zt.grad.numpy(), rel=1e-13, abs=1e-15)


@pytest.mark.parametrize("kind", ["gelu_tanh", "mish"])
def test_forward_table_one_formulas_in_50_digits(kind):
    import mpmath as mp
    mp.mp.dps = 50
    x, b, z = _grid("f32")
    f, fp, _ = oracle.bias_forward(kind, "f32", x, b, ROWS, COLS)

    def fn(t):
        if kind == "mish":
            return t * mp.tanh(mp.log(1 + mp.exp(t)))
        u = mp.sqrt(2 / mp.pi) * (t + mp.mpf(0.044715) * t ** 3)
        return t * (1 + mp.tanh(u)) / 2

    for i in range(0, ROWS * COLS, 3):
        t = mp.mpf(float(z[i]))
        assert f[i] == pytest.approx(float(fn(t)), rel=1e-14, abs=1e-300)
        assert fp[i] == pytest.approx(float(mp.diff(fn, t)), rel=1e-12, abs=1e-15)


def test_bias_follows_the_column_not_the_row():
    # x = 0 everywhere: the result is a function of the column alone
    b = np.array([-2.0, -1.0, 0.0, 1.0, 2.0], np.float32)
    f, fp, z = oracle.bias_forward("swish", "f32", np.zeros(ROWS * COLS, np.float32), b, ROWS, COLS)
    want = b.astype(np.float64) / (1.0 + np.exp(-b.astype(np.float64)))
    assert f.reshape(ROWS, COLS) == pytest.approx(np.tile(want, (ROWS, 1)), rel=1e-15)
    assert np.array_equal(z.reshape(ROWS, COLS)[3], b.astype(np.float64))


def test_sum_is_rounded_once_to_fp32():
    # 1 + 2^-24 is a tie in fp32 and goes to the even neighbour 1; 1 + 3 * 2^-25 goes up to 1 + 2^-23.
    # All four operands are exact in bf16, so an unrounded sum would be visible in double.
    x = _bf16_bits(np.array([1.0, 1.0], np.float32))
    b = _bf16_bits(np.array([2.0 ** -24, 3 * 2.0 ** -25], np.float32))
    f, fp, z = oracle.bias_forward("swish", "bf16", x, b, 1, 2)
    assert z[0] == 1.0 and z[1] == 1.0 + 2.0 ** -23
    s1 = 1.0 / (1.0 + math.exp(-1.0))
    assert f[0] == pytest.approx(s1, rel=1e-15)
    assert abs(f[0] - (1.0 + 2.0 ** -24) / (1.0 + math.exp(-(1.0 + 2.0 ** -24)))) > 1e-9


def test_zero_bias_is_the_plain_activation_value():
    # closed form at z = x: GELU-erf(1) = Phi(1), Swish(0) = 0 with slope 1/2
    x = np.array([1.0, 0.0, -1.0, 2.0, 0.5, 3.0], np.float32)
    f, fp, _ = oracle.bias_forward("gelu_erf", "f32", x, np.zeros(3, np.float32), 2, 3)
    assert f[0] == pytest.approx(0.5 * math.erfc(-1.0 / math.sqrt(2.0)), rel=1e-15)
    assert fp[1] == 0.5


# --------------------------------------------------------------------------- backward

def _exact_rounding(value: Fraction, dtype: str) -> float:
    """Round an exact rational to the storage type by trying the two neighbouring stored values (normal range)."""
    p = {"f32": 24, "bf16": 8, "f16": 11}[dtype]
    if value == 0:
        return 0.0
    sign = -1 if value < 0 else 1
    a = abs(value)
    e = math.floor(math.log2(float(a)))
    while Fraction(2) ** e > a:
        e -= 1
    while Fraction(2) ** (e + 1) <= a:
        e += 1
    q = Fraction(2) ** (e - p + 1)
    k = a / q
    lo = k.numerator // k.denominator
    rem = k - lo
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and lo % 2 == 1):
        lo += 1
    return sign * float(lo * q)


@pytest.mark.parametrize("dtype", ["f32", "bf16", "f16"])
def test_backward_against_exact_rational_arithmetic(dtype):
    rng = np.random.default_rng(5)
    g = _stored(rng.normal(0.0, 1.0, ROWS * COLS), dtype)
    d = _stored(rng.uniform(-0.2, 1.1, ROWS * COLS), dtype)
    gin, gb, gb_abs = oracle.bias_backward(dtype, g, d, ROWS, COLS)
    gv, dv = _bits_to_f64(g, dtype), _bits_to_f64(d, dtype)
    want = np.array([_exact_rounding(Fraction(float(a)) * Fraction(float(c)), dtype) for a, c in zip(gv, dv)])
    got = _bits_to_f64(gin, dtype)
    assert np.array_equal(got, want)
    cols = [sum(Fraction(float(v)) for v in want.reshape(ROWS, COLS)[:, c]) for c in range(COLS)]
    assert gb == pytest.approx([float(c) for c in cols], rel=1e-15, abs=1e-18)
    cols_abs = [sum(abs(Fraction(float(v))) for v in want.reshape(ROWS, COLS)[:, c]) for c in range(COLS)]
    assert gb_abs == pytest.approx([float(c) for c in cols_abs], rel=1e-15)


def test_backward_closed_form_column_sums():
    # grad_out = 1, f' = 2^c in column c: grad_bias[c] = rows * 2^c, exactly
    rows, cols = 9, 4
    d = np.tile(2.0 ** np.arange(cols), (rows, 1)).astype(np.float32).reshape(-1)
    gin, gb, gb_abs = oracle.bias_backward("f32", np.ones(rows * cols, np.float32), d, rows, cols)
    assert np.array_equal(gb, rows * 2.0 ** np.arange(cols))
    assert np.array_equal(gin, d)
    # a sign pattern that cancels: +1, -1, +1, ... down each column leaves one term
    g = np.tile(np.where(np.arange(rows) % 2 == 0, 1.0, -1.0)[:, None], (1, cols)).astype(np.float32).reshape(-1)
    _, gb, gb_abs = oracle.bias_backward("f32", g, d, rows, cols)
    assert np.array_equal(gb, 2.0 ** np.arange(cols))
    assert np.array_equal(gb_abs, rows * 2.0 ** np.arange(cols))


def test_backward_sums_the_rounded_products():
    # bf16: 1.0078125 * 1.0078125 = 1.01568603515625 rounds to 1.015625; three rows give 3.046875, not 3.04705810546875
    v = _bf16_bits(np.full(3, 1.0078125, np.float32))
    gin, gb, _ = oracle.bias_backward("bf16", v, v, 3, 1)
    assert _bits_to_f64(gin, "bf16")[0] == 1.015625
    assert gb[0] == 3.046875


def test_empty_shapes():
    gin, gb, _ = oracle.bias_backward("f32", np.empty(0, np.float32), np.empty(0, np.float32), 0, 3)
    assert gin.size == 0 and np.array_equal(gb, np.zeros(3))
    f, fp, z = oracle.bias_forward("mish", "f32", np.empty(0, np.float32), np.zeros(3, np.float32), 0, 3)
    assert f.size == 0
