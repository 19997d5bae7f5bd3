"""Pins for the CPU oracle: everything here checks ``oracle/`` against something
other than itself -- closed forms, invariants, 50-digit arithmetic on the
literal formulas of Table I, independent double-precision library routines
(torch CPU, scipy), exact rational arithmetic for the roundings.  No GPU.
"""
import math
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle

KINDS = ["gelu_erf", "gelu_tanh", "swish", "mish"]
GRID = [-80.0, -40.0, -20.0, -13.5, -10.0, -7.0, -5.0, -3.0, -2.0, -1.278, -1.19, -1.0, -0.752, -0.5,
        -0.1, -1e-3, -1e-8, 0.0, 1e-8, 1e-3, 0.1, 0.5, 1.0, 1.4142135623730951, 2.0, 3.0, 5.0, 7.0,
        10.0, 20.0, 40.0, 80.0]


# --------------------------------------------------------------------------- closed forms

def test_fixed_points_from_golden_file():
    path = os.path.join(os.path.dirname(__file__), "golden", "fixed_points.txt")
    rows = [l.split() for l in open(path) if l.strip() and not l.startswith("#")]
    assert len(rows) == 8
    for kind, x, what, val in rows:
        f, fp, _, _ = oracle.eval_point(kind, float(x))
        got = f if what == "f" else fp
        assert got == pytest.approx(float(val), abs=1e-16), (kind, what)


def test_mish_prime_at_zero_is_tanh_ln2():
    assert oracle.eval_point("mish", 0.0)[1] == pytest.approx(math.tanh(math.log(2.0)), abs=1e-16)


@pytest.mark.parametrize("kind", ["gelu_erf", "gelu_tanh", "swish"])
def test_reflection_symmetries(kind):
    # h(x) + h(-x) = 1 for Phi, sigmoid(2u) (u odd) and sigmoid, hence
    # f(x) - f(-x) = x and f'(x) + f'(-x) = 1.  Mish has no such symmetry.
    for x in [0.3, 0.7517915, 1.0, 1.2784645, 2.5, 4.0, 6.0, 9.0, 13.0]:
        f1, d1, h1, _ = oracle.eval_point(kind, x)
        f2, d2, h2, _ = oracle.eval_point(kind, -x)
        assert f1 - f2 == pytest.approx(x, rel=1e-15)
        assert d1 + d2 == pytest.approx(1.0, abs=2e-15)
        assert h1 + h2 == pytest.approx(1.0, abs=4e-16)


def test_mish_is_not_symmetric():
    d1 = oracle.eval_point("mish", 1.0)[1]
    d2 = oracle.eval_point("mish", -1.0)[1]
    assert abs(d1 + d2 - 1.0) > 0.05


@pytest.mark.parametrize("kind", KINDS)
def test_limits(kind):
    # f' -> 1, f - x -> 0 as x -> +inf;  f' -> 0-, f -> 0- as x -> -inf
    for x in [40.0, 80.0]:
        f, d, _, _ = oracle.eval_point(kind, x)
        assert d == pytest.approx(1.0, abs=1e-15)
        assert f == pytest.approx(x, rel=1e-15)
    for x in [-40.0, -80.0]:
        f, d, _, _ = oracle.eval_point(kind, x)
        assert -1e-15 < f <= 0.0 and -1e-15 < d <= 0.0
    # strictly negative (not flushed) where the true value is far above double underflow
    f, d, _, _ = oracle.eval_point(kind, -20.0)
    assert f < 0.0 and d < 0.0


@pytest.mark.parametrize("kind", KINDS)
def test_product_rule_split(kind):
    # f = x h and f' = h + x h' (Eq. 3 with v2 = x, v2' = 1)
    for x in GRID:
        f, d, h, xh = oracle.eval_point(kind, x)
        assert d == h + xh
        assert f == pytest.approx(x * h, rel=1e-15, abs=0.0)
        if x > 0:
            assert h > 0 and xh >= 0
        if x < 0:
            assert h >= 0 and xh <= 0      # Phi(-40) is below double underflow
            assert h > 0 or x <= -38


@pytest.mark.parametrize("kind", KINDS)
def test_central_differences_tie_fprime_to_f(kind):
    rng = np.random.default_rng(7)
    xs = np.concatenate([rng.uniform(-6, 6, 48), [-3, -1, -0.5, 0, 0.5, 1, 3]])
    for x in xs:
        h = 1e-5 * max(1.0, abs(x))
        # Richardson-extrapolated central difference: error O(h^4)
        f = lambda t: oracle.eval_point(kind, t)[0]
        d1 = (f(x + h) - f(x - h)) / (2 * h)
        d2 = (f(x + 2 * h) - f(x - 2 * h)) / (4 * h)
        fd = (4 * d1 - d2) / 3
        assert oracle.eval_point(kind, x)[1] == pytest.approx(fd, rel=1e-9, abs=2e-10)


def test_gelu_erf_extrema_of_fprime_at_sqrt2():
    # f'' = phi(x) (2 - x^2): f' has its maximum at +sqrt2 and minimum at -sqrt2,
    # and by the reflection symmetry the two values sum to 1.
    r = math.sqrt(2.0)
    d = lambda t: oracle.eval_point("gelu_erf", t)[1]
    assert d(r) > d(r - 1e-4) and d(r) > d(r + 1e-4)
    assert d(-r) < d(-r - 1e-4) and d(-r) < d(-r + 1e-4)
    assert d(r) == pytest.approx(1.1289041451851548, rel=1e-14)   # Phi(sqrt2) + sqrt2 phi(sqrt2)
    assert d(r) + d(-r) == pytest.approx(1.0, abs=1e-15)


# --------------------------------------------------------------------------- 50-digit arithmetic

def _mp_functions():
    mp = pytest.importorskip("mpmath")
    mp.mp.dps = 50
    c = mp.sqrt(2 / mp.pi)
    a = mp.mpf(0.044715)        # the double the oracle uses for Table I's constant
    fs = {
        # literal formulas: Table I (GELU-tanh, Mish, Swish) and x Phi(x)
        "gelu_erf": lambda x: x * (1 + mp.erf(x / mp.sqrt(2))) / 2,
        "gelu_tanh": lambda x: x * (1 + mp.tanh(c * (x + a * x ** 3))) / 2,
        "swish": lambda x: x / (1 + mp.exp(-x)),
        "mish": lambda x: x * mp.tanh(mp.log(1 + mp.exp(x))),
    }
    return mp, fs


@pytest.mark.parametrize("kind", KINDS)
def test_against_50_digit_literal_formulas(kind):
    mp, fs = _mp_functions()
    f = fs[kind]
    rng = np.random.default_rng(11)
    xs = GRID + list(rng.normal(0, 1.5, 40)) + list(rng.uniform(-20, 20, 40))
    for x in xs:
        # the literal 1+tanh(u), 1+erf(z) lose as many digits as the result is small
        # (1e-15921 for GELU-tanh at x = -80): carry 50 digits beyond that
        lost = {"gelu_erf": x * x / 2, "gelu_tanh": 1.6 * abs(x + 0.044715 * x ** 3)}.get(kind, abs(x)) / math.log(10)
        mp.mp.dps = 50 + int(lost)
        xm = mp.mpf(x)
        fv = f(xm)
        dv = mp.diff(f, xm)
        of, od, oh, oxh = oracle.eval_point(kind, x)
        scale = abs(oh) + abs(oxh)
        if fv == 0:
            assert of == 0
        elif abs(fv) > mp.mpf(10) ** -300:
            assert abs((mp.mpf(of) - fv) / fv) < 2e-13, (kind, x, of, fv)
        if scale > 1e-300:
            assert abs(mp.mpf(od) - dv) < 2e-13 * scale, (kind, x, od, dv)
    mp.mp.dps = 50


@pytest.mark.parametrize("kind,guess", [("gelu_erf", -0.75), ("gelu_tanh", -0.75), ("swish", -1.28), ("mish", -1.19)])
def test_fprime_changes_sign_at_the_true_root(kind, guess):
    mp, fs = _mp_functions()
    f = fs[kind]
    root = mp.findroot(lambda t: mp.diff(f, t), guess)
    r = float(root)
    # the two addends are ~0.3 each, so the double sum is good to ~1e-16 absolute:
    # 1e-12 away from the root the sign (|f'| ~ 5e-13) is already certain
    below = oracle.eval_point(kind, r - 1e-12)[1]
    above = oracle.eval_point(kind, r + 1e-12)[1]
    assert below < 0.0 < above
    # slope there: f'(x) ~ f''(r) (x - r); compare with the 50-digit value a little off the root
    x = r + 1e-6
    assert oracle.eval_point(kind, x)[1] == pytest.approx(float(mp.diff(f, mp.mpf(x))), rel=1e-8)


# --------------------------------------------------------------------------- independent libraries

def test_against_torch_cpu_double_and_autograd():
    torch = pytest.importorskip("torch")
    F = torch.nn.functional
    fns = {
        "gelu_erf": lambda t: F.gelu(t),
        "gelu_tanh": lambda t: F.gelu(t, approximate="tanh"),
        "swish": lambda t: F.silu(t),
        "mish": lambda t: F.mish(t),
    }
    g = torch.Generator().manual_seed(3)
    x = torch.cat([torch.randn(4000, generator=g, dtype=torch.float64) * 1.5,
                   torch.linspace(-6, 6, 1001, dtype=torch.float64)])
    xn = x.numpy().astype(np.float32)            # the oracle takes stored tensors
    xt = torch.from_numpy(xn.astype(np.float64)).requires_grad_(True)
    for kind, fn in fns.items():
        y = fn(xt)
        (d,) = torch.autograd.grad(y.sum(), xt)
        of, od = oracle.forward(kind, "f32", xn)
        # the framework formulas are the literal ones: absolute agreement only
        np.testing.assert_allclose(of, y.detach().numpy(), rtol=0, atol=3e-15)
        np.testing.assert_allclose(od, d.numpy(), rtol=0, atol=3e-15)


def test_against_scipy_special():
    sp = pytest.importorskip("scipy.special")
    x = np.linspace(-30, 30, 2401).astype(np.float32)
    xd = x.astype(np.float64)
    f, d = oracle.forward("gelu_erf", "f32", x)
    np.testing.assert_allclose(f, xd * sp.ndtr(xd), rtol=5e-14, atol=0)
    f, d = oracle.forward("swish", "f32", x)
    s = sp.expit(xd)
    np.testing.assert_allclose(f, xd * s, rtol=5e-15, atol=0)
    np.testing.assert_allclose(d, s + xd * s * sp.expit(-xd), rtol=0, atol=2e-16 * 30)  # Table II


# --------------------------------------------------------------------------- storage formats

def _exact_round(v: float, pbits: int, emin: int, emax: int) -> float:
    """Nearest value of the format, ties to even, by exact rational arithmetic."""
    if v == 0.0:
        return v
    a = Fraction(abs(v))
    e = math.floor(math.log2(a))
    while Fraction(2) ** e > a:
        e -= 1
    while Fraction(2) ** (e + 1) <= a:
        e += 1
    q = max(e, emin) - (pbits - 1)
    k = a / Fraction(2) ** q
    lo = k.numerator // k.denominator
    rem = k - lo
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and lo % 2 == 1):
        lo += 1
    out = Fraction(lo) * Fraction(2) ** q
    if out >= Fraction(2) ** (emax + 1):
        return math.copysign(math.inf, v)
    return math.copysign(float(out), v)


def _interesting_doubles(rng, n):
    base = np.concatenate([
        rng.normal(0, 1, n), rng.uniform(-80, 80, n),
        np.exp(rng.uniform(np.log(1e-46), np.log(1e39), n)) * rng.choice([-1, 1], n),
    ])
    return base


@pytest.mark.parametrize("dtype,pbits,emin,emax", [("bf16", 8, -126, 127), ("f16", 11, -14, 15)])
def test_rounding_against_exact_rational_arithmetic(dtype, pbits, emin, emax):
    rng = np.random.default_rng(5)
    v = _interesting_doubles(rng, 400)
    # exact ties and their neighbours in double
    ties = []
    for m in [1, 3, 5, 255, 256, 257, 1023, 2047]:
        for e in [-140, -133, -130, -126, -30, -24, -20, -14, -1, 0, 7, 15, 16, 100, 127]:
            t = (2 * m + 1) * 2.0 ** (e - pbits)
            ties += [t, np.nextafter(t, 0), np.nextafter(t, np.inf), -t]
    v = np.concatenate([v, np.array(ties)])
    got = oracle.widen(dtype, oracle.round_to(dtype, v))
    want = np.array([_exact_round(float(t), pbits, emin, emax) for t in v])
    np.testing.assert_array_equal(got, want)


def test_rounding_against_numpy_conversions():
    rng = np.random.default_rng(6)
    v = _interesting_doubles(rng, 50000)
    with np.errstate(over="ignore"):
        np.testing.assert_array_equal(oracle.round_to("f16", v).view(np.float16), v.astype(np.float16))
        np.testing.assert_array_equal(oracle.round_to("f32", v), v.astype(np.float32))


def test_widen_every_16_bit_pattern():
    torch = pytest.importorskip("torch")
    bits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    np.testing.assert_array_equal(oracle.widen("f16", bits), bits.view(np.float16).astype(np.float64))
    bf = torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16).to(torch.float64).numpy()
    np.testing.assert_array_equal(oracle.widen("bf16", bits), bf)
    # round-trip: every finite 16-bit value is a fixed point of the rounding
    for dt in ("f16", "bf16"):
        w = oracle.widen(dt, bits)
        fin = np.isfinite(w)
        np.testing.assert_array_equal(oracle.round_to(dt, w[fin]), bits[fin])


# --------------------------------------------------------------------------- backward (Eq. 4)

def test_backward_is_the_exactly_rounded_product():
    rng = np.random.default_rng(9)
    g32 = rng.normal(0, 1, 3000).astype(np.float32)
    d32 = rng.normal(0.5, 0.4, 3000).astype(np.float32)
    got = oracle.backward("f32", g32, d32)
    want = np.array([float(np.float32(float(Fraction(float(a)) * Fraction(float(b))))) for a, b in zip(g32[:300], d32[:300])],
                    dtype=np.float32)
    np.testing.assert_array_equal(got[:300], want)
    np.testing.assert_array_equal(got, (g32.astype(np.float64) * d32.astype(np.float64)).astype(np.float32))
    for dt, pb, emin, emax in (("bf16", 8, -126, 127), ("f16", 11, -14, 15)):
        g = oracle.round_to(dt, rng.normal(0, 1e-2, 500))
        d = oracle.round_to(dt, rng.normal(0.5, 0.4, 500))
        gw, dw = oracle.widen(dt, g), oracle.widen(dt, d)
        want = np.array([_exact_round(float(Fraction(float(a)) * Fraction(float(b))), pb, emin, emax) for a, b in zip(gw, dw)])
        np.testing.assert_array_equal(oracle.widen(dt, oracle.backward(dt, g, d)), want)
    # hand values: 3 * 0.5 = 1.5 ; (-2) * 0.25 = -0.5
    out = oracle.backward("f32", np.array([3.0, -2.0], np.float32), np.array([0.5, 0.25], np.float32))
    assert out.tolist() == [1.5, -0.5]


def test_forward_backward_matches_its_parts():
    rng = np.random.default_rng(10)
    for dt in ("f32", "bf16", "f16"):
        x = oracle.round_to(dt, rng.normal(0, 1.5, 4097))
        g = oracle.round_to(dt, rng.normal(0, 1, 4097))
        for kind in KINDS:
            y, d, gin = oracle.forward_backward(kind, dt, x, g)
            f, fp = oracle.forward(kind, dt, x)
            np.testing.assert_array_equal(y, oracle.round_to(dt, f))
            np.testing.assert_array_equal(d, oracle.round_to(dt, fp))
            np.testing.assert_array_equal(gin, oracle.backward(dt, g, d))


def test_threads_do_not_change_results():
    rng = np.random.default_rng(12)
    x = rng.normal(0, 1, 100003).astype(np.float32)
    oracle.set_threads(1)
    a = oracle.forward("mish", "f32", x)
    oracle.set_threads(max(2, min(4, oracle.max_threads())))
    b = oracle.forward("mish", "f32", x)
    oracle.set_threads(1)
    np.testing.assert_array_equal(a[0], b[0])
    np.testing.assert_array_equal(a[1], b[1])


def test_bad_arguments_are_rejected():
    with pytest.raises(ValueError):
        oracle.eval_point(7, 0.0)
    with pytest.raises(TypeError):
        oracle.forward("swish", "bf16", np.zeros(4, np.float32))


# ----------------------------------------------------------------------------- stored 20-digit values

def _closed_form_rows():
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "closed_forms.txt")
    rows = []
    with open(path) as fh:
        for line in fh:
            line = line.strip()
            if line and not line.startswith("#"):
                tag, kind, x, f, fp = line.split()
                rows.append((tag, kind, float(x), float(f), float(fp)))
    return rows


def test_stored_closed_form_values():
    """f and f' against the stored 50-digit evaluation of the literal definitions (Table I; x Phi(x)): the grid
    into both tails, the stationary points of f', the sign change of f'.  No optional import: these pins hold on
    any box.  f to 1e-13 relative; f' to 1e-13 of |h| + |x h'| (the size of the two terms it is the sum of)."""
    rows = _closed_form_rows()
    assert len(rows) == 54
    assert {r[0] for r in rows} == {"table", "extremum", "root"}
    for tag, kind, x, f_ref, fp_ref in rows:
        f, fp, h, xh = oracle.eval_point(kind, x)
        assert abs(f - f_ref) <= 1e-13 * abs(f_ref), (tag, kind, x, f, f_ref)
        scale = abs(h) + abs(xh)
        assert abs(fp - fp_ref) <= 1e-13 * scale, (tag, kind, x, fp, fp_ref)


def test_stored_roots_and_extrema_have_their_closed_form_properties():
    rows = _closed_form_rows()
    ext = {(k, x > 0): (x, fp) for tag, k, x, f, fp in rows if tag == "extremum"}
    # erf form: f'' = phi(x) (2 - x^2), so the stationary points of f' are +-sqrt(2)
    assert abs(ext[("gelu_erf", True)][0] - math.sqrt(2.0)) < 1e-15 and abs(ext[("gelu_erf", False)][0] + math.sqrt(2.0)) < 1e-15
    # the three kinds with h(x) + h(-x) = 1 have f'(x) + f'(-x) = 1 at their mirrored stationary points
    for kind in ("gelu_erf", "gelu_tanh", "swish"):
        (xp, fpp), (xn, fpn) = ext[(kind, True)], ext[(kind, False)]
        assert abs(xp + xn) < 1e-15 and abs(fpp + fpn - 1.0) < 1e-15
    # Swish: at the sign change of f', x s = x + 1
    (xr, fr), = [(x, f) for tag, k, x, f, fp in rows if tag == "root" and k == "swish"]
    assert abs(fr - (xr + 1.0)) < 1e-15
    # a stationary point is a maximum (x > 0) or minimum (x < 0) of the oracle's f' too
    for (kind, pos), (x, fp) in ext.items():
        for dx in (-1e-3, 1e-3):
            other = oracle.eval_point(kind, x + dx)[1]
            assert (other < fp) if pos else (other > fp), (kind, x, dx)
