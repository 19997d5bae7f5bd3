"""Pins for the fp64 FAD-sequence oracle: the four activations written as programs must agree
with the closed-form oracle (itself pinned in test_oracle_pins.py); every primitive's
derivative is tied to its value by central differences; hand-computed values; a two-result
sequence against closed forms; malformed programs are refused.  No GPU."""
import math

import numpy as np
import pytest

import oracle
from paper_2209_10778_b200 import sequence

XS = np.concatenate([np.linspace(-12, 12, 481), [-40.0, -20.0, 20.0, 40.0, 1e-8, -1e-8, 0.0]])


@pytest.mark.parametrize("kind", ["swish", "mish", "gelu_tanh", "gelu_erf"])
def test_programs_of_the_four_activations_match_the_closed_forms(kind):
    prog = sequence.PROGRAMS[kind]()
    x32 = XS.astype(np.float32)
    y, d = oracle.seq_forward(prog.ops, x32.astype(np.float64), 1)
    f, fp, cond = oracle.forward(kind, "f32", x32, want_cond=True)
    np.testing.assert_allclose(y[0], f, rtol=2e-13, atol=1e-300)
    assert (np.abs(d[0] - fp) <= 2e-13 * np.maximum(cond, 1e-300) + 1e-300).all()


def test_literal_gelu_tanh_program_is_the_same_function_where_it_does_not_cancel():
    x = np.linspace(-4, 8, 241)
    y1, d1 = oracle.seq_forward(sequence.gelu_tanh_program().ops, x, 1)
    y2, d2 = oracle.seq_forward(sequence.gelu_tanh_literal_program().ops, x, 1)
    np.testing.assert_allclose(y1, y2, rtol=0, atol=2e-15)
    np.testing.assert_allclose(d1, d2, rtol=0, atol=4e-15)


@pytest.mark.parametrize("name,lo,hi", [("exp", -5, 5), ("log1p", -0.9, 5), ("tanh", -4, 4), ("erf", -3, 3), ("softplus", -6, 6),
                                       ("sigmoid", -6, 6), ("half_one_plus_tanh", -3, 3), ("half_one_plus_erf", -3, 3)])
def test_each_primitive_derivative_by_central_differences(name, lo, hi):
    prog = [(name, 0, 0, 1, 0.0), ("out", 1, 1, 0, 0.0)]
    x = np.linspace(lo, hi, 41)
    h = 1e-5
    y, d = oracle.seq_forward(prog, x, 1)
    yp, _ = oracle.seq_forward(prog, x + h, 1)
    ym, _ = oracle.seq_forward(prog, x - h, 1)
    yp2, _ = oracle.seq_forward(prog, x + 2 * h, 1)
    ym2, _ = oracle.seq_forward(prog, x - 2 * h, 1)
    fd = (4 * (yp - ym) / (2 * h) - (yp2 - ym2) / (4 * h)) / 3
    np.testing.assert_allclose(d[0], fd[0], rtol=2e-9, atol=2e-10)
    ref = {"exp": math.exp, "log1p": math.log1p, "tanh": math.tanh, "erf": math.erf,
           "softplus": lambda v: math.log1p(math.exp(v)), "sigmoid": lambda v: 1 / (1 + math.exp(-v)),
           "half_one_plus_tanh": lambda v: 0.5 * (1 + math.tanh(v)), "half_one_plus_erf": lambda v: 0.5 * (1 + math.erf(v))}[name]
    np.testing.assert_allclose(y[0], [ref(v) for v in x], rtol=1e-14, atol=1e-16)


def test_linear_ops_product_rule_and_two_results_by_hand():
    # r1 = 3x ; r2 = 2 + r1 ; r3 = r1 * r2 = 9x^2 + 6x ; r4 = r3 + x ; results: r3 (18x + 6) and r4 (18x + 7)
    prog = [("scale", 0, 0, 1, 3.0), ("add_const", 1, 1, 2, 2.0), ("mul", 1, 2, 3, 0.0), ("add", 3, 0, 4, 0.0),
            ("out", 3, 3, 0, 0.0), ("out", 4, 4, 1, 0.0)]
    x = np.array([-2.0, 0.0, 0.5, 3.0])
    y, d = oracle.seq_forward(prog, x, 2)
    np.testing.assert_array_equal(y[0], 9 * x * x + 6 * x)
    np.testing.assert_array_equal(d[0], 18 * x + 6)
    np.testing.assert_array_equal(y[1], 9 * x * x + 7 * x)
    np.testing.assert_array_equal(d[1], 18 * x + 7)
    g = np.array([[1.0, 2.0, -1.0, 0.5], [3.0, -2.0, 1.0, 0.25]])
    s, sa = oracle.seq_backward(g, d)
    np.testing.assert_array_equal(s, g[0] * d[0] + g[1] * d[1])
    np.testing.assert_array_equal(sa, np.abs(g[0] * d[0]) + np.abs(g[1] * d[1]))


def test_malformed_programs_are_refused():
    x = np.zeros(3)
    with pytest.raises(ValueError):
        oracle.seq_forward([("exp", 3, 3, 1, 0.0), ("out", 1, 1, 0, 0.0)], x, 1)      # reads an unwritten register
    with pytest.raises(ValueError):
        oracle.seq_forward([("exp", 0, 0, 1, 0.0), ("out", 1, 1, 2, 0.0)], x, 1)      # result slot out of range
    with pytest.raises(ValueError):
        oracle.seq_forward([("exp", 0, 0, 0, 0.0), ("out", 0, 0, 0, 0.0)], x, 1)      # writes the source register
