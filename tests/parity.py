"""Shared parity checks: CUDA results against the fp64 oracle on the same arrays.

Tolerances (stated once, used by every GPU test):
  fp32 y      : |got - o| <= 4 ulp32(o)                      (normal-range o)
  fp32 f'     : x >= 0: |got - o| <= 4 ulp32(o)
                x <  0: |got - o| <= 4 ulp32(T), T = |h| + |x h'|, because f' = h + x h'
                        is there a difference of two fp32-evaluated terms and changes sign;
                        no fp32-internal evaluation can hold 4 ulp of a result that is ~0
  fp32, |o| < 2^-126 (subnormal result): |got - o| <= 4 * 2^-149
  bf16 / fp16 : |ord(got) - ord(RN(o))| <= 1, RN = one rounding from fp64
  backward    : the same bits as RN(fp64(g) * fp64(f'_saved)), the sign of a zero included (any NaN for a NaN),
                f'_saved being the GPU's own tensor
"""
from __future__ import annotations

import numpy as np
import torch

import oracle
import ulp
from paper_2209_10778_b200 import binding as nfad
from paper_2209_10778_b200 import workloads as W

FP32_ULPS = 4.0
SUBNORMAL_SLACK = 4 * 2.0 ** -149
MIN_NORMAL = 2.0 ** -126


def gpu_forward(kind: str, x: torch.Tensor):
    y = torch.empty_like(x)
    d = torch.empty_like(x)
    nfad.nfad_act_forward(kind, x, y, d)
    return y, d


def gpu_backward(kind: str, g: torch.Tensor, d: torch.Tensor):
    gin = torch.empty_like(g)
    nfad.nfad_act_backward(kind, g, d, gin)
    return gin


def _fail_report(name, bad, x, got, want, err):
    idx = np.flatnonzero(bad)
    worst = idx[np.argmax(err[idx])]
    return (f"{name}: {idx.size} of {bad.size} elements out of tolerance; worst at i={worst}: x={x[worst]!r} "
            f"got={got[worst]!r} oracle={want[worst]!r} err={err[worst]:.3f}")


def check_forward_fp32(kind: str, x_raw: np.ndarray, y: np.ndarray, d: np.ndarray, stats: dict | None = None):
    f, fp, cond = oracle.forward(kind, "f32", x_raw, want_cond=True)
    check_forward_fp32_values(kind, x_raw, f, fp, cond, y, d, stats)


def check_forward_fp32_values(kind: str, x_raw: np.ndarray, f: np.ndarray, fp: np.ndarray, cond: np.ndarray, y: np.ndarray,
                              d: np.ndarray, stats: dict | None = None):
    """x_raw: the point the activation was evaluated at; f, fp, cond: the oracle's values there."""
    xd = x_raw.astype(np.float64)
    # value
    ey = ulp.err_strict32(y, f)
    sub = np.abs(f) < MIN_NORMAL
    bad = np.where(sub, np.abs(y.astype(np.float64) - f) > SUBNORMAL_SLACK, ey > FP32_ULPS) | ~np.isfinite(y)
    assert not bad.any(), _fail_report(f"{kind} fp32 y", bad, x_raw, y, f, ey)
    # derivative
    es = ulp.err_strict32(d, fp)
    ec = ulp.err_scaled32(d, fp, cond)
    gate = np.where(xd >= 0, es, ec)
    subd = np.abs(fp) < MIN_NORMAL
    # (a subnormal f' next to its sign change still has normal-sized addends: scaled gate)
    tail = subd & (cond < 2.0 ** -100)
    badd = np.where(tail, np.abs(d.astype(np.float64) - fp) > SUBNORMAL_SLACK, gate > FP32_ULPS) | ~np.isfinite(d)
    assert not badd.any(), _fail_report(f"{kind} fp32 f'", badd, x_raw, d, fp, gate)
    if stats is not None:
        neg = xd < 0
        stats.update(
            y_max_ulp=float(ey[~sub].max(initial=0.0)),
            d_gate_max=float(gate[~subd].max(initial=0.0)),
            d_strict_max=float(es[~subd].max(initial=0.0)),
            d_strict_p999=float(np.quantile(es[neg & ~subd], 0.999)) if (neg & ~subd).any() else 0.0,
            d_only_scaled=int(((es > FP32_ULPS) & ~subd).sum()),
        )


def check_forward_16(kind: str, dtype: str, x_raw: np.ndarray, y_bits: np.ndarray, d_bits: np.ndarray,
                     stats: dict | None = None):
    f, fp = oracle.forward(kind, dtype, x_raw)
    check_forward_16_values(kind, dtype, oracle.widen(dtype, x_raw), f, fp, y_bits, d_bits, stats)


def check_forward_16_values(kind: str, dtype: str, xw: np.ndarray, f: np.ndarray, fp: np.ndarray, y_bits: np.ndarray,
                            d_bits: np.ndarray, stats: dict | None = None):
    """xw: the point the activation was evaluated at (fp64); f, fp: the oracle's unrounded values there."""
    want_y = oracle.round_to(dtype, f)
    want_d = oracle.round_to(dtype, fp)
    dy = ulp.ulp_distance16(y_bits, want_y)
    dd = ulp.ulp_distance16(d_bits, want_d)
    bad = (dy > 1) | ulp.is_nan16(y_bits, dtype)
    assert not bad.any(), _fail_report(f"{kind} {dtype} y", bad, xw, oracle.widen(dtype, y_bits), f, dy.astype(np.float64))
    badd = (dd > 1) | ulp.is_nan16(d_bits, dtype)
    assert not badd.any(), _fail_report(f"{kind} {dtype} f'", badd, xw, oracle.widen(dtype, d_bits), fp, dd.astype(np.float64))
    if stats is not None:
        stats.update(y_off_by_one=int((dy == 1).sum()), d_off_by_one=int((dd == 1).sum()))


def check_backward(dtype: str, g_raw: np.ndarray, d_raw: np.ndarray, gin_raw: np.ndarray):
    want = oracle.backward(dtype, g_raw, d_raw)
    same = ulp.same_bits_or_both_nan(gin_raw, want, dtype)
    if not same.all():
        i = int(np.flatnonzero(~same)[0])
        raise AssertionError(f"backward {dtype}: {int((~same).sum())} mismatches; first at i={i}: "
                             f"g={oracle.widen(dtype, g_raw[i:i+1])[0]!r} f'={oracle.widen(dtype, d_raw[i:i+1])[0]!r} "
                             f"got={oracle.widen(dtype, gin_raw[i:i+1])[0]!r} want={oracle.widen(dtype, want[i:i+1])[0]!r}")


def full_check(kind: str, dtype: str, x: torch.Tensor, g: torch.Tensor, stats: dict | None = None):
    """Forward + backward through the C-ABI on CUDA tensors x, g; compare everything with the oracle."""
    y, d = gpu_forward(kind, x)
    gin = gpu_backward(kind, g, d)
    torch.cuda.synchronize()
    x_raw, g_raw = W.raw_numpy(x), W.raw_numpy(g)
    y_raw, d_raw, gin_raw = W.raw_numpy(y), W.raw_numpy(d), W.raw_numpy(gin)
    if dtype == "f32":
        check_forward_fp32(kind, x_raw, y_raw, d_raw, stats)
    else:
        check_forward_16(kind, dtype, x_raw, y_raw, d_raw, stats)
    check_backward(dtype, g_raw, d_raw, gin_raw)
    return y, d, gin


def recompute_backward_ok(kind: str, dtype: str, g_raw: np.ndarray, x_raw: np.ndarray, gin_raw: np.ndarray) -> np.ndarray:
    """The recomputation comparator against the oracle's g f'(x), with the tolerance its arithmetic has and no more.
    It forms g h + g x s(x, h) from the gate h ROUNDED to the storage type (unit roundoff u) and a slope s derived
    from that rounded h by the operator's usual rule, then rounds once more:
        |error| <= |g| ( u |h| (1 + |x| K) + 2^-20 (|h| + |x h'|) ) + u |g f'|
    with K = max |ds/dh| (sigmoid: |1 - 2h| <= 1; the tanh form: that times 2 sqrt(2/pi) (1 + 3 a x^2); erf: the slope
    does not use h, 0; tanh(softplus): 2 |t| sigmoid <= 2) and 2^-20 for the fp32 arithmetic of the rule itself.
    |h| is bounded by |h| + |x h'|, which the oracle returns.  At small |x| this is a few roundings of g h: a wrong
    constant in a slope rule fails it."""
    f, fp, cond = oracle.forward(kind, dtype, x_raw, want_cond=True)
    g, x, got = oracle.widen(dtype, g_raw), oracle.widen(dtype, x_raw), oracle.widen(dtype, gin_raw)
    u = {"f32": 2.0 ** -24, "bf16": 2.0 ** -8, "f16": 2.0 ** -11}[dtype]      # half a unit in the last place
    k = {"swish": 1.0, "gelu_erf": 0.0, "mish": 2.0, "gelu_tanh": 1.5957691216 * (1.0 + 0.134145 * x * x)}[kind]
    tiny = {"f32": 2.0 ** -149, "bf16": 2.0 ** -133, "f16": 2.0 ** -24}[dtype]
    tol = np.abs(g) * cond * (u * (1.0 + np.abs(x) * k) + 2.0 ** -20) + u * np.abs(g * fp) * 1.0001 + tiny
    return np.abs(got - g * fp) <= tol
