"""Every fp32 input (or every k-th) through the fp32-storage forward pass, against the fp64 oracle.

The fp32 line has 2 x 1.12e9 bit patterns with |x| <= 130 (beyond that every kind is saturated).  By default every
251st pattern is taken (8.9 million per kind, seconds); set NFAD_EXHAUSTIVE_STRIDE=1 to run them all (about three
minutes per kind on a 16-core host: the oracle is what takes the time).  Measured per kind: the worst value error in
fp32 ulp, the worst derivative error in the gate's metric (strict for x >= 0, scaled by |h| + |x h'| for x < 0: see
parity.py), the worst subnormal-result errors in units of 2^-149, the count of non-finite outputs.  The bounds asserted
here are those of the arithmetic (double-precision chains, one rounding at the store; the erf gate's polynomial runs in
fp32), well inside the 4-ulp tolerance of the pass, so that a regression shows long before the tolerance is reached.
The strict entry point is held to 4 ulp of f' itself for every x.
"""
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2209_10778_b200 import binding as nfad

pytestmark = pytest.mark.gpu
STRIDE = int(os.environ.get("NFAD_EXHAUSTIVE_STRIDE", "251"))
HI_BITS = int(np.float32(130.0).view(np.uint32))
CHUNK = 1 << 25
# (value ulp, derivative in the gate's metric): the all-inputs maxima are 2.28 / 2.34 for the erf form and 0.53 for the others
BOUNDS = {"gelu_erf": (2.6, 2.6), "gelu_tanh": (0.6, 0.6), "swish": (0.6, 0.6), "mish": (0.6, 0.6)}


def _spacing32(v):
    return np.maximum(np.spacing(np.abs(v).astype(np.float32)).astype(np.float64), 2.0 ** -149)


def _sweep(kind, strict):
    oracle.set_threads(oracle.max_threads())
    worst = dict(y=0.0, y_x=0.0, d=0.0, d_x=0.0, sub_y=0.0, sub_d=0.0, bad=0, count=0)
    call = nfad.nfad_act_forward_strict if strict else nfad.nfad_act_forward
    for sign in (0, 1 << 31):
        for start in range(0, HI_BITS + 1, CHUNK * STRIDE):
            stop = min(start + CHUNK * STRIDE, HI_BITS + 1)
            bits = torch.arange(start, stop, STRIDE, dtype=torch.int64, device="cuda") + sign
            x = torch.where(bits >= 2 ** 31, bits - 2 ** 32, bits).to(torch.int32).view(torch.float32).contiguous()
            y, d = torch.empty_like(x), torch.empty_like(x)
            call(kind, x, y, d)
            torch.cuda.synchronize()
            xh, yh, dh = x.cpu().numpy(), y.cpu().numpy(), d.cpu().numpy()
            f, fp, t = oracle.forward(kind, "f32", xh, want_cond=True)
            ey = np.abs(yh.astype(np.float64) - f) / _spacing32(f)
            es = np.abs(dh.astype(np.float64) - fp) / _spacing32(fp)
            ec = np.abs(dh.astype(np.float64) - fp) / _spacing32(np.maximum(t, np.abs(fp)))
            gate = es if strict else np.where(xh >= 0, es, ec)
            sub_y = np.abs(f) < 2.0 ** -126
            sub_d = (np.abs(fp) < 2.0 ** -126) & ((t < 2.0 ** -100) | strict)
            ny, nd = np.where(sub_y, 0, ey), np.where(sub_d, 0, gate)
            i, j = int(ny.argmax()), int(nd.argmax())
            if ny[i] > worst["y"]:
                worst["y"], worst["y_x"] = float(ny[i]), float(xh[i])
            if nd[j] > worst["d"]:
                worst["d"], worst["d_x"] = float(nd[j]), float(xh[j])
            if sub_y.any():
                worst["sub_y"] = max(worst["sub_y"], float((np.abs(yh.astype(np.float64) - f)[sub_y] / 2.0 ** -149).max()))
            if sub_d.any():
                worst["sub_d"] = max(worst["sub_d"], float((np.abs(dh.astype(np.float64) - fp)[sub_d] / 2.0 ** -149).max()))
            worst["bad"] += int((~np.isfinite(yh)).sum() + (~np.isfinite(dh)).sum())
            worst["count"] += xh.size
    return worst


@pytest.mark.parametrize("kind", list(BOUNDS))
def test_every_kth_fp32_input(kind):
    w = _sweep(kind, strict=False)
    print(kind, "stride", STRIDE, w)
    by, bd = BOUNDS[kind]
    assert w["bad"] == 0
    assert w["y"] <= by and w["d"] <= bd, w
    # a subnormal result is rounded once, by the final conversion: within a spacing, or two where the gate itself carries
    # a couple of fp32 ulp (the erf form)
    assert w["sub_y"] <= 2.0 and w["sub_d"] <= 2.0, w


@pytest.mark.parametrize("kind", list(BOUNDS))
def test_every_kth_fp32_input_strict_entry_point(kind):
    w = _sweep(kind, strict=True)
    print(kind, "strict, stride", STRIDE, w)
    assert w["bad"] == 0
    assert w["y"] <= 1.0 and w["d"] <= 2.0, w                   # the strict chain is good to the last bits of a double
    assert w["sub_y"] <= 1.0 and w["sub_d"] <= 1.0, w
