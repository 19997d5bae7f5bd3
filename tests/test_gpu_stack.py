"""Stacked activations (layer i+1 reads layer i's output) under the three single-tensor layouts: nested Forward-AD
(keeps f'(x_i)), conventional (keeps x_i, re-derives f' in backward) and recomputation (keeps x_i, re-materialises the
gate in backward) -- Section II-C approaches 3, 1 (fused) and 2.

Every layer is held to the oracle on the tensors that layer really saw (its input as the GPU produced it, the upstream
gradient as the GPU produced it): forward by the usual gates, the nested backward bit for bit, the comparators by the
tolerance their arithmetic has.  On top of that the input gradient of the whole stack is compared with a chain that
only the oracle computed (its own roundings at every layer), within a bound that grows with depth.
"""
import numpy as np
import pytest
import torch

import oracle
import parity
from paper_2209_10778_b200 import binding as nfad
from paper_2209_10778_b200 import workloads as W
from test_gpu_edges import _conv_tolerance_ok

pytestmark = pytest.mark.gpu
DEV = "cuda"
LAYERS = 3


def _oracle_chain(kind, dtype, x_raw, g_raw):
    """Forward through LAYERS layers and back, every tensor rounded to the storage type as it would be stored."""
    xs = [x_raw]
    ds = []
    for _ in range(LAYERS):
        f, fp = oracle.forward(kind, dtype, xs[-1])
        xs.append(oracle.round_to(dtype, f))
        ds.append(oracle.round_to(dtype, fp))
    g = g_raw
    for i in reversed(range(LAYERS)):
        g = oracle.backward(dtype, g, ds[i])
    return g


@pytest.mark.parametrize("kind", ["gelu_erf", "swish"])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_three_layers_under_three_layouts(kind, dtype):
    n = 50003
    x0 = W.normal(n, dtype, 90, 1.0, DEV)
    gL = W.normal(n, dtype, 91, 1.0, DEV)
    new = lambda: torch.empty_like(x0)

    # ---- nested: forward keeps f'(x_i); backward is the multiply
    xs, ds = [x0], []
    for _ in range(LAYERS):
        y, d = new(), new()
        nfad.nfad_act_forward(kind, xs[-1], y, d)
        xs.append(y)
        ds.append(d)
    gs = [gL]
    for i in reversed(range(LAYERS)):
        gi = new()
        nfad.nfad_act_backward(kind, gs[-1], ds[i], gi)
        gs.append(gi)
    torch.cuda.synchronize()
    for i in range(LAYERS):
        xr, yr, dr = W.raw_numpy(xs[i]), W.raw_numpy(xs[i + 1]), W.raw_numpy(ds[i])
        if dtype == "f32":
            parity.check_forward_fp32(kind, xr, yr, dr)
        else:
            parity.check_forward_16(kind, dtype, xr, yr, dr)
    for j, i in enumerate(reversed(range(LAYERS))):
        parity.check_backward(dtype, W.raw_numpy(gs[j]), W.raw_numpy(ds[i]), W.raw_numpy(gs[j + 1]))
    nested_grad = oracle.widen(dtype, W.raw_numpy(gs[-1]))

    # ---- conventional and recomputation: the value-only forward keeps x_i
    xc = [x0]
    for _ in range(LAYERS):
        y = new()
        nfad.nfad_act_forward_infer(kind, xc[-1], y)
        xc.append(y)
    torch.cuda.synchronize()
    for i in range(LAYERS):                                     # same inputs, same chain: the same values as above
        assert np.array_equal(W.raw_numpy(xc[i + 1]), W.raw_numpy(xs[i + 1])) or (kind == "gelu_erf" and dtype != "f32")
    grads = {}
    for layout in ("conventional", "recompute"):
        g = gL
        scratch = torch.empty(nfad.nfad_cmp_recompute_scratch_bytes(kind, dtype, n), dtype=torch.uint8, device=DEV)
        for i in reversed(range(LAYERS)):
            gi = new()
            if layout == "conventional":
                nfad.nfad_cmp_conv_backward(kind, g, xc[i], gi)
            else:
                nfad.nfad_cmp_recompute_backward(kind, g, xc[i], scratch, gi)
            torch.cuda.synchronize()
            g_raw, x_raw, gi_raw = W.raw_numpy(g), W.raw_numpy(xc[i]), W.raw_numpy(gi)
            ok = _conv_tolerance_ok(dtype, gi_raw, g_raw, x_raw, kind) if layout == "conventional" else \
                parity.recompute_backward_ok(kind, dtype, g_raw, x_raw, gi_raw)
            assert ok.all(), (layout, i, int((~ok).sum()))
            g = gi
        grads[layout] = oracle.widen(dtype, W.raw_numpy(g))

    # ---- the whole stack against a chain only the oracle computed
    want = oracle.widen(dtype, _oracle_chain(kind, dtype, W.raw_numpy(x0), W.raw_numpy(gL)))
    u = {"f32": 2.0 ** -24, "bf16": 2.0 ** -8}[dtype]
    # every layer contributes a rounding or two of its output, its derivative and its gradient, and a one-ulp change of a
    # layer's input moves that layer's derivative by |f''| <= 1.2 input ulps: 8 u per layer relative to the scale of
    # the gradient (|gL|, since |f'| <= 1.13) is generous without hiding a wrong layer
    scale = np.abs(oracle.widen(dtype, W.raw_numpy(gL)))
    for name, got in (("nested", nested_grad), ("conventional", grads["conventional"]), ("recompute", grads["recompute"])):
        bad = np.abs(got - want) > 8 * LAYERS * u * scale + 1e-30
        assert not bad.any(), (name, int(bad.sum()), float(np.abs(got - want).max()))
