"""The entry point that brings its own scratch (`nfad_cmp_recompute_backward_noalloc`).

It exists for callers that cannot allocate device memory at the call site (all memory
handed out up front by a host application, or an allocation's device-wide synchronisation
being unacceptable there).  It must give exactly what `nfad_cmp_recompute_backward` gives
with caller-owned scratch -- the two run the same two kernels -- also when the shared
built-in array still holds another call's data.  Collected last on purpose: a run that
stops at the first failure has then already run every other test.
"""
import numpy as np
import pytest
import torch

import parity
from paper_2209_10778_b200 import binding as nfad
from paper_2209_10778_b200 import workloads as W

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _reference(kind, g, x):
    scratch = torch.empty(nfad.nfad_cmp_recompute_scratch_bytes(kind, x.dtype, x.numel()), dtype=torch.uint8, device=DEV)
    out = torch.empty_like(g)
    nfad.nfad_cmp_recompute_backward(kind, g, x, scratch, out)
    return out


@pytest.mark.parametrize("dtype", ["f32", "bf16", "f16"])
def test_two_calls_in_a_row_match_the_caller_scratch_entry_point(dtype):
    n1, n2 = 200003, 70001                       # several tiles + ragged tails; second call smaller than the first
    cases = [("gelu_erf", n1, 51), ("mish", n2, 52)]
    outs, refs = [], []
    for kind, n, seed in cases:                  # two calls back to back on the same stream, sharing the array
        x = W.draw("normal", n, dtype, seed, DEV)
        g = W.normal(n, dtype, seed + 100, 1.0, DEV)
        out = torch.full_like(g, 7.0)
        nfad.nfad_cmp_recompute_backward_noalloc(kind, g, x, out)
        outs.append(out)
        refs.append((kind, g, x))
    torch.cuda.synchronize()
    for out, (kind, g, x) in zip(outs, refs):
        want = _reference(kind, g, x)
        torch.cuda.synchronize()
        assert np.array_equal(W.raw_numpy(out), W.raw_numpy(want)), kind
        # and, like that entry point, what the oracle's g f'(x) allows for this arithmetic
        assert parity.recompute_backward_ok(kind, dtype, W.raw_numpy(g), W.raw_numpy(x), W.raw_numpy(out)).all(), kind


def test_in_place_gradient_and_size_limit():
    n = 4099
    x = W.draw("mix", n, "bf16", 61, DEV)
    g = W.normal(n, "bf16", 62, 1.0, DEV)
    want = _reference("swish", g, x)
    gi = g.clone()
    nfad.nfad_cmp_recompute_backward_noalloc("swish", gi, x, gi)          # grad_in == grad_out
    torch.cuda.synchronize()
    assert np.array_equal(W.raw_numpy(gi), W.raw_numpy(want))
    # one element more than the built-in array can serve: refused, nothing launched, output untouched
    too_many = nfad.NOALLOC_SCRATCH_BYTES // 4 + 1
    xb = torch.zeros(too_many, device=DEV)
    ob = torch.full((too_many,), 7.0, device=DEV)
    with pytest.raises(nfad.NfadError) as e:
        nfad.nfad_cmp_recompute_backward_noalloc("swish", xb, xb.clone(), ob)
    assert e.value.status == 9
    torch.cuda.synchronize()
    assert bool((ob == 7.0).all())
    # exactly at the limit it runs
    n_max = nfad.NOALLOC_SCRATCH_BYTES // 4
    xm = W.normal(n_max, "f32", 63, 1.0, DEV)
    gm = W.normal(n_max, "f32", 64, 1.0, DEV)
    om = torch.empty_like(gm)
    nfad.nfad_cmp_recompute_backward_noalloc("gelu_tanh", gm, xm, om)
    torch.cuda.synchronize()
    assert np.array_equal(W.raw_numpy(om), W.raw_numpy(_reference("gelu_tanh", gm, xm)))
