"""Parity of the bias-fused entry points (nfad_bias_act_forward / nfad_bias_act_backward) with the fp64 oracle.

Tolerances.  fp32 storage: y, f' exactly as for the plain pass (tests/parity.py), at the pre-activation
z = fl32(x + bias) that both sides form with one fp32 addition.  16-bit storage: within 1 ulp of the oracle rounded
once to the type, as for the plain pass -- except that here z is an fp32 number and can fall arbitrarily close to the
sign change of f' (a 16-bit x cannot), where f' = h + z h' is the difference of two fp32-evaluated terms: an element
also passes if |got - o| <= ulp16(o) + ulp16(T)/16, T = |h| + |z h'| (the plain pass's fp32 arithmetic is good to
2^-16 T, which is ulp16(T)/32 for fp16 and less for bf16).  grad_in: bit-equal.  grad_bias (fp32 accumulation in a
fixed order: each chunk of consecutive rows summed in row order, then the chunks in order) is compared with the
oracle's fp64 column sums of the same rounded grad_in values under the standard bound of recursive summation,
|err| <= depth * 2^-24 * sum|terms| * (1 + small), depth = additions any one term passes through
<= chunk_rows + (chunks - 1); the test takes the chunk count from the library's scratch size.
"""
import math

import numpy as np
import pytest
import torch

import oracle
import parity
import ulp
from paper_2209_10778_b200 import binding as nfad
from paper_2209_10778_b200 import workloads as W

pytestmark = pytest.mark.gpu

KINDS = ["gelu_erf", "gelu_tanh", "swish", "mish"]
DTYPES = ["f32", "bf16", "f16"]
DEV = "cuda"
# (rows, cols): whole strips; a ragged last strip (125 / 250 packets per row); cols not a multiple of the packet
SHAPES = [(300, 768), (67, 1000), (41, 1003), (1, 64), (9, 8)]


def _scratch(dtype, rows, cols):
    nbytes = nfad.nfad_bias_act_backward_scratch_bytes(W.TORCH_DTYPES[dtype], rows, cols)
    return (torch.empty(max(nbytes, 4) // 4, dtype=torch.float32, device=DEV) if nbytes else None), nbytes


def _depth(rows, cols, nbytes):
    chunks = max(1, nbytes // (4 * cols))
    chunk_rows = -(-rows // chunks)
    chunk_rows = -(-chunk_rows // 4) * 4 + 4
    return chunk_rows + (chunks - 1)


def _ulp16(v, dtype):
    """Spacing of the 16-bit type at |v| (the subnormal spacing below the normal range)."""
    p, emin = (8, -126) if dtype == "bf16" else (11, -14)
    e = np.floor(np.log2(np.maximum(np.abs(v), 2.0 ** emin)))
    return 2.0 ** (np.maximum(e, emin) - (p - 1))


def _check_forward(kind, dtype, x, bias, y, d, rows, cols, stats=None):
    x_raw, b_raw = W.raw_numpy(x), W.raw_numpy(bias)
    f, fp, z, cond = oracle.bias_forward(kind, dtype, x_raw, b_raw, rows, cols, want_cond=True)
    if dtype == "f32":
        parity.check_forward_fp32_values(kind, z.astype(np.float32), f, fp, cond, W.raw_numpy(y), W.raw_numpy(d), stats)
    else:
        y_bits, d_bits = W.raw_numpy(y), W.raw_numpy(d)
        want_y, want_d = oracle.round_to(dtype, f), oracle.round_to(dtype, fp)
        dy, dd = ulp.ulp_distance16(y_bits, want_y), ulp.ulp_distance16(d_bits, want_d)
        assert not ((dy > 1) | ulp.is_nan16(y_bits, dtype)).any(), f"{kind} {dtype} y: max distance {dy.max()}"
        err = np.abs(oracle.widen(dtype, d_bits) - fp)
        near_root = err <= _ulp16(fp, dtype) + _ulp16(cond, dtype) / 16
        bad = ((dd > 1) & ~((z < 0) & near_root)) | ulp.is_nan16(d_bits, dtype)
        assert not bad.any(), (f"{kind} {dtype} f': {int(bad.sum())} out of tolerance, first z={z[np.flatnonzero(bad)[0]]!r} "
                               f"got={oracle.widen(dtype, d_bits)[np.flatnonzero(bad)[0]]!r} want={fp[np.flatnonzero(bad)[0]]!r}")


def _check_backward(dtype, g, d, gin, gb, rows, cols, nbytes):
    want_gin, want_gb, want_abs = oracle.bias_backward(dtype, W.raw_numpy(g), W.raw_numpy(d), rows, cols)
    same = ulp.same_bits_or_both_nan(W.raw_numpy(gin), want_gin, dtype)
    assert same.all(), f"grad_in: {int((~same).sum())} mismatches, first at {int(np.flatnonzero(~same)[0])}"
    got = gb.double().cpu().numpy()
    tol = (_depth(rows, cols, nbytes) + 1) * 2.0 ** -24 * want_abs * 1.01 + 2.0 ** -149
    err = np.abs(got - want_gb)
    assert (err <= tol).all(), (f"grad_bias: worst column {int(np.argmax(err / np.maximum(tol, 1e-300)))}: "
                                f"err {err.max():.3e} tol {tol[np.argmax(err)]:.3e}")
    return err, tol


def _run(kind, dtype, rows, cols, seed, x_std=1.5):
    n = rows * cols
    x = W.normal(n, dtype, seed, x_std, DEV)
    bias = W.normal(cols, dtype, seed + 1, 0.5, DEV)
    g = W.normal(n, dtype, seed + 2, 1.0, DEV)
    y, d, gin = torch.empty_like(x), torch.empty_like(x), torch.empty_like(x)
    gb = torch.full((cols,), float("nan"), dtype=torch.float32, device=DEV)
    scratch, nbytes = _scratch(dtype, rows, cols)
    nfad.nfad_bias_act_forward(kind, x, bias, y, d)
    nfad.nfad_bias_act_backward(kind, g, d, gin, gb, scratch)
    torch.cuda.synchronize()
    _check_forward(kind, dtype, x, bias, y, d, rows, cols)
    _check_backward(dtype, g, d, gin, gb, rows, cols, nbytes)
    return x, bias, g, y, d, gin, gb


@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("kind", KINDS)
def test_parity_several_shapes(kind, dtype):
    for i, (rows, cols) in enumerate(SHAPES):
        _run(kind, dtype, rows, cols, 100 + i)


@pytest.mark.parametrize("dtype", DTYPES)
def test_wide_inputs_and_tails(dtype):
    # pre-activations out to the saturated tails: x from the mixed distribution plus a bias
    rows, cols = 128, 512
    x = W.mix(rows * cols, dtype, 7, DEV)
    bias = W.uniform(cols, dtype, 8, -3.0, 3.0, DEV)
    for kind in KINDS:
        y, d = torch.empty_like(x), torch.empty_like(x)
        nfad.nfad_bias_act_forward(kind, x, bias, y, d)
        torch.cuda.synchronize()
        _check_forward(kind, dtype, x, bias, y, d, rows, cols)


@pytest.mark.parametrize("dtype", DTYPES)
def test_unaligned_pointers_give_the_same_bits(dtype):
    # the same data one element off the 16-byte grid takes the element-wise kernels: identical y, f', grad_in, grad_bias
    rows, cols, kind = 50, 256, "gelu_erf"
    n = rows * cols
    x, bias, g, y, d, gin, gb = _run(kind, dtype, rows, cols, 31)
    def shifted(t):
        buf = torch.empty(t.numel() + 1, dtype=t.dtype, device=DEV)
        buf[1:].copy_(t)
        return buf[1:]
    xs, bs, gs = shifted(x), shifted(bias), shifted(g)
    ys, ds, gins = shifted(torch.empty_like(x)), shifted(torch.empty_like(x)), shifted(torch.empty_like(x))
    gb2 = torch.empty_like(gb)
    scratch, _ = _scratch(dtype, rows, cols)
    nfad.nfad_bias_act_forward(kind, xs, bs, ys, ds)
    nfad.nfad_bias_act_backward(kind, gs, ds, gins, gb2, scratch)
    torch.cuda.synchronize()
    for a, b in ((y, ys), (d, ds), (gin, gins)):
        assert np.array_equal(W.raw_numpy(a), W.raw_numpy(b.contiguous()))
    assert torch.equal(gb.view(torch.int32), gb2.view(torch.int32))


def test_matches_the_unfused_calls_bit_for_bit():
    # fp32: adding the bias with torch and calling the plain pass is the same arithmetic
    rows, cols = 64, 384
    x = W.normal(rows * cols, "f32", 3, 1.5, DEV)
    bias = W.normal(cols, "f32", 4, 0.5, DEV)
    z = (x.view(rows, cols) + bias).reshape(-1).contiguous()
    for kind in KINDS:
        y0, d0, y1, d1 = (torch.empty_like(x) for _ in range(4))
        nfad.nfad_act_forward(kind, z, y0, d0)
        nfad.nfad_bias_act_forward(kind, x, bias, y1, d1)
        assert torch.equal(y0.view(torch.int32), y1.view(torch.int32))
        assert torch.equal(d0.view(torch.int32), d1.view(torch.int32))


def test_two_calls_give_the_same_grad_bias_bits():
    rows, cols = 2048, 1024
    g = W.normal(rows * cols, "bf16", 5, 1.0, DEV)
    d = W.uniform(rows * cols, "bf16", 6, -0.2, 1.1, DEV)
    gin = torch.empty_like(g)
    scratch, _ = _scratch("bf16", rows, cols)
    out = []
    for _ in range(2):
        gb = torch.empty(cols, dtype=torch.float32, device=DEV)
        nfad.nfad_bias_act_backward("swish", g, d, gin, gb, scratch)
        out.append(gb)
    torch.cuda.synchronize()
    assert torch.equal(out[0].view(torch.int32), out[1].view(torch.int32))


def test_in_place_and_degenerate_shapes():
    rows, cols = 40, 128
    x = W.normal(rows * cols, "bf16", 9, 1.0, DEV)
    bias = W.normal(cols, "bf16", 10, 0.5, DEV)
    y, d = torch.empty_like(x), torch.empty_like(x)
    nfad.nfad_bias_act_forward("mish", x, bias, y, d)
    xin = x.clone()
    nfad.nfad_bias_act_forward("mish", xin, bias, xin, d.clone())        # y in place of x
    assert torch.equal(xin.view(torch.int16), y.view(torch.int16))
    g = W.normal(rows * cols, "bf16", 11, 1.0, DEV)
    gin, gb, gb2 = torch.empty_like(g), torch.empty(cols, dtype=torch.float32, device=DEV), torch.empty(cols, dtype=torch.float32, device=DEV)
    scratch, _ = _scratch("bf16", rows, cols)
    nfad.nfad_bias_act_backward("mish", g, d, gin, gb, scratch)
    gi = g.clone()
    nfad.nfad_bias_act_backward("mish", gi, d, gi, gb2, scratch)          # grad_in in place of grad_out
    assert torch.equal(gi.view(torch.int16), gin.view(torch.int16)) and torch.equal(gb, gb2)
    # no rows: grad_bias is zero, nothing else is touched
    e = torch.empty(0, dtype=torch.bfloat16, device=DEV)
    gbz = torch.full((cols,), 7.0, dtype=torch.float32, device=DEV)
    nfad.nfad_bias_act_backward("mish", e, e, e, gbz, None)
    nfad.nfad_bias_act_forward("mish", e, bias, e, e)
    torch.cuda.synchronize()
    assert (gbz == 0).all()


def test_argument_errors():
    lib = nfad.load()
    rows, cols = 16, 64
    x = torch.zeros(rows * cols, dtype=torch.float32, device=DEV)
    y, d = torch.empty_like(x), torch.empty_like(x)
    b = torch.zeros(cols, dtype=torch.float32, device=DEV)
    gb = torch.zeros(cols, dtype=torch.float32, device=DEV)
    st = torch.cuda.current_stream().cuda_stream
    p = lambda t: t.data_ptr()
    assert lib.nfad_bias_act_forward(9, 0, p(x), p(b), p(y), p(d), rows, cols, st) == 1
    assert lib.nfad_bias_act_forward(0, 5, p(x), p(b), p(y), p(d), rows, cols, st) == 2
    assert lib.nfad_bias_act_forward(0, 0, p(x), None, p(y), p(d), rows, cols, st) == 3
    assert lib.nfad_bias_act_forward(0, 0, p(x), p(b), p(y), p(y), rows, cols, st) == 4
    assert lib.nfad_bias_act_forward(0, 0, p(x), p(y), p(y), p(d), rows, cols, st) == 4          # bias inside an output
    assert lib.nfad_bias_act_forward(0, 0, p(x), p(b), p(y), p(d), rows, 1 << 31, st) == 9
    big_rows = 4096
    xb = torch.zeros(big_rows * cols, dtype=torch.float32, device=DEV)
    need = nfad.nfad_bias_act_backward_scratch_bytes(torch.float32, big_rows, cols)
    assert need > 0
    s = torch.empty(need // 4, dtype=torch.float32, device=DEV)
    assert lib.nfad_bias_act_backward(0, 0, p(xb), p(xb), p(xb), p(gb), p(s), need - 4, big_rows, cols, st) == 7
    assert lib.nfad_bias_act_backward(0, 0, p(xb), p(xb), p(xb), p(gb), None, 0, big_rows, cols, st) == 3
    assert lib.nfad_bias_act_backward(0, 0, p(xb), p(xb), p(xb), None, p(s), need, big_rows, cols, st) == 3
    assert lib.nfad_bias_act_backward(0, 0, p(xb), p(xb), p(xb), p(xb), p(s), need, big_rows, cols, st) == 4
    assert lib.nfad_bias_act_backward(0, 0, p(xb), p(xb), p(xb), p(gb), p(s), need, big_rows, cols, st) == 0
    torch.cuda.synchronize()


@pytest.mark.parametrize("kind", ["gelu_erf", "gelu_tanh"])
def test_bert_ffn_shape_full_size(kind):
    # the bench workload's tensor, [32*128, 3072] bf16, every element against the oracle
    rows, cols = 32 * 128, 3072
    _run(kind, "bf16", rows, cols, 77, x_std=1.0)


def test_autograd_wrapper_against_torch_double():
    # the wrapper's gradients for x and the bias against torch's own autograd of gelu(x + b) in fp64
    from paper_2209_10778_b200 import autograd as nfad_autograd
    rows, cols = 96, 256
    x = W.normal(rows * cols, "f32", 41, 1.5, DEV).view(4, rows // 4, cols).requires_grad_(True)
    b = W.normal(cols, "f32", 42, 0.5, DEV).requires_grad_(True)
    g = W.normal(rows * cols, "f32", 43, 1.0, DEV).view(4, rows // 4, cols)
    for approx in ("none", "tanh"):
        x.grad = b.grad = None
        y = nfad_autograd.bias_gelu(x, b, approx)
        y.backward(g)
        x64 = x.detach().double().requires_grad_(True)
        b64 = b.detach().double().requires_grad_(True)
        y64 = torch.nn.functional.gelu(x64 + b64, approximate=approx)
        y64.backward(g.double())
        torch.cuda.synchronize()
        assert torch.allclose(y.detach().double(), y64.detach(), rtol=1e-6, atol=1e-7)
        assert torch.allclose(x.grad.double(), x64.grad, rtol=2e-6, atol=2e-6)
        assert ((b.grad.double() - b64.grad).abs() <= 1e-5 * x64.grad.view(rows, cols).abs().sum(0) + 1e-6).all()


def test_tall_narrow_tensor_covers_the_row_chunk_loop():
    # more row chunks than one grid dimension holds (rows / 4 > 65535): the forward kernel's chunk loop, and a backward
    # whose strips are narrower than one warp-wide access
    _run("swish", "bf16", 300000, 64, 55)


@pytest.mark.parametrize("dtype", DTYPES)
def test_value_only_forward_against_the_training_value(dtype):
    for rows, cols in ((300, 768), (41, 1003)):
        x = W.normal(rows * cols, dtype, 81, 1.5, DEV)
        bias = W.normal(cols, dtype, 82, 0.5, DEV)
        for kind in KINDS:
            y, d, yi = torch.empty_like(x), torch.empty_like(x), torch.full_like(x, 3.0)
            nfad.nfad_bias_act_forward(kind, x, bias, y, d)
            nfad.nfad_bias_act_forward_infer(kind, x, bias, yi)
            torch.cuda.synchronize()
            if kind == "gelu_erf" and dtype != "f32":     # the 16-bit erf gate has a cheaper value-only form: one ulp at most
                assert (ulp.ulp_distance16(W.raw_numpy(y), W.raw_numpy(yi)) <= 1).all(), (kind, dtype, rows, cols)
            else:
                assert np.array_equal(W.raw_numpy(y), W.raw_numpy(yi)), (kind, dtype, rows, cols)
    xs = torch.tensor([float("inf"), float("-inf"), float("nan"), 0.0], device=DEV, dtype=W.TORCH_DTYPES[dtype])
    b1 = torch.zeros(4, device=DEV, dtype=W.TORCH_DTYPES[dtype])
    out = torch.empty_like(xs)
    for kind in KINDS:
        nfad.nfad_bias_act_forward_infer(kind, xs, b1, out)
        o = out.float().cpu().numpy()
        assert o[0] == np.inf and o[1] == 0.0 and np.signbit(o[1]) and np.isnan(o[2]) and o[3] == 0.0
