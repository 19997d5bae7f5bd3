"""GPU edge cases: sizes around packet and tile boundaries, unaligned and mutually
misaligned pointers, in-place use, guard bands around every output, error returns,
and the two comparator layouts."""
import numpy as np
import pytest
import torch

import oracle
import parity
import ulp
from paper_2209_10778_b200 import binding as nfad
from paper_2209_10778_b200 import workloads as W

pytestmark = pytest.mark.gpu
DEV = "cuda"
KINDS = list(W.KINDS)
SIZES = [0, 1, 2, 3, 7, 8, 9, 15, 16, 17, 255, 256, 257, 1023, 1025, 4095, 4096, 4097, 8191, 8193, 32767, 32769, 65535, 65537]


def _guarded(n, td, pad=64, fill=7.0):
    """A tensor of n elements inside a larger buffer whose margins must stay untouched."""
    buf = torch.full((n + 2 * pad,), fill, dtype=td, device=DEV)
    return buf, buf[pad:pad + n]


@pytest.mark.parametrize("dtype", ["f32", "bf16", "f16"])
def test_sizes_and_guard_bands(dtype):
    td = W.TORCH_DTYPES[dtype]
    kind = "gelu_tanh"
    for n in SIZES:
        x = W.draw("normal", max(n, 1), dtype, n, DEV)[:n].contiguous()
        g = W.normal(max(n, 1), dtype, n + 1, 1.0, DEV)[:n].contiguous()
        yb, y = _guarded(n, td)
        db, d = _guarded(n, td)
        gb, gin = _guarded(n, td)
        nfad.nfad_act_forward(kind, x, y, d)
        nfad.nfad_act_backward(kind, g, d, gin)
        torch.cuda.synchronize()
        for b in (yb, db, gb):
            assert (b[:64] == 7.0).all() and (b[64 + n:] == 7.0).all(), f"guard band touched at n={n}"
        if n:
            xr = W.raw_numpy(x)
            if dtype == "f32":
                parity.check_forward_fp32(kind, xr, W.raw_numpy(y), W.raw_numpy(d))
            else:
                parity.check_forward_16(kind, dtype, xr, W.raw_numpy(y), W.raw_numpy(d))
            parity.check_backward(dtype, W.raw_numpy(g), W.raw_numpy(d), W.raw_numpy(gin))


@pytest.mark.parametrize("kind", ["mish", "gelu_erf"])      # one element per call; two per call in whole packets (16-bit)
@pytest.mark.parametrize("dtype", ["f32", "bf16", "f16"])
def test_unaligned_and_misaligned_pointers_give_identical_bits(dtype, kind):
    td = W.TORCH_DTYPES[dtype]
    n = 20011
    x0 = W.draw("mix", n, dtype, 11, DEV)
    y0, d0 = parity.gpu_forward(kind, x0)
    per16 = 16 // x0.element_size()
    for ox, oy, od in [(1, 1, 1), (3, 3, 3), (per16 - 1, per16 - 1, per16 - 1), (0, 1, 2), (1, 0, 0), (2, 2, 1)]:
        xb = torch.zeros(n + 16, dtype=td, device=DEV)
        yb = torch.full((n + 16,), 7.0, dtype=td, device=DEV)
        db = torch.full((n + 16,), 7.0, dtype=td, device=DEV)
        xb[ox:ox + n] = x0
        nfad.nfad_act_forward(kind, xb[ox:ox + n], yb[oy:oy + n], db[od:od + n])
        torch.cuda.synchronize()
        assert np.array_equal(W.raw_numpy(yb[oy:oy + n]), W.raw_numpy(y0)), (ox, oy, od)
        assert np.array_equal(W.raw_numpy(db[od:od + n]), W.raw_numpy(d0)), (ox, oy, od)
        assert (yb[:oy] == 7.0).all() and (yb[oy + n:] == 7.0).all()
        assert (db[:od] == 7.0).all() and (db[od + n:] == 7.0).all()


@pytest.mark.parametrize("kind", KINDS)
@pytest.mark.parametrize("dtype", ["bf16", "f16"])
def test_value_only_forward_is_the_same_on_every_path(kind, dtype):
    """The value-only forward of 16-bit storage runs two elements per call on packed fp32 arithmetic where the
    pointers allow whole packets, and one element per call otherwise (ragged ends, mutually misaligned pointers):
    over every finite value of the type (and the non-finite ones) the two must agree bit for bit."""
    td = W.TORCH_DTYPES[dtype]
    fin = W.all_finite_16bit(dtype)
    special = torch.tensor([float("inf"), float("-inf"), float("nan")], dtype=td)
    x0 = torch.cat([fin, special, fin.flip(0)]).to(DEV)          # odd length: a ragged tail on the packet path
    n = x0.numel()
    y0 = torch.empty_like(x0)
    nfad.nfad_act_forward_infer(kind, x0, y0)                    # aligned: packets
    xb = torch.zeros(n + 16, dtype=td, device=DEV)
    yb = torch.full((n + 16,), 7.0, dtype=td, device=DEV)
    xb[1:1 + n] = x0
    nfad.nfad_act_forward_infer(kind, xb[1:1 + n], yb[2:2 + n])  # offsets differ modulo a packet: element by element
    torch.cuda.synchronize()
    assert ulp.same_bits_or_both_nan(W.raw_numpy(yb[2:2 + n]), W.raw_numpy(y0), dtype).all()
    assert (yb[:2] == 7.0).all() and (yb[2 + n:] == 7.0).all()


@pytest.mark.parametrize("dtype", ["bf16", "f16"])
def test_training_forward_is_the_same_on_every_path(dtype):
    """GELU-erf's training forward runs two elements per call in whole packets and one per call elsewhere: over
    every value of the type both outputs must agree bit for bit."""
    td = W.TORCH_DTYPES[dtype]
    fin = W.all_finite_16bit(dtype)
    special = torch.tensor([float("inf"), float("-inf"), float("nan")], dtype=td)
    x0 = torch.cat([fin, special, fin.flip(0)]).to(DEV)
    n = x0.numel()
    y0, d0 = parity.gpu_forward("gelu_erf", x0)                   # aligned: packets
    xb = torch.zeros(n + 16, dtype=td, device=DEV)
    yb = torch.full((n + 16,), 7.0, dtype=td, device=DEV)
    db = torch.full((n + 16,), 7.0, dtype=td, device=DEV)
    xb[1:1 + n] = x0
    nfad.nfad_act_forward("gelu_erf", xb[1:1 + n], yb[2:2 + n], db[3:3 + n])   # no common packet grid: element by element
    torch.cuda.synchronize()
    assert ulp.same_bits_or_both_nan(W.raw_numpy(yb[2:2 + n]), W.raw_numpy(y0), dtype).all()
    assert ulp.same_bits_or_both_nan(W.raw_numpy(db[3:3 + n]), W.raw_numpy(d0), dtype).all()


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_in_place(dtype):
    n = 50001
    kind = "swish"
    x = W.draw("normal", n, dtype, 21, DEV)
    g = W.normal(n, dtype, 22, 1.0, DEV)
    y0, d0 = parity.gpu_forward(kind, x)
    gin0 = parity.gpu_backward(kind, g, d0)
    # y in place of x
    xa = x.clone(); da = torch.empty_like(x)
    nfad.nfad_act_forward(kind, xa, xa, da)
    # dfdx in place of x
    xb = x.clone(); yb = torch.empty_like(x)
    nfad.nfad_act_forward(kind, xb, yb, xb)
    # grad_in in place of grad_out, and of dfdx
    ga = g.clone(); nfad.nfad_act_backward(kind, ga, d0, ga)
    dc = d0.clone(); nfad.nfad_act_backward(kind, g, dc, dc)
    torch.cuda.synchronize()
    assert torch.equal(xa, y0) and torch.equal(da, d0)
    assert torch.equal(yb, y0) and torch.equal(xb, d0)
    assert torch.equal(ga, gin0) and torch.equal(dc, gin0)


def test_error_returns_on_device_pointers():
    x = torch.zeros(1024, device=DEV)
    y = torch.zeros(1024, device=DEV)
    with pytest.raises(nfad.NfadError) as e:
        nfad.nfad_act_forward("swish", x, y, y)            # two outputs overlap
    assert e.value.status == 4
    with pytest.raises(nfad.NfadError) as e:
        nfad.nfad_act_forward("swish", x[:512], x[256:768], y[:512])   # partial overlap of input and output
    assert e.value.status == 4
    with pytest.raises(nfad.NfadError) as e:
        nfad.nfad_act_forward(11, x, y, torch.zeros(1024, device=DEV))
    assert e.value.status == 1
    torch.cuda.synchronize()


def _conv_tolerance_ok(dtype, gin_raw, g_raw, x_raw, kind):
    """Conventional backward multiplies g by an fp32 f'(x) that is never rounded to the storage
    type: |gin - g f'| <= |g| * 4 ulp32(T) plus one rounding of the product to the storage type."""
    f, fp, cond = oracle.forward(kind, dtype, x_raw, want_cond=True)
    g = oracle.widen(dtype, g_raw)
    want = g * fp
    got = oracle.widen(dtype, gin_raw)
    # fp32 storage: the 4-ulp gate of f' itself; 16-bit storage: the fast policy's f' is good to
    # ~2^-16 of its addends, far inside one 16-bit ulp
    tol32 = np.abs(g) * (4 * ulp.ulp32(cond) if dtype == "f32" else cond * 2.0 ** -16)
    if dtype == "f32":
        tol = tol32 + 0.5 * ulp.ulp32(want) * 1.0001
    else:
        rn = oracle.widen(dtype, oracle.round_to(dtype, want))
        up = oracle.widen(dtype, oracle.round_to(dtype, want + tol32))
        lo = oracle.widen(dtype, oracle.round_to(dtype, want - tol32))
        return (got >= np.minimum(lo, rn)) & (got <= np.maximum(up, rn))
    return np.abs(got - want) <= tol + 64 * 2.0 ** -149


@pytest.mark.parametrize("kind", KINDS)
@pytest.mark.parametrize("dtype", ["f32", "bf16", "f16"])
def test_conventional_comparator(kind, dtype):
    n = (1 << 16) + 5
    x = W.draw("normal", n, dtype, 31, DEV)
    g = W.normal(n, dtype, 32, 1.0, DEV)
    gin = torch.empty_like(g)
    nfad.nfad_cmp_conv_backward(kind, g, x, gin)
    torch.cuda.synchronize()
    ok = _conv_tolerance_ok(dtype, W.raw_numpy(gin), W.raw_numpy(g), W.raw_numpy(x), kind)
    assert ok.all(), f"{(~ok).sum()} of {n} outside tolerance"


@pytest.mark.parametrize("kind", KINDS)
@pytest.mark.parametrize("dtype", ["f32", "bf16", "f16"])
def test_recompute_comparator(kind, dtype):
    # operator-by-operator rules through a stored intermediate: the tolerance is the one that arithmetic has
    # (parity.recompute_backward_ok)
    n = (1 << 16) + 5
    x = W.draw("normal", n, dtype, 41, DEV)
    g = W.normal(n, dtype, 42, 1.0, DEV)
    gin = torch.empty_like(g)
    nbytes = nfad.nfad_cmp_recompute_scratch_bytes(kind, dtype, n)
    assert nbytes >= n * x.element_size()
    scratch = torch.empty(nbytes, dtype=torch.uint8, device=DEV)
    nfad.nfad_cmp_recompute_backward(kind, g, x, scratch, gin)
    torch.cuda.synchronize()
    ok = parity.recompute_backward_ok(kind, dtype, W.raw_numpy(g), W.raw_numpy(x), W.raw_numpy(gin))
    assert ok.all(), f"{(~ok).sum()} of {n} outside tolerance"
    with pytest.raises(nfad.NfadError) as e:
        nfad.nfad_cmp_recompute_backward(kind, g, x, scratch[:16], gin)
    assert e.value.status == 7


def test_saved_bytes_per_element_table():
    for dtype, s in (("f32", 4), ("bf16", 2), ("f16", 2)):
        for kind in KINDS:
            assert nfad.nfad_saved_bytes_per_element(kind, dtype, "nested") == s
            assert nfad.nfad_saved_bytes_per_element(kind, dtype, "conventional") == s
            assert nfad.nfad_saved_bytes_per_element(kind, dtype, "recompute") == s
            assert nfad.nfad_saved_bytes_per_element(kind, dtype, "op_by_op") >= 2 * s
        assert nfad.nfad_saved_bytes_per_element("swish", dtype, "op_by_op") == 2 * s   # x and sigmoid(x)
