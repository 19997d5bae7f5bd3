"""GPU tests of run-time FAD sequences: the fused executor and the operator-by-operator
executor against the fp64 sequence oracle, the M-result backward, the autograd wrappers.

Tolerances:
  fp32     (double-precision primitives, one rounding at the store) |got - o| <= 8 ulp32(o), plus 2^-40 (1 + |x|)
           of absolute slack for a derivative that passes through zero; inputs reach |x| = 20;
  16-bit   (plain fp32 primitives) within 1 ulp of the rounded oracle value, or within 2e-5 * max(|o|, 1 + |x|):
           a few fp32 ulp of the largest intermediate term feeding the result.
A program that forms 1 + tanh(u) literally has the cancellation that expression has: it is held to these bounds where
the expression is well conditioned, and a separate test shows that it loses digits in the tail while the fused
primitive does not.
"""
import numpy as np
import pytest
import torch

import oracle
import ulp
from paper_2209_10778_b200 import autograd as nfad_autograd
from paper_2209_10778_b200 import binding as nfad
from paper_2209_10778_b200 import sequence
from paper_2209_10778_b200 import workloads as W

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _two_result_program():
    # results: sigmoid(x) * tanh(x)   and   exp(-x^2/2-ish) + x : merges of same-source branches, M = 2
    p = sequence.FadProgram()
    x = p.x()
    a = p.mul(p.unary("sigmoid", x), p.unary("tanh", x))
    b = p.add(p.unary("exp", p.scale(-0.5, p.mul(x, x))), x)
    p.output(a)
    p.output(b)
    return p


PROGRAMS = {
    "swish": sequence.swish_program, "mish": sequence.mish_program, "gelu_tanh": sequence.gelu_tanh_program,
    "gelu_erf": sequence.gelu_erf_program, "gelu_tanh_literal": sequence.gelu_tanh_literal_program,
    "two_results": _two_result_program,
    "log1p_softplus_erf": lambda: (lambda p: (p.output(p.add(p.unary("log1p", p.unary("softplus", p.x())), p.unary("erf", p.x()))), p)[1])(sequence.FadProgram()),
}


FP32_SEQ_ULPS = 8.0


def _as_passed(ops):
    """The program as it crosses the boundary: its constants are fp32 there (nfad_seq_op.c is a float), so the oracle is
    given those very constants, not the doubles they were written as."""
    return [(o, a, b, d, float(np.float32(c))) for o, a, b, d, c in ops]


def _close(dtype, got_t, want64, x64):
    got_raw = W.raw_numpy(got_t)
    got = oracle.widen(dtype, got_raw)
    if dtype == "f32":
        return np.abs(got - want64) <= FP32_SEQ_ULPS * ulp.ulp32(want64) + 2.0 ** -40 * (1.0 + np.abs(x64))
    tol32 = 2e-5 * np.maximum(np.abs(want64), 1.0 + np.abs(x64))
    return (np.abs(got - want64) <= tol32) | (ulp.ulp_distance16(got_raw, oracle.round_to(dtype, want64)) <= 1)


def _inputs(name, dtype, n, seed):
    """N(0, 4^2) clamped to |x| <= 20 for fp32 (16-bit: |x| <= 7, where plain fp32 primitives hold their bound); the
    literal 1 + tanh program only where that sum is well conditioned."""
    lim = 20.0 if dtype == "f32" else 7.0
    x = W.normal(n, "f32", seed, 4.0 if dtype == "f32" else 2.0, DEV).clamp_(-lim, lim)
    if name == "gelu_tanh_literal":
        x = x.clamp_(min=-4.0)
    return x.to(W.TORCH_DTYPES[dtype])


@pytest.fixture(params=["interpreter", "compiled"])
def executor(request):
    """Runs a test under each of the two executors of a sequence; the compiled one must really be the one that ran."""
    nfad.nfad_seq_set_executor(request.param)
    if request.param == "compiled":
        # a machine without the run-time compiler's libraries cannot run these cases (it would use the interpreter)
        try:
            x = torch.zeros(64, device=DEV)
            sequence.run_fused(sequence.swish_program(), x)
        except nfad.NfadError:
            log = nfad.nfad_seq_compile_log()
            nfad.nfad_seq_set_executor("auto")
            if "not found" in log:
                pytest.skip(f"run-time compiler unavailable here: {log}")
            raise AssertionError(f"the compiled executor failed: {log}")
    yield request.param
    nfad.nfad_seq_set_executor("auto")


@pytest.mark.parametrize("name", list(PROGRAMS))
@pytest.mark.parametrize("dtype", ["f32", "bf16", "f16"])
def test_fused_executor_against_the_sequence_oracle(name, dtype, executor):
    prog = PROGRAMS[name]()
    n = 70001
    x = _inputs(name, dtype, n, 5)
    try:
        ys, ds = sequence.run_fused(prog, x)
    except Exception:
        print(nfad.nfad_seq_compile_log())
        raise
    torch.cuda.synchronize()
    assert nfad.nfad_seq_last_executor() == executor
    x64 = oracle.widen(dtype, W.raw_numpy(x))
    y, d = oracle.seq_forward(_as_passed(prog.ops), x64, prog.n_out)
    for k in range(prog.n_out):
        assert _close(dtype, ys[k], y[k], x64).all(), (name, dtype, "value", k)
        assert _close(dtype, ds[k], d[k], x64).all(), (name, dtype, "derivative", k)


def test_automatic_mode_compiles_and_caches():
    import time
    nfad.nfad_seq_set_executor("auto")
    p = sequence.FadProgram()
    p.output(p.unary("tanh", p.scale(0.37, p.x())))          # a program no other test uses: first call compiles
    x = W.normal(1 << 20, "bf16", 9, 1.0, DEV)
    t0 = time.perf_counter()
    sequence.run_fused(p, x)
    torch.cuda.synchronize()
    first = time.perf_counter() - t0
    assert nfad.nfad_seq_last_executor() == "compiled", nfad.nfad_seq_compile_log()
    t0 = time.perf_counter()
    for _ in range(10):
        sequence.run_fused(p, x)
    torch.cuda.synchronize()
    later = (time.perf_counter() - t0) / 10
    assert later < first / 20, (first, later)                # cached: no recompilation


@pytest.mark.parametrize("dtype", ["f32", "bf16", "f16"])
def test_fused_executor_edges_and_unaligned(dtype, executor):
    prog = sequence.swish_program()
    td = W.TORCH_DTYPES[dtype]
    for n in (1, 7, 8, 9, 255, 257, 4099):
        buf = W.normal(n + 16, dtype, n, 1.0, DEV)
        for off in (0, 1, 3):
            x = buf[off:off + n]
            yb = torch.full((n + 16,), 7.0, dtype=td, device=DEV)
            db = torch.full((n + 16,), 7.0, dtype=td, device=DEV)
            nfad.nfad_seq_forward(prog.ops, x, [yb[off:off + n]], [db[off + 1:off + 1 + n]] if off == 3 else [db[off:off + n]])
            torch.cuda.synchronize()
            x64 = oracle.widen(dtype, W.raw_numpy(x))
            y, d = oracle.seq_forward(_as_passed(prog.ops), x64, 1)
            assert _close(dtype, yb[off:off + n], y[0], x64).all()
            assert (yb[:off] == 7.0).all() and (yb[off + n:] == 7.0).all()
            dsl = db[off + 1:off + 1 + n] if off == 3 else db[off:off + n]
            assert _close(dtype, dsl, d[0], x64).all()


@pytest.mark.parametrize("dtype", ["f32", "bf16", "f16"])
def test_backward_of_a_two_result_sequence(dtype):
    prog = _two_result_program()
    n = 50003
    x = W.normal(n, dtype, 7, 1.5, DEV)
    gs = [W.normal(n, dtype, 8 + k, 1.0, DEV) for k in range(2)]
    ys, ds = sequence.run_fused(prog, x)
    gin = sequence.backward_fused(gs, ds)
    torch.cuda.synchronize()
    g64 = np.stack([oracle.widen(dtype, W.raw_numpy(g)) for g in gs])
    d64 = np.stack([oracle.widen(dtype, W.raw_numpy(d)) for d in ds])       # the GPU's own saved derivatives
    s, sa = oracle.seq_backward(g64, d64)
    got_raw = W.raw_numpy(gin)
    got = oracle.widen(dtype, got_raw)
    # fp32 accumulation of exact products: one fp32 rounding per term of size <= sa, then the store's rounding
    tol = 2.0 ** -23 * sa
    ok = np.abs(got - s) <= tol
    if dtype != "f32":
        ok |= ulp.ulp_distance16(got_raw, oracle.round_to(dtype, s)) <= 1
    assert ok.all()
    # m == 1 is the plain backward, bit for bit
    one = sequence.backward_fused(gs[:1], ds[:1])
    ref = torch.empty_like(one)
    nfad.nfad_act_backward("swish", gs[0], ds[0], ref)
    torch.cuda.synchronize()
    assert np.array_equal(W.raw_numpy(one), W.raw_numpy(ref))


@pytest.mark.parametrize("dtype", ["f32", "bf16", "f16"])
@pytest.mark.parametrize("name", ["swish", "gelu_tanh", "mish", "two_results"])
def test_operator_by_operator_executor(name, dtype):
    """One kernel per operator, every intermediate ROUNDED to the storage type on its way through memory: the bound is
    a few storage-type roundings of the largest term, not the fused executor's."""
    prog = PROGRAMS[name]()
    n = 40009
    x = W.normal(n, "f32", 9, 1.5, DEV).clamp_(-6, 6).to(W.TORCH_DTYPES[dtype])
    es = x.element_size()
    eps = {"f32": 2.0 ** -24, "bf16": 2.0 ** -8, "f16": 2.0 ** -11}[dtype]       # half a unit in the last place
    ex = sequence.OpByOp(prog)
    outs = ex.forward(x)
    kept = ex.saved_bytes()
    gs = [W.normal(n, dtype, 20 + k, 1.0, DEV) for k in range(prog.n_out)]
    gin = ex.backward(gs)
    torch.cuda.synchronize()
    x64 = oracle.widen(dtype, W.raw_numpy(x))
    y, d = oracle.seq_forward(_as_passed(prog.ops), x64, prog.n_out)
    ops_deep = 8.0                                           # roundings on the longest path of these programs
    for k in range(prog.n_out):
        got = oracle.widen(dtype, W.raw_numpy(outs[k]))
        assert (np.abs(got - y[k]) <= ops_deep * eps * np.maximum(np.abs(y[k]), 1.0 + np.abs(x64))).all(), (name, dtype, k)
    g64 = np.stack([oracle.widen(dtype, W.raw_numpy(g)) for g in gs])
    s, sa = oracle.seq_backward(g64, d)
    got = oracle.widen(dtype, W.raw_numpy(gin))
    assert (np.abs(got - s) <= 4 * ops_deep * eps * np.maximum(sa, np.abs(g64).sum(0) * (1 + np.abs(x64)))).all(), (name, dtype)
    # what operator-by-operator back-propagation keeps: Swish keeps x and sigmoid(x) (the paper's v1, v2)
    if name == "swish":
        assert kept == 2 * n * es
    assert kept >= 2 * n * es


def test_autograd_wrappers():
    n = 7 * 2859
    for kind, fn in (("gelu_erf", lambda t: nfad_autograd.gelu(t)), ("gelu_tanh", lambda t: nfad_autograd.gelu(t, "tanh")),
                     ("swish", nfad_autograd.silu), ("mish", nfad_autograd.mish)):
        x = W.normal(n, "bf16", 3, 1.5, DEV).view(7, -1).requires_grad_(True)
        g = W.normal(n, "bf16", 4, 1.0, DEV).view(7, -1)
        y = fn(x)
        y.backward(g)
        y0, d0, gin0 = torch.empty(n, dtype=x.dtype, device=DEV), torch.empty(n, dtype=x.dtype, device=DEV), torch.empty(n, dtype=x.dtype, device=DEV)
        nfad.nfad_act_forward(kind, x.detach().view(-1), y0, d0)
        nfad.nfad_act_backward(kind, g.view(-1), d0, gin0)
        torch.cuda.synchronize()
        assert torch.equal(y.detach().view(-1), y0) and torch.equal(x.grad.view(-1), gin0)
        # the conventional wrapper gives the same value and a gradient within one bf16 ulp-ish of it
        x2 = x.detach().clone().requires_grad_(True)
        y2 = nfad_autograd.ConventionalActivation.apply(x2, kind)
        y2.backward(g)
        torch.cuda.synchronize()
        if kind == "gelu_erf":      # the 16-bit erf gate has a cheaper value-only form: one unit in the last place at most
            assert (ulp.ulp_distance16(W.raw_numpy(y2.detach()), W.raw_numpy(y.detach())) <= 1).all()
        else:
            assert torch.equal(y2.detach(), y.detach())
        assert torch.allclose(x2.grad.float(), x.grad.float(), rtol=2e-2, atol=1e-3)
    # a two-result sequence through autograd
    prog = _two_result_program()
    x = W.normal(n, "f32", 5, 1.0, DEV).requires_grad_(True)
    a, b = nfad_autograd.FadSequence.apply(x, prog)
    (a.sum() * 2.0 + b.sum()).backward()
    torch.cuda.synchronize()
    x64 = x.detach().double().cpu().numpy()
    y, d = oracle.seq_forward(_as_passed(prog.ops), x64, 2)
    want = 2.0 * d[0] + d[1]
    assert np.allclose(x.grad.double().cpu().numpy(), want, rtol=2e-5, atol=2e-5)


def test_malformed_programs_are_refused():
    x = torch.zeros(64, device=DEV)
    y, d = torch.zeros(64, device=DEV), torch.zeros(64, device=DEV)
    bad = [
        [("exp", 3, 3, 1, 0.0), ("out", 1, 1, 0, 0.0)],          # reads a register nobody wrote
        [("exp", 0, 0, 1, 0.0), ("out", 1, 1, 1, 0.0)],          # result slot out of range
        [("exp", 0, 0, 0, 0.0), ("out", 0, 0, 0, 0.0)],          # writes the source register
        [("exp", 0, 0, 1, 0.0)],                                 # produces no result
        [(99, 0, 0, 1, 0.0), ("out", 1, 1, 0, 0.0)],             # unknown opcode
    ]
    for prog in bad:
        with pytest.raises(nfad.NfadError) as e:
            nfad.nfad_seq_forward(prog, x, [y], [d])
        assert e.value.status == 10
    torch.cuda.synchronize()


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_four_results_forward_and_backward(dtype, executor):
    # one source, four results (the most the interface takes): x^2, sigmoid(x), tanh(x) * x, exp(-|..|)-free softplus(x)
    p = sequence.FadProgram()
    x = p.x()
    p.output(p.mul(x, x))
    p.output(p.unary("sigmoid", x))
    p.output(p.mul(p.unary("tanh", x), x))
    p.output(p.unary("softplus", x))
    n = 40003
    xt = (W.normal(n, "f32", 15, 1.5, DEV).clamp_(-6, 6)).to(W.TORCH_DTYPES[dtype])
    ys, ds = sequence.run_fused(p, xt)
    assert nfad.nfad_seq_last_executor() == executor
    gs = [W.normal(n, dtype, 20 + k, 1.0, DEV) for k in range(4)]
    gin = sequence.backward_fused(gs, ds)
    torch.cuda.synchronize()
    x64 = oracle.widen(dtype, W.raw_numpy(xt))
    y, d = oracle.seq_forward(_as_passed(p.ops), x64, 4)
    for k in range(4):
        assert _close(dtype, ys[k], y[k], x64).all(), ("value", k)
        assert _close(dtype, ds[k], d[k], x64).all(), ("derivative", k)
    g64 = np.stack([oracle.widen(dtype, W.raw_numpy(g)) for g in gs])
    d_saved = np.stack([oracle.widen(dtype, W.raw_numpy(t)) for t in ds])
    want, want_abs = oracle.seq_backward(g64, d_saved)
    got = oracle.widen(dtype, W.raw_numpy(gin))
    tol = (2.0 ** -22 if dtype == "f32" else 2.0 ** -7) * want_abs + 1e-30
    assert (np.abs(got - want) <= tol).all()


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_large_sliced_views_use_the_whole_device(dtype, executor):
    """A view that starts one element into an allocation (every tensor sliced alike: one common offset modulo 16 bytes) and
    views that share no offset (no packet grid at all) give the same bits as aligned tensors, and the second case -- where
    every element goes through the element-wise path -- must not crawl through one CTA: it is timed against the aligned run."""
    prog = _two_result_program()
    td = W.TORCH_DTYPES[dtype]
    n = (1 << 22) + 3
    base = W.normal(n + 8, dtype, 31, 1.5, DEV)
    gbase = [W.normal(n + 8, dtype, 32 + k, 1.0, DEV) for k in range(2)]

    def run(ox, oy, od, og):
        x = base[ox:ox + n]
        ys = [torch.empty(n + 8, dtype=td, device=DEV)[oy:oy + n] for _ in range(2)]
        ds = [torch.empty(n + 8, dtype=td, device=DEV)[od:od + n] for _ in range(2)]
        gs = [g[og:og + n] for g in gbase]
        gin = torch.empty(n + 8, dtype=td, device=DEV)[ox:ox + n]
        nfad.nfad_seq_forward(prog.ops, x, ys, ds)                # warm-up (and compilation)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        nfad.nfad_seq_forward(prog.ops, x, ys, ds)
        nfad.nfad_seq_backward(gs, ds, gin)
        e1.record()
        torch.cuda.synchronize()
        # a third tensor through the one-operator kernels on the same views
        t = torch.empty(n + 8, dtype=td, device=DEV)[oy:oy + n]
        nfad.nfad_ew_op("tanh", False, 0.0, x, None, None, t)
        torch.cuda.synchronize()
        return [W.raw_numpy(v) for v in ys + ds + [t]], W.raw_numpy(gin), e0.elapsed_time(e1)

    ref, gin_ref, ms_ref = run(0, 0, 0, 0)
    same, gin_same, _ = run(1, 1, 1, 1)
    # x shifted by one element: compare against a reference computed from that very view
    x1 = base[1:1 + n].clone()                                   # aligned copy of the shifted view
    ys1 = [torch.empty(n, dtype=td, device=DEV) for _ in range(2)]
    ds1 = [torch.empty(n, dtype=td, device=DEV) for _ in range(2)]
    nfad.nfad_seq_forward(prog.ops, x1, ys1, ds1)
    t1 = torch.empty(n, dtype=td, device=DEV)
    nfad.nfad_ew_op("tanh", False, 0.0, x1, None, None, t1)
    torch.cuda.synchronize()
    want1 = [W.raw_numpy(v) for v in ys1 + ds1 + [t1]]
    for a, b in zip(same, want1):
        assert np.array_equal(a, b)
    gin1 = torch.empty(n, dtype=td, device=DEV)
    nfad.nfad_seq_backward([g[1:1 + n].clone() for g in gbase], ds1, gin1)
    torch.cuda.synchronize()
    assert np.array_equal(gin_same, W.raw_numpy(gin1))
    mixed, gin_mixed, ms_mixed = run(1, 2, 3, 1)                  # three different offsets: no common packet grid
    for a, b in zip(mixed, want1):
        assert np.array_equal(a, b)
    assert np.array_equal(gin_mixed, W.raw_numpy(gin1))
    assert nfad.nfad_seq_last_executor() == executor
    # the element-wise path over the whole grid costs a small multiple of the packet path, not the ~10^3 of one CTA
    assert ms_mixed < 40 * ms_ref, (ms_mixed, ms_ref)


def test_literal_one_plus_tanh_loses_digits_where_the_fused_primitive_does_not(executor):
    """Table I's GELU written with a literal 1 + tanh(u) against the same function with the fused (1 + tanh u)/2
    primitive, in the negative tail where tanh(u) -> -1.  fp32 storage (double-precision primitives): both agree with
    the oracle down to x = -4; from x = -6.5 on the literal sum has lost its digits (1 + tanh u < 2^-38, and the
    rounding of tanh u is 2^-53) while the fused program still holds 8 ulp.  bf16 storage (fp32 primitives): the same
    happens from x = -5 on, where 1 + tanh u is below the 2^-24 rounding of tanh u."""
    lit, fused = sequence.gelu_tanh_literal_program(), sequence.gelu_tanh_program()
    for dtype, lo, hi in (("f32", -9.0, -6.5), ("bf16", -7.0, -5.0)):
        n = 20001
        x = torch.linspace(lo, hi, n, device=DEV).to(W.TORCH_DTYPES[dtype])
        x64 = oracle.widen(dtype, W.raw_numpy(x))
        want, _ = oracle.seq_forward(_as_passed(fused.ops), x64, 1)
        (yf,), _ = sequence.run_fused(fused, x)
        (yl,), _ = sequence.run_fused(lit, x)
        torch.cuda.synchronize()
        assert _close(dtype, yf, want[0], x64).all()
        rel = np.abs(oracle.widen(dtype, W.raw_numpy(yl)) - want[0]) / np.abs(want[0])
        worst_allowed = 2.0 ** -20 if dtype == "f32" else 2.0 ** -7
        assert np.median(rel) > worst_allowed, (dtype, float(np.median(rel)))
