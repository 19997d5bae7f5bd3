"""GPU parity: the CUDA path, called through the C-ABI binding, against the fp64
oracle on the same seeded arrays.  Sizes span many tiles (one tile = 4096 fp32 or
8192 16-bit elements) plus a ragged tail."""
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


def test_config_gelu_erf_fp32_1m():
    # GELU (erf) on one fp32 vector of 2^20 elements, x ~ N(0,1) seed 0, g ~ N(0,1) seed 1
    w = W.WORKLOADS["gelu_erf_f32_1m"]
    x, g = W.workload_tensors(w, 0, DEV)
    stats = {}
    parity.full_check("gelu_erf", "f32", x, g, stats)
    print("gelu_erf f32 2^20:", stats)


@pytest.mark.parametrize("kind", KINDS)
@pytest.mark.parametrize("dist", W.SWEEP_DISTRIBUTIONS)
def test_fp32_all_kinds_all_distributions(kind, dist):
    n = (1 << 18) + 37
    x = W.draw(dist, n, "f32", 100, DEV)
    g = W.normal(n, "f32", 101, 1.0, DEV)
    stats = {}
    parity.full_check(kind, "f32", x, g, stats)
    print(kind, dist, stats)


@pytest.mark.parametrize("kind", KINDS)
@pytest.mark.parametrize("dtype", ["bf16", "f16"])
@pytest.mark.parametrize("dist", W.SWEEP_DISTRIBUTIONS)
def test_16bit_all_kinds_all_distributions(kind, dtype, dist):
    n = (1 << 18) + 37
    x = W.draw(dist, n, dtype, 200, DEV)
    g = W.normal(n, dtype, 201, 1.0, DEV)
    stats = {}
    parity.full_check(kind, dtype, x, g, stats)
    print(kind, dtype, dist, stats)


@pytest.mark.parametrize("kind", KINDS)
@pytest.mark.parametrize("dtype", ["bf16", "f16"])
def test_every_finite_16bit_input(kind, dtype):
    # exhaustive: 65 280 bf16 / 63 488 fp16 inputs, restricted to the configs' |x| <= 80.5 for the
    # gate and checked for finiteness beyond
    x_all = W.all_finite_16bit(dtype).to(DEV)
    y, d = parity.gpu_forward(kind, x_all)
    torch.cuda.synchronize()
    assert torch.isfinite(y.float()).all() and torch.isfinite(d.float()).all()
    x = x_all[x_all.float().abs() <= 80.5].contiguous()
    g = W.normal(x.numel(), dtype, 5, 1.0, DEV)
    stats = {}
    parity.full_check(kind, dtype, x, g, stats)
    print(kind, dtype, "exhaustive", x.numel(), stats)


@pytest.mark.parametrize("name", ["bert_base_ffn", "resnet50_stages"])
def test_workload_shapes_full_size(name):
    w = W.WORKLOADS[name]
    for si in range(len(w.shapes)):
        x, g = W.workload_tensors(w, si, DEV)
        for kind in w.kinds:
            parity.full_check(kind, w.dtype, x, g)


def test_backward_bf16_products_below_fp32_normal_range():
    # products that land under 2^-126 must still be ONE rounding of the exact product
    rng = np.random.default_rng(3)
    a = np.exp(rng.uniform(np.log(1e-30), np.log(1e-10), 50000)) * rng.choice([-1, 1], 50000)
    b = np.exp(rng.uniform(np.log(1e-30), np.log(1e-8), 50000)) * rng.choice([-1, 1], 50000)
    g_raw, d_raw = oracle.round_to("bf16", a), oracle.round_to("bf16", b)
    g = W.from_raw_numpy(g_raw, "bf16", DEV)
    d = W.from_raw_numpy(d_raw, "bf16", DEV)
    gin = parity.gpu_backward("swish", g, d)
    torch.cuda.synchronize()
    parity.check_backward("bf16", g_raw, d_raw, W.raw_numpy(gin))


@pytest.mark.parametrize("dtype", ["f32", "bf16", "f16"])
def test_backward_extreme_values(dtype):
    td = W.TORCH_DTYPES[dtype]
    fi = torch.finfo(td)
    vals = torch.tensor([0.0, -0.0, fi.tiny, -fi.tiny, fi.max, -fi.max, 1.0, -1.0, 0.5, 3.0, fi.eps, 1e-3, 1e3],
                        dtype=torch.float64).to(td)
    sub = torch.tensor([1, 2, 3], dtype=torch.int32 if dtype == "f32" else torch.int16).view(td)
    vals = torch.cat([vals, sub, -sub])
    g = vals.repeat_interleave(vals.numel()).to(DEV)
    d = vals.repeat(vals.numel()).to(DEV)
    gin = parity.gpu_backward("mish", g, d)
    torch.cuda.synchronize()
    parity.check_backward(dtype, W.raw_numpy(g), W.raw_numpy(d), W.raw_numpy(gin))


@pytest.mark.parametrize("kind", KINDS)
@pytest.mark.parametrize("dtype", ["f32", "bf16", "f16"])
def test_infer_against_the_oracle_and_the_training_value(kind, dtype):
    """The value-only pass is held to the oracle like the training pass.  It gives the training pass's very bits wherever it
    runs the same chain; the 16-bit erf gate has a cheaper value-only form (a lower-degree fit, good to a quarter of an fp16
    ulp), whose results may differ from the training value by one unit in the last place, never more."""
    n = 70001
    x = W.draw("mix", n, dtype, 7, DEV)
    y, _ = parity.gpu_forward(kind, x)
    y2 = torch.empty_like(x)
    nfad.nfad_act_forward_infer(kind, x, y2)
    torch.cuda.synchronize()
    x_raw, y2_raw = W.raw_numpy(x), W.raw_numpy(y2)
    if dtype == "f32":
        assert np.array_equal(W.raw_numpy(y), y2_raw)
    else:
        f, _ = oracle.forward(kind, dtype, x_raw)
        dist = ulp.ulp_distance16(y2_raw, oracle.round_to(dtype, f))
        assert (dist <= 1).all() and not ulp.is_nan16(y2_raw, dtype).any()
        if kind == "gelu_erf":
            assert (ulp.ulp_distance16(y2_raw, W.raw_numpy(y)) <= 1).all()
        else:
            assert np.array_equal(W.raw_numpy(y), y2_raw)


@pytest.mark.parametrize("kind", KINDS)
@pytest.mark.parametrize("dtype", ["f32", "bf16", "f16"])
def test_non_finite_inputs(kind, dtype):
    td = W.TORCH_DTYPES[dtype]
    x = torch.tensor([float("nan"), float("inf"), -float("inf"), 3e38, -3e38, 1e4, -1e4], dtype=torch.float32).to(td).to(DEV)
    y, d = parity.gpu_forward(kind, x)
    torch.cuda.synchronize()
    y, d = y.float().cpu(), d.float().cpu()
    assert torch.isnan(y[0]) and torch.isnan(d[0])
    assert y[1] == float("inf") and d[1] == 1.0
    assert y[2] == 0.0 and d[2] == 0.0
    xf = x.float().cpu()
    for i in (3, 5):
        assert y[i] == xf[i] and d[i] == 1.0
    for i in (4, 6):
        assert y[i] == 0.0 and d[i] == 0.0


def test_backward_bf16_products_that_round_to_signed_zero_or_the_smallest_subnormal():
    # products between 2^-150 and 2^-130: fp32 cannot hold them exactly, the bf16 result is +-0 or a few subnormals;
    # the bits (sign of a zero included) must be those of ONE rounding of the exact product
    rng = np.random.default_rng(11)
    n = 200000
    a = 2.0 ** rng.uniform(-80, -60, n) * rng.choice([-1, 1], n)
    b = 2.0 ** rng.uniform(-72, -66, n) * rng.choice([-1, 1], n)
    g_raw, d_raw = oracle.round_to("bf16", a), oracle.round_to("bf16", b)
    g = W.from_raw_numpy(g_raw, "bf16", DEV)
    d = W.from_raw_numpy(d_raw, "bf16", DEV)
    gin = parity.gpu_backward("gelu_erf", g, d)
    torch.cuda.synchronize()
    got = W.raw_numpy(gin)
    parity.check_backward("bf16", g_raw, d_raw, got)
    assert (got == 0x8000).any() and (got == 0x0000).any() and ((got & 0x7FFF) == 1).any()   # the cases are really there
