"""Parity at the largest sizes, in the launch configuration the benchmark times.

The 12-layer-stack tensor (100.7M bf16 elements) is compared in full.  At 2^30 fp32 elements
and beyond 2^31 bf16 elements (64-bit indexing) the oracle is run on a sample: an element-wise
pass is correct on a tensor iff it is correct on every element, so the sample is chosen to hit
what can differ by position -- the first and last packets, elements around tile boundaries and
around multiples of 2^31 and 2^32 bytes, and a stride coprime to every tile size."""
import numpy as np
import pytest
import torch

import parity
from paper_2209_10778_b200 import binding as nfad
from paper_2209_10778_b200 import workloads as W

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _sample_indices(n: int, es: int) -> torch.Tensor:
    idx = [torch.arange(0, min(n, 20000)), torch.arange(max(0, n - 20000), n), torch.arange(0, n, 100003)]
    for packets in (4, 5):                           # elements per tile: 256 threads x 4 (or, 16-bit forward, 5) packets
        per_tile = 256 * packets * 16 // es
        for k in (1, 2, 3, 1000, n // per_tile - 1, n // per_tile):
            c = k * per_tile
            idx.append(torch.arange(max(0, c - 40), min(n, c + 40)))
    for byte_mark in (1 << 31, 1 << 32, 3 << 31):
        c = byte_mark // es
        if 40 < c < n - 40:
            idx.append(torch.arange(c - 40, c + 40))
    return torch.unique(torch.cat(idx)).to(DEV)


def _sampled_check(kind: str, dtype: str, n: int, dist: str):
    x = W.draw(dist, n, dtype, 300, DEV)
    g = W.normal(n, dtype, 301, 1.0, DEV)
    y, d = parity.gpu_forward(kind, x)
    gin = parity.gpu_backward(kind, g, d)
    torch.cuda.synchronize()
    idx = _sample_indices(n, x.element_size())
    xs, gs, ys, ds, gis = (W.raw_numpy(t[idx]) for t in (x, g, y, d, gin))
    if dtype == "f32":
        parity.check_forward_fp32(kind, xs, ys, ds)
    else:
        parity.check_forward_16(kind, dtype, xs, ys, ds)
    parity.check_backward(dtype, gs, ds, gis)
    # properties that hold at any size, over the whole tensor: finite, sign of y follows x, f' within its range
    assert bool(torch.isfinite(y).all()) and bool(torch.isfinite(d).all()) and bool(torch.isfinite(gin).all())
    assert float(d.float().max()) <= 1.2 and float(d.float().min()) >= -0.2
    del x, g, y, d, gin
    torch.cuda.empty_cache()


def test_stack_tensor_full_compare():
    w = W.WORKLOADS["gelu_stack_12"]
    x, g = W.workload_tensors(w, 0, DEV)
    parity.full_check("gelu_erf", w.dtype, x, g)


def test_fp32_two_to_the_thirty_sampled():
    _sampled_check("mish", "f32", 1 << 30, "normal")


def test_bf16_beyond_two_to_the_thirty_one_elements_sampled():
    _sampled_check("gelu_tanh", "bf16", (1 << 31) + 5, "normal")


def test_fp16_quarter_billion_mix_sampled():
    _sampled_check("swish", "f16", 1 << 28, "mix")


def test_bert_ffn_step_replayed_from_a_cuda_graph():
    # the benchmark's launch configuration: the step's four launches (programmatic dependent launch between them)
    # captured in a CUDA graph and replayed; every element of both kinds against the oracle
    w = W.WORKLOADS["bert_base_ffn"]
    x, g = W.workload_tensors(w, 0, DEV)
    bufs = {k: [torch.empty_like(x) for _ in range(3)] for k in w.kinds}

    def step():
        for k in w.kinds:
            y, d, gin = bufs[k]
            nfad.nfad_act_forward(k, x, y, d)
            nfad.nfad_act_backward(k, g, d, gin)

    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        step()
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    for k in w.kinds:
        for t in bufs[k]:
            t.zero_()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step()
    graph.replay()
    graph.replay()
    torch.cuda.synchronize()
    x_raw, g_raw = W.raw_numpy(x), W.raw_numpy(g)
    for k in w.kinds:
        y, d, gin = (W.raw_numpy(t) for t in bufs[k])
        parity.check_forward_16(k, w.dtype, x_raw, y, d)
        parity.check_backward(w.dtype, g_raw, d, gin)
