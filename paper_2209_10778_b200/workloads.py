"""Seeded synthetic inputs shaped like the paper's workloads.

This module holds NO arithmetic of the method: it only draws numbers and names
tensor shapes.  It is the one module that both the CUDA path's callers and the
CPU oracle's callers use, so that both see the same arrays.

The paper trains BERT-base (sequence length 128, GLUE) and ResNet-50 (ImageNet)
with GELU / Mish / Swish (Section V-A).  Neither dataset nor any weight is
needed by an element-wise pass: only the shapes of the activation tensors and a
plausible value distribution matter, so seeded Gaussian / uniform / tail-heavy
draws of those shapes stand in for them.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Sequence, Tuple

import torch

TORCH_DTYPES = {"f32": torch.float32, "bf16": torch.bfloat16, "f16": torch.float16}
KINDS = ("gelu_erf", "gelu_tanh", "swish", "mish")
DTYPES = ("f32", "bf16", "f16")

# Where each derivative changes sign (x < 0), to ~17 digits; used only to place
# probe points next to the cancellation, never to compute anything.
FPRIME_ROOTS = {
    "gelu_erf": -0.751791524693564,
    "gelu_tanh": -0.752461422071016,
    "swish": -1.278464542761074,
    "mish": -1.192431214515495,
}


@dataclass(frozen=True)
class Workload:
    """One named configuration: tensor shapes, storage type, activations, value recipe."""
    name: str
    dtype: str
    kinds: Tuple[str, ...]
    shapes: Tuple[Tuple[int, ...], ...]
    x_std: float = 1.0
    g_std: float = 1.0
    x_seed: int = 0
    g_seed: int = 1
    layers: int = 1
    note: str = ""

    def numel(self, i: int = 0) -> int:
        return math.prod(self.shapes[i])


WORKLOADS = {
    # a single fp32 vector: parity case the oracle finishes in a blink
    "gelu_erf_f32_1m": Workload("gelu_erf_f32_1m", "f32", ("gelu_erf",), ((1 << 20,),)),
    # BERT-base feed-forward activation: batch 32, sequence 128, hidden 3072
    "bert_base_ffn": Workload("bert_base_ffn", "bf16", ("gelu_erf", "gelu_tanh"), ((32, 128, 3072),),
                              x_std=1.5, g_std=1e-2),
    # ResNet-50 stage outputs, NCHW, batch 64, with Mish / Swish in place of ReLU
    "resnet50_stages": Workload("resnet50_stages", "f16", ("mish", "swish"),
                                ((64, 64, 112, 112), (64, 256, 56, 56), (64, 512, 28, 28),
                                 (64, 1024, 14, 14), (64, 2048, 7, 7))),
    # one feed-forward activation tensor of the 12-layer stack below (100.7M elements, 192 MiB: larger than L2),
    # both GELU forms: the size class the bandwidth target is stated on
    "gelu_ffn_100m": Workload("gelu_ffn_100m", "bf16", ("gelu_erf", "gelu_tanh"), ((64, 512, 3072),)),
    # 12 stacked GELU layers on [64, 512, 3072]
    "gelu_stack_12": Workload("gelu_stack_12", "bf16", ("gelu_erf",), ((64, 512, 3072),), layers=12),
}

SWEEP_SIZES = tuple(1 << p for p in range(16, 31, 2))       # 2^16 ... 2^30, powers of 4
SWEEP_DISTRIBUTIONS = ("normal", "uniform20", "mix")


def _gen(device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def normal(n: int, dtype: str, seed: int, std: float = 1.0, device="cpu") -> torch.Tensor:
    """N(0, std^2): drawn in fp32, scaled, rounded to nearest-even into the storage type."""
    v = torch.randn(n, generator=_gen(device, seed), device=device, dtype=torch.float32)
    if std != 1.0:
        v = v * std
    return v.to(TORCH_DTYPES[dtype])


def uniform(n: int, dtype: str, seed: int, lo: float = -20.0, hi: float = 20.0, device="cpu") -> torch.Tensor:
    v = torch.rand(n, generator=_gen(device, seed), device=device, dtype=torch.float32)
    return (v * (hi - lo) + lo).to(TORCH_DTYPES[dtype])


def log_uniform_signed(n: int, dtype: str, seed: int, lo: float = 1e-6, hi: float = 80.0, device="cpu") -> torch.Tensor:
    """Sign * exp(U(ln lo, ln hi)): magnitudes from tiny to where exp(|x|) nears fp32 overflow."""
    g = _gen(device, seed)
    u = torch.rand(n, generator=g, device=device, dtype=torch.float32)
    s = torch.rand(n, generator=g, device=device, dtype=torch.float32)
    mag = torch.exp(u * (math.log(hi) - math.log(lo)) + math.log(lo)).clamp_(max=hi)
    return torch.where(s < 0.5, -mag, mag).to(TORCH_DTYPES[dtype])


def special_values(dtype: str) -> torch.Tensor:
    """Finite probe points: signed zeros, smallest subnormal/normal, +-1, each derivative's
    sign change with its two neighbours in the storage type, +-sqrt2, the band where the
    erf-GELU result turns subnormal in fp32, and saturated-tail magnitudes up to 80."""
    td = TORCH_DTYPES[dtype]
    fi = torch.finfo(td)
    vals: List[float] = [0.0, -0.0, fi.tiny, -fi.tiny, 1.0, -1.0,
                         math.sqrt(2.0), -math.sqrt(2.0), 20.0, -20.0, 40.0, -40.0, 80.0, -80.0]
    out = torch.tensor(vals, dtype=torch.float64).to(td)
    # smallest subnormal of the format, both signs
    one = torch.tensor([1], dtype=torch.int16 if td != torch.float32 else torch.int32)
    sub = one.view(td)
    out = torch.cat([out, sub, -sub])
    # neighbours of each root and of 80, via the integer ordering of the bit patterns
    it = torch.int32 if td == torch.float32 else torch.int16
    centres = torch.tensor(list(FPRIME_ROOTS.values()) + [80.0, -80.0], dtype=torch.float64).to(td)
    bits = centres.view(it)
    neigh = torch.cat([bits - 1, bits, bits + 1]).view(td)
    band = torch.arange(-14.5, -12.95, 0.1, dtype=torch.float64).to(td)
    return torch.cat([out, neigh, band])


def mix(n: int, dtype: str, seed: int, device="cpu") -> torch.Tensor:
    """Element i takes, by i mod 4: N(0,1) / U(-20,20) / +-log-uniform |x| in [1e-6, 80] /
    the cycled list of special values."""
    q = (n + 3) // 4
    a = normal(q, dtype, seed, 1.0, device)
    b = uniform(q, dtype, seed + 1000, -20.0, 20.0, device)
    c = log_uniform_signed(q, dtype, seed + 2000, 1e-6, 80.0, device)
    sp = special_values(dtype).to(device)
    d = sp[torch.arange(q, device=device) % sp.numel()]
    return torch.stack([a, b, c, d], dim=1).reshape(-1)[:n].contiguous()


def draw(dist: str, n: int, dtype: str, seed: int, device="cpu") -> torch.Tensor:
    if dist == "normal":
        return normal(n, dtype, seed, 1.0, device)
    if dist == "uniform20":
        return uniform(n, dtype, seed, -20.0, 20.0, device)
    if dist == "mix":
        return mix(n, dtype, seed, device)
    raise ValueError(f"unknown distribution {dist!r}")


def workload_tensors(w: Workload, shape_index: int = 0, device="cpu") -> Tuple[torch.Tensor, torch.Tensor]:
    """(x, grad_out) for one shape of a workload, flat, in the workload's storage type."""
    n = w.numel(shape_index)
    x = normal(n, w.dtype, w.x_seed + 17 * shape_index, w.x_std, device)
    g = normal(n, w.dtype, w.g_seed + 17 * shape_index, w.g_std, device)
    return x, g


def all_finite_16bit(dtype: str) -> torch.Tensor:
    """Every finite value of a 16-bit storage type (65 280 for bf16, 63 488 for fp16)."""
    td = TORCH_DTYPES[dtype]
    bits = torch.arange(-32768, 32768, dtype=torch.int32).to(torch.int16)
    v = bits.view(td)
    return v[torch.isfinite(v.to(torch.float32))].contiguous()


def raw_numpy(t: torch.Tensor):
    """A tensor's stored values as a host numpy array of raw bit patterns
    (float32 for fp32, uint16 for bf16 / fp16): marshalling only."""
    import numpy as np
    t = t.detach().reshape(-1).cpu().contiguous()
    if t.dtype == torch.float32:
        return t.numpy()
    return t.view(torch.int16).numpy().view(np.uint16)


def from_raw_numpy(a, dtype: str, device="cpu") -> torch.Tensor:
    import numpy as np
    if dtype == "f32":
        return torch.from_numpy(np.ascontiguousarray(a, np.float32)).to(device)
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).view(TORCH_DTYPES[dtype]).to(device)
