"""FAD sequences composed at run time, and the two ways to execute them.

A `FadProgram` is a straight-line program over dual registers (register 0 = the
source x): the run of FAD-compatible primitive operations between the paper's NY
and YN states (Section IV), with one source and M >= 1 results.

* `run_fused` executes it the nested-Forward-AD way: ONE kernel, dual numbers in
  registers, and per result only y_k and dy_k/dx reach memory (the saved tensor).
* `OpByOp` executes the same program the way plain back-propagation does when every
  operator is a node of the graph (Section II-C approach 1): one kernel per
  operator, every intermediate is a tensor, every operator keeps what its own
  backward rule needs.  It exists to MEASURE that layout: kept bytes and time.

Both call the CUDA library through the binding; nothing is computed in Python.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence, Tuple

import torch

from . import binding as nfad

_UNARY = ("exp", "log1p", "tanh", "erf", "softplus", "sigmoid", "half_one_plus_tanh", "half_one_plus_erf")
# what each operator's backward rule keeps: "in" = its input, "out" = its output, "both" = both operands
_KEEPS = {"mul": "both", "exp": "out", "log1p": "in", "tanh": "out", "erf": "in", "softplus": "in", "sigmoid": "out",
          "half_one_plus_tanh": "out", "half_one_plus_erf": "in", "add": None, "scale": None, "add_const": None}


@dataclass
class FadProgram:
    ops: List[Tuple[str, int, int, int, float]] = field(default_factory=list)
    n_regs: int = 1          # register 0 is x
    n_out: int = 0

    def _new(self) -> int:
        if self.n_regs >= 12:
            raise ValueError("a FAD sequence has 12 registers")
        self.n_regs += 1
        return self.n_regs - 1

    def x(self) -> int:
        return 0

    def add(self, a: int, b: int) -> int:
        d = self._new(); self.ops.append(("add", a, b, d, 0.0)); return d

    def mul(self, a: int, b: int) -> int:
        d = self._new(); self.ops.append(("mul", a, b, d, 0.0)); return d

    def scale(self, c: float, a: int) -> int:
        d = self._new(); self.ops.append(("scale", a, a, d, float(c))); return d

    def add_const(self, c: float, a: int) -> int:
        d = self._new(); self.ops.append(("add_const", a, a, d, float(c))); return d

    def unary(self, name: str, a: int) -> int:
        if name not in _UNARY:
            raise ValueError(name)
        d = self._new(); self.ops.append((name, a, a, d, 0.0)); return d

    def output(self, a: int) -> int:
        self.ops.append(("out", a, a, self.n_out, 0.0))
        self.n_out += 1
        return self.n_out - 1


def swish_program() -> FadProgram:
    p = FadProgram(); x = p.x(); p.output(p.mul(x, p.unary("sigmoid", x))); return p


def mish_program() -> FadProgram:
    p = FadProgram(); x = p.x(); p.output(p.mul(x, p.unary("tanh", p.unary("softplus", x)))); return p


def gelu_tanh_program() -> FadProgram:
    """Table I: 0.5 x (1 + tanh(sqrt(2/pi) (x + 0.044715 x^3))), with the (1 + tanh)/2 fusion."""
    p = FadProgram(); x = p.x()
    b = p.add_const(1.0, p.scale(0.044715, p.mul(x, x)))
    u = p.scale(0.7978845608028654, p.mul(x, b))
    p.output(p.mul(x, p.unary("half_one_plus_tanh", u)))
    return p


def gelu_erf_program() -> FadProgram:
    p = FadProgram(); x = p.x()
    p.output(p.mul(x, p.unary("half_one_plus_erf", p.scale(0.7071067811865476, x))))
    return p


def gelu_tanh_literal_program() -> FadProgram:
    """The same function written with plain tanh, 1 + and 0.5 *: what a user's code looks like."""
    p = FadProgram(); x = p.x()
    x3 = p.mul(x, p.mul(x, x))
    u = p.scale(0.7978845608028654, p.add(x, p.scale(0.044715, x3)))
    p.output(p.mul(p.scale(0.5, x), p.add_const(1.0, p.unary("tanh", u))))
    return p


PROGRAMS = {"swish": swish_program, "mish": mish_program, "gelu_tanh": gelu_tanh_program, "gelu_erf": gelu_erf_program}


def run_fused(prog: FadProgram, x: torch.Tensor):
    """(ys, dfdxs): every result and its derivative, from one kernel."""
    ys = [torch.empty_like(x) for _ in range(prog.n_out)]
    ds = [torch.empty_like(x) for _ in range(prog.n_out)]
    nfad.nfad_seq_forward(prog.ops, x, ys, ds)
    return ys, ds


def backward_fused(grad_outs: Sequence[torch.Tensor], dfdxs: Sequence[torch.Tensor]) -> torch.Tensor:
    gin = torch.empty_like(grad_outs[0])
    nfad.nfad_seq_backward(list(grad_outs), list(dfdxs), gin)
    return gin


class OpByOp:
    """Runs a FadProgram one operator per kernel, keeping what each backward rule needs."""

    def __init__(self, prog: FadProgram):
        self.prog = prog
        self.kept: Dict[int, torch.Tensor] = {}     # id(tensor) -> tensor kept alive for backward
        self.tape: List[Tuple[str, int, int, int, float, Optional[torch.Tensor], Optional[torch.Tensor]]] = []

    def forward(self, x: torch.Tensor) -> List[torch.Tensor]:
        regs: Dict[int, torch.Tensor] = {0: x}
        outs: List[Optional[torch.Tensor]] = [None] * self.prog.n_out
        self.kept.clear()
        self.tape.clear()
        for name, a, b, dst, c in self.prog.ops:
            if name == "out":
                outs[dst] = regs[a]
                continue
            out = torch.empty_like(x)
            if name in ("add", "mul"):
                nfad.nfad_ew_op(name, False, c, regs[a], regs[b], None, out)
            else:
                nfad.nfad_ew_op(name, False, c, regs[a], None, None, out)
            regs[dst] = out
            keep = _KEEPS[name]
            s0 = s1 = None
            if keep == "both":
                s0, s1 = regs[a], regs[b]
            elif keep == "in":
                s0 = regs[a]
            elif keep == "out":
                s0 = out
            for t in (s0, s1):
                if t is not None:
                    self.kept[id(t)] = t
            self.tape.append((name, a, b, dst, c, s0, s1))
        return outs  # type: ignore[return-value]

    def saved_bytes(self) -> int:
        return sum(t.numel() * t.element_size() for t in self.kept.values())

    def backward(self, grad_outs: Sequence[torch.Tensor]) -> torch.Tensor:
        grads: Dict[int, torch.Tensor] = {}

        def accumulate(reg: int, g: torch.Tensor):
            if reg in grads:
                s = torch.empty_like(g)
                nfad.nfad_ew_op("add", False, 0.0, grads[reg], g, None, s)
                grads[reg] = s
            else:
                grads[reg] = g

        k = 0
        for name, a, b, dst, c in self.prog.ops:
            if name == "out":
                accumulate(a, grad_outs[dst])
        for name, a, b, dst, c, s0, s1 in reversed(self.tape):
            g = grads.pop(dst, None)
            if g is None:
                continue
            if name == "add":
                accumulate(a, g); accumulate(b, g)
            elif name == "add_const":
                accumulate(a, g)
            elif name == "mul":
                ga, gb = torch.empty_like(g), torch.empty_like(g)
                nfad.nfad_ew_op("mul", True, c, g, s0, s1, ga, gb)
                accumulate(a, ga); accumulate(b, gb)
            else:
                ga = torch.empty_like(g)
                nfad.nfad_ew_op(name, True, c, g, s0, None, ga)
                accumulate(a, ga)
        self.kept.clear()
        self.tape.clear()
        return grads[0]
