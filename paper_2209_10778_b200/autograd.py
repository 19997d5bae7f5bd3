"""`torch.autograd.Function` wrappers: the paper's YN post-process in PyTorch terms
(Section IV, component C: the saved tensor of the node becomes the FAD result, and its
backward function becomes a direct multiplication).  The wrappers only allocate tensors
and call the CUDA library.
"""
from __future__ import annotations

import torch

from . import binding as nfad
from . import sequence


class NestedActivation(torch.autograd.Function):
    """y = f(x) with f'(x) as the only saved tensor; backward = grad_out * f'(x)."""

    @staticmethod
    def forward(ctx, x: torch.Tensor, kind: str):
        xc = x.contiguous()
        y = torch.empty_like(xc)
        d = torch.empty_like(xc)
        nfad.nfad_act_forward(kind, xc.view(-1), y.view(-1), d.view(-1))
        ctx.save_for_backward(d)
        ctx.kind = kind
        return y

    @staticmethod
    def backward(ctx, grad_out: torch.Tensor):
        (d,) = ctx.saved_tensors
        g = grad_out.contiguous()
        gin = torch.empty_like(g)
        nfad.nfad_act_backward(ctx.kind, g.view(-1), d.view(-1), gin.view(-1))
        return gin, None


class NestedBiasActivation(torch.autograd.Function):
    """y = f(x + bias) for x of shape [..., cols] and bias of shape [cols]: f'(x + bias) is the only saved tensor;
    backward gives grad_x = grad_out * f' and grad_bias = its column sums, from one kernel."""

    @staticmethod
    def forward(ctx, x: torch.Tensor, bias: torch.Tensor, kind: str):
        xc, bc = x.contiguous(), bias.contiguous()
        y = torch.empty_like(xc)
        d = torch.empty_like(xc)
        nfad.nfad_bias_act_forward(kind, xc.view(-1), bc, y.view(-1), d.view(-1))
        ctx.save_for_backward(d)
        ctx.kind, ctx.cols, ctx.bias_dtype = kind, bc.numel(), bias.dtype
        return y

    @staticmethod
    def backward(ctx, grad_out: torch.Tensor):
        (d,) = ctx.saved_tensors
        g = grad_out.contiguous()
        gin = torch.empty_like(g)
        gb = torch.empty(ctx.cols, dtype=torch.float32, device=g.device)
        nbytes = nfad.nfad_bias_act_backward_scratch_bytes(g.dtype, g.numel() // ctx.cols, ctx.cols, g.device)
        scratch = torch.empty(nbytes, dtype=torch.uint8, device=g.device) if nbytes else None
        nfad.nfad_bias_act_backward(ctx.kind, g.view(-1), d.view(-1), gin.view(-1), gb, scratch)
        return gin, gb.to(ctx.bias_dtype), None


class ConventionalActivation(torch.autograd.Function):
    """The comparator that saves x and re-derives f'(x) in one fused backward kernel."""

    @staticmethod
    def forward(ctx, x: torch.Tensor, kind: str):
        xc = x.contiguous()
        y = torch.empty_like(xc)
        nfad.nfad_act_forward_infer(kind, xc.view(-1), y.view(-1))
        ctx.save_for_backward(xc)
        ctx.kind = kind
        return y

    @staticmethod
    def backward(ctx, grad_out: torch.Tensor):
        (x,) = ctx.saved_tensors
        g = grad_out.contiguous()
        gin = torch.empty_like(g)
        nfad.nfad_cmp_conv_backward(ctx.kind, g.view(-1), x.view(-1), gin.view(-1))
        return gin, None


class FadSequence(torch.autograd.Function):
    """A run-time FAD sequence with M results: saves one derivative tensor per result."""

    @staticmethod
    def forward(ctx, x: torch.Tensor, prog: sequence.FadProgram):
        xc = x.contiguous()
        ys, ds = sequence.run_fused(prog, xc.view(-1))
        ctx.save_for_backward(*ds)
        ctx.shape = xc.shape
        return tuple(y.view(xc.shape) for y in ys)

    @staticmethod
    def backward(ctx, *grad_outs):
        ds = ctx.saved_tensors
        gs = [g.contiguous().view(-1) for g in grad_outs]
        return sequence.backward_fused(gs, list(ds)).view(ctx.shape), None


def bias_gelu(x, bias, approximate: str = "none"):
    return NestedBiasActivation.apply(x, bias, "gelu_tanh" if approximate == "tanh" else "gelu_erf")


def gelu(x, approximate: str = "none"):
    return NestedActivation.apply(x, "gelu_tanh" if approximate == "tanh" else "gelu_erf")


def silu(x):
    return NestedActivation.apply(x, "swish")


def mish(x):
    return NestedActivation.apply(x, "mish")
