"""Thin ctypes binding over libnfad.so: same names as the C interface
(``include/nfad.h``), argument marshalling only.  Every step of the path runs
in the library's CUDA kernels; there is no fallback of any kind: if the
library cannot be loaded, or a tensor is not a contiguous CUDA tensor of a
supported type, the call raises.

PyTorch appears here only as the owner of device memory and streams.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

KINDS = {"gelu_erf": 0, "gelu_tanh": 1, "swish": 2, "mish": 3}
DTYPES = {"f32": 0, "bf16": 1, "f16": 2}
LAYOUTS = {"nested": 0, "conventional": 1, "recompute": 2, "op_by_op": 3}
_TORCH_TO_CODE = {torch.float32: 0, torch.bfloat16: 1, torch.float16: 2}

NFAD_OK = 0

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libnfad.so")

EXPORTS = (
    "nfad_act_forward", "nfad_act_forward_infer", "nfad_act_backward",
    "nfad_cmp_conv_backward", "nfad_cmp_recompute_backward", "nfad_cmp_recompute_scratch_bytes",
    "nfad_saved_bytes_per_element", "nfad_last_cuda_error", "nfad_status_string", "nfad_version",
    "nfad_probe_stream", "nfad_cmp_recompute_backward_noalloc",
    "nfad_seq_forward", "nfad_seq_backward", "nfad_ew_op",
    "nfad_bias_act_forward", "nfad_bias_act_forward_infer", "nfad_bias_act_backward", "nfad_bias_act_backward_scratch_bytes",
    "nfad_act_forward_strict",
    "nfad_host_step", "nfad_host_step_workspace_bytes",
    "nfad_seq_set_executor", "nfad_seq_last_executor", "nfad_seq_compile_log", "nfad_seq_compiled_source",
)
OPCODES = {"add": 0, "mul": 1, "scale": 2, "add_const": 3, "exp": 4, "log1p": 5, "tanh": 6, "erf": 7, "softplus": 8,
           "sigmoid": 9, "half_one_plus_tanh": 10, "half_one_plus_erf": 11, "out": 12}


class SeqOp(ctypes.Structure):
    """One instruction of a FAD sequence: `nfad_seq_op` of the C interface."""
    _fields_ = [("op", ctypes.c_int), ("a", ctypes.c_int), ("b", ctypes.c_int), ("dst", ctypes.c_int), ("c", ctypes.c_float)]
NOALLOC_SCRATCH_BYTES = 8388608

_lib: Optional[ctypes.CDLL] = None


class NfadError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        lib = load()
        msg = lib.nfad_status_string(status).decode()
        if status == 5:
            msg += f" [cudaError {lib.nfad_last_cuda_error()}]"
        super().__init__(f"{where}: {msg} (status {status})")


def load() -> ctypes.CDLL:
    """Loads libnfad.so from the package directory.  Raises if it has not been built
    (``python -m paper_2209_10778_b200.build``): nothing else can run the path."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2209_10778_b200.build` "
                              "(needs nvcc); there is no other implementation of the path")
        lib = ctypes.CDLL(LIB_PATH)
        vp, sz, ci = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int
        lib.nfad_act_forward.argtypes = [ci, ci, vp, vp, vp, sz, vp]
        lib.nfad_act_forward_strict.argtypes = [ci, ci, vp, vp, vp, sz, vp]
        lib.nfad_act_forward_strict.restype = ci
        lib.nfad_act_forward_infer.argtypes = [ci, ci, vp, vp, sz, vp]
        lib.nfad_act_backward.argtypes = [ci, ci, vp, vp, vp, sz, vp]
        lib.nfad_cmp_conv_backward.argtypes = [ci, ci, vp, vp, vp, sz, vp]
        lib.nfad_cmp_recompute_backward.argtypes = [ci, ci, vp, vp, vp, sz, vp, sz, vp]
        lib.nfad_cmp_recompute_backward_noalloc.argtypes = [ci, ci, vp, vp, vp, sz, vp]
        lib.nfad_cmp_recompute_backward_noalloc.restype = ci
        lib.nfad_seq_forward.argtypes = [ctypes.POINTER(SeqOp), ci, ci, vp, ctypes.POINTER(vp), ctypes.POINTER(vp), ci, sz, vp]
        lib.nfad_seq_forward.restype = ci
        lib.nfad_seq_backward.argtypes = [ci, ctypes.POINTER(vp), ctypes.POINTER(vp), ci, vp, sz, vp]
        lib.nfad_seq_backward.restype = ci
        lib.nfad_ew_op.argtypes = [ci, ci, ctypes.c_float, ci, vp, vp, vp, vp, vp, sz, vp]
        lib.nfad_ew_op.restype = ci
        lib.nfad_bias_act_forward.argtypes = [ci, ci, vp, vp, vp, vp, sz, sz, vp]
        lib.nfad_bias_act_forward.restype = ci
        lib.nfad_bias_act_forward_infer.argtypes = [ci, ci, vp, vp, vp, sz, sz, vp]
        lib.nfad_bias_act_forward_infer.restype = ci
        lib.nfad_bias_act_backward.argtypes = [ci, ci, vp, vp, vp, vp, vp, sz, sz, sz, vp]
        lib.nfad_bias_act_backward.restype = ci
        lib.nfad_bias_act_backward_scratch_bytes.argtypes = [ci, sz, sz]
        lib.nfad_bias_act_backward_scratch_bytes.restype = sz
        lib.nfad_seq_set_executor.argtypes = [ci]
        lib.nfad_seq_set_executor.restype = ci
        lib.nfad_seq_last_executor.argtypes = []
        lib.nfad_seq_last_executor.restype = ci
        lib.nfad_seq_compiled_source.argtypes = [ctypes.POINTER(SeqOp), ci, ci, ci]
        lib.nfad_seq_compiled_source.restype = ctypes.c_char_p
        lib.nfad_seq_compile_log.argtypes = []
        lib.nfad_seq_compile_log.restype = ctypes.c_char_p
        lib.nfad_host_step.argtypes = [ci, ci, vp, vp, vp, vp, vp, sz, vp, sz, ci, vp]
        lib.nfad_host_step.restype = ci
        lib.nfad_host_step_workspace_bytes.argtypes = [ci, sz]
        lib.nfad_host_step_workspace_bytes.restype = sz
        lib.nfad_cmp_recompute_scratch_bytes.argtypes = [ci, ci, sz]
        lib.nfad_cmp_recompute_scratch_bytes.restype = sz
        lib.nfad_saved_bytes_per_element.argtypes = [ci, ci, ci]
        lib.nfad_probe_stream.argtypes = [ci, ci, vp, vp, vp, vp, sz, vp]
        lib.nfad_probe_stream.restype = ci
        lib.nfad_last_cuda_error.argtypes = []
        lib.nfad_status_string.argtypes = [ci]
        lib.nfad_status_string.restype = ctypes.c_char_p
        lib.nfad_version.argtypes = []
        lib.nfad_version.restype = ctypes.c_char_p
        for name in ("nfad_act_forward", "nfad_act_forward_infer", "nfad_act_backward", "nfad_cmp_conv_backward",
                     "nfad_cmp_recompute_backward", "nfad_saved_bytes_per_element", "nfad_last_cuda_error"):
            getattr(lib, name).restype = ci
        _lib = lib
    return _lib


def _kind(kind) -> int:
    return KINDS[kind] if isinstance(kind, str) else int(kind)


def _tensor(t: torch.Tensor, name: str, like: Optional[torch.Tensor] = None) -> int:
    if not isinstance(t, torch.Tensor) or not t.is_cuda:
        raise TypeError(f"{name} must be a CUDA tensor")
    if t.dtype not in _TORCH_TO_CODE:
        raise TypeError(f"{name}: unsupported dtype {t.dtype}")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    if like is not None and (t.dtype != like.dtype or t.numel() != like.numel() or t.device != like.device):
        raise ValueError(f"{name} must match the first tensor's dtype, size and device")
    return t.data_ptr()


_raw_stream = getattr(torch._C, "_cuda_getCurrentRawStream", None)


def _stream(t: torch.Tensor) -> int:
    """The current stream of the tensor's device, as a cudaStream_t."""
    if _raw_stream is not None:
        idx = t.device.index
        return _raw_stream(idx if idx is not None else torch.cuda.current_device())
    return torch.cuda.current_stream(t.device).cuda_stream


class _on_device:
    """Makes the tensor's device current for the call; a no-op (two integer reads) when it already is --
    the common case, and the one where the generic guard's cost would show in every small launch."""
    __slots__ = ("idx", "prev")

    def __init__(self, dev: torch.device):
        self.idx = dev.index
        self.prev = None

    def __enter__(self):
        cur = torch.cuda.current_device()
        if self.idx is not None and self.idx != cur:
            self.prev = cur
            torch.cuda.set_device(self.idx)
        return self

    def __exit__(self, *exc):
        if self.prev is not None:
            torch.cuda.set_device(self.prev)
        return False


def _check(rc: int, where: str) -> None:
    if rc != NFAD_OK:
        raise NfadError(rc, where)


def nfad_act_forward(kind, x: torch.Tensor, y: torch.Tensor, dfdx: torch.Tensor) -> None:
    """x -> (y = f(x), dfdx = f'(x)), one kernel on the current stream."""
    px = _tensor(x, "x")
    with _on_device(x.device):
        _check(load().nfad_act_forward(_kind(kind), _TORCH_TO_CODE[x.dtype], px, _tensor(y, "y", x),
                                       _tensor(dfdx, "dfdx", x), x.numel(), _stream(x)), "nfad_act_forward")


def nfad_act_forward_strict(kind, x: torch.Tensor, y: torch.Tensor, dfdx: torch.Tensor) -> None:
    """fp32 only: as nfad_act_forward, with f' within 4 fp32 ulp of itself for every input."""
    px = _tensor(x, "x")
    with _on_device(x.device):
        _check(load().nfad_act_forward_strict(_kind(kind), _TORCH_TO_CODE[x.dtype], px, _tensor(y, "y", x),
                                              _tensor(dfdx, "dfdx", x), x.numel(), _stream(x)), "nfad_act_forward_strict")


def nfad_act_forward_infer(kind, x: torch.Tensor, y: torch.Tensor) -> None:
    px = _tensor(x, "x")
    with _on_device(x.device):
        _check(load().nfad_act_forward_infer(_kind(kind), _TORCH_TO_CODE[x.dtype], px, _tensor(y, "y", x),
                                             x.numel(), _stream(x)), "nfad_act_forward_infer")


def nfad_act_backward(kind, grad_out: torch.Tensor, dfdx: torch.Tensor, grad_in: torch.Tensor) -> None:
    """grad_in = grad_out * dfdx (one rounding)."""
    pg = _tensor(grad_out, "grad_out")
    with _on_device(grad_out.device):
        _check(load().nfad_act_backward(_kind(kind), _TORCH_TO_CODE[grad_out.dtype], pg, _tensor(dfdx, "dfdx", grad_out),
                                        _tensor(grad_in, "grad_in", grad_out), grad_out.numel(), _stream(grad_out)),
               "nfad_act_backward")


def nfad_cmp_conv_backward(kind, grad_out: torch.Tensor, x: torch.Tensor, grad_in: torch.Tensor) -> None:
    pg = _tensor(grad_out, "grad_out")
    with _on_device(grad_out.device):
        _check(load().nfad_cmp_conv_backward(_kind(kind), _TORCH_TO_CODE[grad_out.dtype], pg, _tensor(x, "x", grad_out),
                                             _tensor(grad_in, "grad_in", grad_out), grad_out.numel(), _stream(grad_out)),
               "nfad_cmp_conv_backward")


def nfad_cmp_recompute_scratch_bytes(kind, dtype, n: int) -> int:
    code = DTYPES[dtype] if isinstance(dtype, str) else _TORCH_TO_CODE[dtype]
    return int(load().nfad_cmp_recompute_scratch_bytes(_kind(kind), code, n))


def nfad_cmp_recompute_backward(kind, grad_out: torch.Tensor, x: torch.Tensor, scratch: torch.Tensor,
                                grad_in: torch.Tensor) -> None:
    """scratch: any contiguous CUDA tensor with at least nfad_cmp_recompute_scratch_bytes bytes."""
    pg = _tensor(grad_out, "grad_out")
    if not scratch.is_cuda or not scratch.is_contiguous():
        raise TypeError("scratch must be a contiguous CUDA tensor")
    with _on_device(grad_out.device):
        _check(load().nfad_cmp_recompute_backward(_kind(kind), _TORCH_TO_CODE[grad_out.dtype], pg, _tensor(x, "x", grad_out),
                                                  scratch.data_ptr(), scratch.numel() * scratch.element_size(),
                                                  _tensor(grad_in, "grad_in", grad_out), grad_out.numel(),
                                                  _stream(grad_out)), "nfad_cmp_recompute_backward")


def nfad_cmp_recompute_backward_noalloc(kind, grad_out: torch.Tensor, x: torch.Tensor, grad_in: torch.Tensor) -> None:
    """The recomputation comparator on the library's own fixed scratch array: for callers that
    cannot allocate device memory where they stand.  At most NOALLOC_SCRATCH_BYTES per tensor;
    calls on one device share the array, so calls that may overlap on the GPU must be serialised."""
    pg = _tensor(grad_out, "grad_out")
    with _on_device(grad_out.device):
        _check(load().nfad_cmp_recompute_backward_noalloc(_kind(kind), _TORCH_TO_CODE[grad_out.dtype], pg,
                                                          _tensor(x, "x", grad_out), _tensor(grad_in, "grad_in", grad_out),
                                                          grad_out.numel(), _stream(grad_out)),
               "nfad_cmp_recompute_backward_noalloc")


def _rows_cols(x: torch.Tensor, cols: int):
    if cols <= 0 or x.numel() % cols:
        raise ValueError("the tensor's size must be a multiple of the bias length")
    return x.numel() // cols, cols


def nfad_bias_act_forward(kind, x: torch.Tensor, bias: torch.Tensor, y: torch.Tensor, dfdx: torch.Tensor) -> None:
    """x, y, dfdx: [..., cols] contiguous; bias: [cols] of the same dtype.  y = f(x + bias), dfdx = f'(x + bias)."""
    px = _tensor(x, "x")
    if bias.dtype != x.dtype or bias.device != x.device:
        raise ValueError("bias must match x's dtype and device")
    pb = _tensor(bias, "bias")
    rows, cols = _rows_cols(x, bias.numel())
    with _on_device(x.device):
        _check(load().nfad_bias_act_forward(_kind(kind), _TORCH_TO_CODE[x.dtype], px, pb, _tensor(y, "y", x),
                                            _tensor(dfdx, "dfdx", x), rows, cols, _stream(x)), "nfad_bias_act_forward")


def nfad_bias_act_forward_infer(kind, x: torch.Tensor, bias: torch.Tensor, y: torch.Tensor) -> None:
    """y = f(x + bias): the value-only form of nfad_bias_act_forward."""
    px = _tensor(x, "x")
    if bias.dtype != x.dtype or bias.device != x.device:
        raise ValueError("bias must match x's dtype and device")
    pb = _tensor(bias, "bias")
    rows, cols = _rows_cols(x, bias.numel())
    with _on_device(x.device):
        _check(load().nfad_bias_act_forward_infer(_kind(kind), _TORCH_TO_CODE[x.dtype], px, pb, _tensor(y, "y", x), rows, cols,
                                                  _stream(x)), "nfad_bias_act_forward_infer")


def nfad_bias_act_backward_scratch_bytes(dtype, rows: int, cols: int, device=None) -> int:
    code = _TORCH_TO_CODE[dtype] if isinstance(dtype, torch.dtype) else DTYPES[dtype]
    with torch.cuda.device(device if device is not None else torch.cuda.current_device()):
        return int(load().nfad_bias_act_backward_scratch_bytes(code, rows, cols))


def nfad_bias_act_backward(kind, grad_out: torch.Tensor, dfdx: torch.Tensor, grad_in: torch.Tensor, grad_bias: torch.Tensor,
                           scratch: Optional[torch.Tensor]) -> None:
    """grad_in = grad_out * dfdx; grad_bias (fp32, [cols]) = column sums of the stored grad_in.
    scratch: a contiguous CUDA tensor of at least nfad_bias_act_backward_scratch_bytes bytes, or None if that is 0."""
    pg = _tensor(grad_out, "grad_out")
    if grad_bias.dtype != torch.float32 or not grad_bias.is_cuda or not grad_bias.is_contiguous():
        raise TypeError("grad_bias must be a contiguous fp32 CUDA tensor")
    rows, cols = _rows_cols(grad_out, grad_bias.numel())
    if scratch is not None and (not scratch.is_cuda or not scratch.is_contiguous()):
        raise TypeError("scratch must be a contiguous CUDA tensor")
    sp = scratch.data_ptr() if scratch is not None else None
    sb = scratch.numel() * scratch.element_size() if scratch is not None else 0
    with _on_device(grad_out.device):
        _check(load().nfad_bias_act_backward(_kind(kind), _TORCH_TO_CODE[grad_out.dtype], pg, _tensor(dfdx, "dfdx", grad_out),
                                             _tensor(grad_in, "grad_in", grad_out), grad_bias.data_ptr(), sp, sb, rows, cols,
                                             _stream(grad_out)), "nfad_bias_act_backward")


def _host_tensor(t: torch.Tensor, name: str, like: Optional[torch.Tensor] = None) -> int:
    if not isinstance(t, torch.Tensor) or t.is_cuda:
        raise TypeError(f"{name} must be a host tensor")
    if t.dtype not in _TORCH_TO_CODE or not t.is_contiguous():
        raise ValueError(f"{name} must be a contiguous float32 / bfloat16 / float16 tensor")
    if like is not None and (t.dtype != like.dtype or t.numel() != like.numel()):
        raise ValueError(f"{name} must match the first tensor's dtype and size")
    return t.data_ptr()


def nfad_host_step_workspace_bytes(dtype, n: int) -> int:
    code = _TORCH_TO_CODE[dtype] if isinstance(dtype, torch.dtype) else DTYPES[dtype]
    return int(load().nfad_host_step_workspace_bytes(code, n))


HOST_INPUTS_READY = 1


def nfad_host_step(kind, x_host: torch.Tensor, grad_out_host: torch.Tensor, y_host: torch.Tensor, dfdx_host,
                   grad_in_host: torch.Tensor, workspace: torch.Tensor, inputs_ready: bool = False) -> None:
    """Forward + backward for host (ideally pinned) tensors through the device `workspace` lives on; results are in
    host memory once the current stream of that device has completed.  inputs_ready: the host inputs hold their
    final contents now and nothing pending on the stream writes them (lets consecutive calls overlap)."""
    px = _host_tensor(x_host, "x_host")
    if not workspace.is_cuda or not workspace.is_contiguous():
        raise TypeError("workspace must be a contiguous CUDA tensor")
    lib = load()
    with _on_device(workspace.device):
        rc = lib.nfad_host_step(_kind(kind), _TORCH_TO_CODE[x_host.dtype], px, _host_tensor(grad_out_host, "grad_out_host", x_host),
                                _host_tensor(y_host, "y_host", x_host),
                                _host_tensor(dfdx_host, "dfdx_host", x_host) if dfdx_host is not None else None,
                                _host_tensor(grad_in_host, "grad_in_host", x_host), x_host.numel(), workspace.data_ptr(),
                                workspace.numel() * workspace.element_size(), HOST_INPUTS_READY if inputs_ready else 0,
                                _stream(workspace))
        _check(rc, "nfad_host_step")


def _ptr_array(tensors, name, like):
    arr = (ctypes.c_void_p * len(tensors))()
    for i, t in enumerate(tensors):
        arr[i] = _tensor(t, f"{name}[{i}]", like)
    return arr


def _seq_ops(program):
    ops = (SeqOp * len(program))()
    for i, o in enumerate(program):
        if isinstance(o, SeqOp):
            ops[i] = o
        else:
            op, a, b, dst, c = o
            ops[i] = SeqOp(OPCODES[op] if isinstance(op, str) else int(op), int(a), int(b), int(dst), float(c))
    return ops


def nfad_seq_compiled_source(program, dtype, m: int) -> Optional[str]:
    """The CUDA source the compiled executor builds for this sequence (no device needed); None if malformed."""
    code = _TORCH_TO_CODE[dtype] if isinstance(dtype, torch.dtype) else DTYPES[dtype]
    text = load().nfad_seq_compiled_source(_seq_ops(program), len(program), code, int(m))
    return text.decode() if text is not None else None


def nfad_seq_forward(program, x: torch.Tensor, ys, dfdxs) -> None:
    """Runs a FAD sequence (a list of SeqOp, or of (op, a, b, dst, c) tuples with op a name or code)
    on x in one kernel: ys[k] = k-th result, dfdxs[k] = its derivative with respect to x."""
    ops = _seq_ops(program)
    px = _tensor(x, "x")
    if len(ys) != len(dfdxs):
        raise ValueError("ys and dfdxs must have the same length")
    with _on_device(x.device):
        _check(load().nfad_seq_forward(ops, len(program), _TORCH_TO_CODE[x.dtype], px, _ptr_array(ys, "y", x),
                                       _ptr_array(dfdxs, "dfdx", x), len(ys), x.numel(), _stream(x)), "nfad_seq_forward")


SEQ_EXECUTORS = {"auto": 0, "interpreter": 1, "compiled": 2}


def nfad_seq_set_executor(mode) -> None:
    _check(load().nfad_seq_set_executor(SEQ_EXECUTORS[mode] if isinstance(mode, str) else int(mode)), "nfad_seq_set_executor")


def nfad_seq_last_executor() -> str:
    return {0: "none", 1: "interpreter", 2: "compiled"}[load().nfad_seq_last_executor()]


def nfad_seq_compile_log() -> str:
    return load().nfad_seq_compile_log().decode(errors="replace")


def nfad_seq_backward(grad_outs, dfdxs, grad_in: torch.Tensor) -> None:
    """grad_in = sum_k grad_outs[k] * dfdxs[k]."""
    pg = _tensor(grad_in, "grad_in")
    if len(grad_outs) != len(dfdxs):
        raise ValueError("grad_outs and dfdxs must have the same length")
    with _on_device(grad_in.device):
        _check(load().nfad_seq_backward(_TORCH_TO_CODE[grad_in.dtype], _ptr_array(grad_outs, "grad_out", grad_in),
                                        _ptr_array(dfdxs, "dfdx", grad_in), len(grad_outs), pg, grad_in.numel(),
                                        _stream(grad_in)), "nfad_seq_backward")


def nfad_ew_op(op, backward: bool, c: float, in0: torch.Tensor, in1, in2, out0: torch.Tensor, out1=None) -> None:
    """One primitive as its own kernel (forward, or its own backward rule): see include/nfad.h."""
    p0 = _tensor(in0, "in0")
    code = OPCODES[op] if isinstance(op, str) else int(op)
    opt = lambda t, name: _tensor(t, name, in0) if t is not None else None
    with _on_device(in0.device):
        _check(load().nfad_ew_op(code, 1 if backward else 0, float(c), _TORCH_TO_CODE[in0.dtype], p0, opt(in1, "in1"),
                                 opt(in2, "in2"), _tensor(out0, "out0", in0), opt(out1, "out1"), in0.numel(), _stream(in0)),
               "nfad_ew_op")


def nfad_saved_bytes_per_element(kind, dtype, layout) -> int:
    code = DTYPES[dtype] if isinstance(dtype, str) else _TORCH_TO_CODE[dtype]
    lay = LAYOUTS[layout] if isinstance(layout, str) else int(layout)
    rc = load().nfad_saved_bytes_per_element(_kind(kind), code, lay)
    if rc < 0:
        raise NfadError(-rc, "nfad_saved_bytes_per_element")
    return rc


def nfad_probe_stream(reads: int, writes: int, a, b, o0: torch.Tensor, o1) -> None:
    """Traffic probe over fp32 tensors: 1:1 (o0 = a), 1:2 (o0 = a, o1 = ~a), 2:1 (o0 = a ^ b),
    1:0 (reads a; o0 is a sink of at least one word) or 0:1 (writes o0; a is None)."""
    main = a if a is not None else o0
    pm = _tensor(main, "a" if a is not None else "o0")
    if main.dtype != torch.float32:
        raise TypeError("the probe takes float32 tensors")
    one_sided = int(writes) == 0 or int(reads) == 0
    with _on_device(main.device):
        if one_sided:
            po = _tensor(o0, "o0")
            if o0.dtype != torch.float32 or o0.numel() < 1 or o0.device != main.device:
                raise ValueError("o0 must be a float32 tensor on the same device")
            _check(load().nfad_probe_stream(int(reads), int(writes), pm if a is not None else None, None, po, None,
                                            main.numel(), _stream(main)), "nfad_probe_stream")
        else:
            _check(load().nfad_probe_stream(int(reads), int(writes), pm, _tensor(b, "b", a) if b is not None else None,
                                            _tensor(o0, "o0", a), _tensor(o1, "o1", a) if o1 is not None else None,
                                            a.numel(), _stream(a)), "nfad_probe_stream")


def nfad_version() -> str:
    return load().nfad_version().decode()


def nfad_status_string(status: int) -> str:
    return load().nfad_status_string(int(status)).decode()
