"""Host-side checks of the C-ABI library that need no GPU: it loads, exports exactly
the symbols the header declares, and validates arguments before touching CUDA."""
import ctypes
import os
import re

import pytest

from paper_2209_10778_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build_library()
    return binding.load()


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "nfad.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"NFAD_API\s+[\w\s\*]+?\b(nfad_\w+)\s*\(", text)))


def test_header_and_binding_agree_on_the_exports():
    assert _declared_symbols() == sorted(binding.EXPORTS)


def test_library_exports_every_declared_symbol(lib):
    for name in _declared_symbols():
        assert hasattr(lib, name), name


def test_no_other_nfad_symbols_are_exported(lib):
    import subprocess
    out = subprocess.run(["nm", "-D", "--defined-only", binding.LIB_PATH], capture_output=True, text=True).stdout
    exported = sorted(l.split()[-1] for l in out.splitlines() if " T " in l)
    assert exported == _declared_symbols()


def test_version_and_status_strings(lib):
    assert re.fullmatch(r"\d+\.\d+\.\d+", binding.nfad_version())
    assert binding.nfad_status_string(0) == "ok"
    assert len({binding.nfad_status_string(i) for i in range(9)}) == 9


def test_validation_needs_no_device(lib):
    fake = ctypes.c_void_p(0x1000)
    assert lib.nfad_act_forward(4, 0, fake, fake, fake, 8, None) == 1        # kind
    assert lib.nfad_act_forward(-1, 0, fake, fake, fake, 8, None) == 1
    assert lib.nfad_act_forward(0, 3, fake, fake, fake, 8, None) == 2        # dtype
    assert lib.nfad_act_forward(0, 0, None, fake, fake, 8, None) == 3        # null
    assert lib.nfad_act_backward(0, 0, fake, None, fake, 8, None) == 3
    assert lib.nfad_act_forward(0, 0, fake, ctypes.c_void_p(0x2000), ctypes.c_void_p(0x2010), 8, None) == 4   # y, dfdx overlap
    assert lib.nfad_act_forward_infer(0, 0, fake, ctypes.c_void_p(0x1004), 8, None) == 4                      # partial overlap
    assert lib.nfad_act_forward(0, 0, ctypes.c_void_p(0x1002), fake, ctypes.c_void_p(0x3000), 8, None) == 6   # alignment
    assert lib.nfad_act_forward(0, 1, ctypes.c_void_p(0x1001), fake, ctypes.c_void_p(0x3000), 8, None) == 6
    # n == 0 is valid with any pointers and launches nothing
    assert lib.nfad_act_forward(0, 0, None, None, None, 0, None) == 0
    assert lib.nfad_act_backward(3, 2, None, None, None, 0, None) == 0
    assert lib.nfad_cmp_recompute_backward(0, 0, fake, fake, fake, 0, fake, 8, None) == 7                    # scratch too small


def test_saved_bytes_and_scratch_size(lib):
    assert lib.nfad_saved_bytes_per_element(2, 1, 0) == 2
    assert lib.nfad_saved_bytes_per_element(2, 1, 3) == 4
    assert lib.nfad_saved_bytes_per_element(1, 0, 3) == 16
    assert lib.nfad_saved_bytes_per_element(0, 0, 9) == -8
    assert lib.nfad_saved_bytes_per_element(7, 0, 0) == -1
    assert lib.nfad_cmp_recompute_scratch_bytes(0, 1, 1000) == 2000
    assert lib.nfad_cmp_recompute_scratch_bytes(0, 0, 3) == 16
    assert lib.nfad_cmp_recompute_scratch_bytes(9, 0, 3) == 0


def test_binding_refuses_cpu_tensors():
    import torch
    x = torch.zeros(8)
    with pytest.raises(TypeError):
        binding.nfad_act_forward("swish", x, x.clone(), x.clone())


def test_newer_entry_points_validate_without_a_device(lib):
    fake, other = ctypes.c_void_p(0x10000), ctypes.c_void_p(0x90000)
    # bias-fused pass: shape limits and pointers are checked before any CUDA call
    assert lib.nfad_bias_act_forward(0, 0, fake, other, fake, ctypes.c_void_p(0x50000), 4, 1 << 31, None) == 9
    assert lib.nfad_bias_act_forward(5, 0, fake, other, fake, fake, 4, 8, None) == 1
    assert lib.nfad_bias_act_forward(0, 0, fake, None, ctypes.c_void_p(0x20000), ctypes.c_void_p(0x30000), 4, 8, None) == 3
    assert lib.nfad_bias_act_forward(0, 0, None, None, None, None, 0, 8, None) == 0
    assert lib.nfad_bias_act_backward(0, 4, fake, fake, fake, None, None, 0, 4, 8, None) == 2
    # strict forward is fp32 only
    assert lib.nfad_act_forward_strict(0, 1, fake, other, ctypes.c_void_p(0x50000), 8, None) == 2
    assert lib.nfad_act_forward_strict(0, 0, None, None, None, 0, None) == 0
    # host pipeline
    assert lib.nfad_host_step(0, 0, fake, fake, fake, None, fake, 8, None, 0, 0, None) == 3
    assert lib.nfad_host_step(0, 0, fake, fake, fake, None, fake, 8, fake, 1 << 20, 4, None) == 8
    assert lib.nfad_host_step_workspace_bytes(1, 1 << 24) == 4 * 5 * (8 << 20)
    assert lib.nfad_host_step_workspace_bytes(0, 1000) == 4 * 5 * 2048 * 4
    assert lib.nfad_host_step_workspace_bytes(7, 1000) == 0
    # executors of a run-time sequence
    assert lib.nfad_seq_set_executor(3) == 8 and lib.nfad_seq_set_executor(-1) == 8
    assert lib.nfad_seq_set_executor(1) == 0 and lib.nfad_seq_set_executor(0) == 0
    assert lib.nfad_seq_last_executor() in (0, 1, 2)
    # one-sided probes
    assert lib.nfad_probe_stream(1, 0, ctypes.c_void_p(0x10004), None, other, None, 1024, None) == 6
    assert lib.nfad_probe_stream(0, 1, None, None, None, None, 1024, None) == 3


def test_binding_refuses_wrong_placements():
    import torch
    x = torch.zeros(8)
    with pytest.raises(TypeError):
        binding.nfad_bias_act_forward("swish", x, x.clone(), x.clone(), x.clone())
    with pytest.raises(TypeError):
        binding.nfad_act_forward_strict("swish", x, x.clone(), x.clone())


def test_sequence_programs_are_validated_without_a_device(lib):
    Op = binding.SeqOp
    fake = ctypes.c_void_p(0x10000)
    outs = (ctypes.c_void_p * 1)(0x20000)
    ds = (ctypes.c_void_p * 1)(0x30000)

    def run(ops, m=1, n=0):
        arr = (Op * len(ops))(*[Op(*o) for o in ops])
        return lib.nfad_seq_forward(arr, len(ops), 0, fake, outs, ds, m, n, None)

    ok = [(9, 0, 0, 1, 0.0), (1, 0, 1, 2, 0.0), (12, 2, 0, 0, 0.0)]            # swish: sigmoid, mul, out
    assert run(ok) == 0
    assert run([(99, 0, 0, 1, 0.0), (12, 1, 0, 0, 0.0)]) == 10                  # unknown opcode
    assert run([(9, 3, 0, 1, 0.0), (12, 1, 0, 0, 0.0)]) == 10                   # reads a register never written
    assert run([(9, 0, 0, 0, 0.0), (12, 0, 0, 0, 0.0)]) == 10                   # writes the source register
    assert run([(9, 0, 0, 12, 0.0), (12, 1, 0, 0, 0.0)]) == 10                  # register out of range
    assert run([(9, 0, 0, 1, 0.0)]) == 10                                       # no result produced
    assert run([(9, 0, 0, 1, 0.0), (12, 1, 0, 1, 0.0)]) == 10                   # result slot out of range for m = 1
    assert run(ok, m=5) == 10 and run(ok, m=0) == 10
    assert lib.nfad_seq_forward(None, 3, 0, fake, outs, ds, 1, 0, None) == 3
    assert run(ok * 11) == 10                                                    # more than 32 instructions
