"""The run-time compiler's code generator, without a GPU: the source it emits for a sequence is what the
program says, and it compiles for sm_100a with NVRTC against this library's own headers."""
import os

import pytest

from paper_2209_10778_b200 import binding, build, sequence

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
CSRC = os.path.join(ROOT, "paper_2209_10778_b200", "csrc")


@pytest.fixture(scope="module", autouse=True)
def _lib():
    build.build_library()
    binding.load()


def _programs_covering_every_primitive():
    p = sequence.FadProgram()
    x = p.x()
    p.output(p.mul(x, p.unary("sigmoid", x)))
    p.output(p.add(p.unary("tanh", p.scale(0.25, x)), p.unary("erf", p.add_const(0.5, x))))
    q = sequence.FadProgram()
    x = q.x()
    q.output(q.unary("softplus", q.unary("log1p", q.unary("exp", q.scale(-1.0, q.mul(x, x))))))
    q.output(q.add(q.unary("half_one_plus_tanh", x), q.unary("half_one_plus_erf", x)))
    q.output(x)
    return [p, q]


def test_generated_source_follows_the_program():
    prog = sequence.swish_program()
    src = binding.nfad_seq_compiled_source(prog.ops, "bf16", 1)
    assert "dual_sigmoid(v_src)" in src and "dual_mul(" in src and "yv[0]" in src
    assert "jit_forward<nfad::StoreBF16, 1>" in src
    assert "StoreF32" in binding.nfad_seq_compiled_source(prog.ops, "f32", 1)
    # constants are emitted as exact bit patterns
    p = sequence.FadProgram()
    p.output(p.scale(0.1, p.x()))
    assert "__int_as_float(0x3dcccccd)" in binding.nfad_seq_compiled_source(p.ops, "f16", 1)
    # malformed programs give no source
    assert binding.nfad_seq_compiled_source([("sigmoid", 5, 0, 1, 0.0), ("out", 1, 0, 0, 0.0)], "f32", 1) is None
    assert binding.nfad_seq_compiled_source(prog.ops, "f32", 0) is None


@pytest.mark.parametrize("dtype", ["f32", "bf16", "f16"])
def test_generated_source_compiles_with_nvrtc(dtype):
    nvrtc = pytest.importorskip("cuda.bindings.nvrtc")
    include = os.environ.get("CUDA_HOME", "/usr/local/cuda") + "/include"
    if not os.path.exists(os.path.join(include, "cuda_bf16.h")):
        pytest.skip("CUDA toolkit headers not found")
    for prog in _programs_covering_every_primitive():
        src = binding.nfad_seq_compiled_source(prog.ops, dtype, prog.n_out)
        assert src is not None
        err, handle = nvrtc.nvrtcCreateProgram(src.encode(), b"nfad_seq_compiled.cu", 0, [], [])
        assert err == nvrtc.nvrtcResult.NVRTC_SUCCESS
        opts = [b"--gpu-architecture=sm_100a", b"--std=c++17", b"--fmad=true", f"-I{CSRC}".encode(), f"-I{include}".encode()]
        (err,) = nvrtc.nvrtcCompileProgram(handle, len(opts), opts)
        _, n = nvrtc.nvrtcGetProgramLogSize(handle)
        log = b" " * n
        nvrtc.nvrtcGetProgramLog(handle, log)
        assert err == nvrtc.nvrtcResult.NVRTC_SUCCESS, log.decode(errors="replace")
        _, size = nvrtc.nvrtcGetCUBINSize(handle)
        assert size > 0
