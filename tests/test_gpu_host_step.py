"""nfad_host_step: forward + backward for tensors in host memory through the chunked copy / compute / copy pipeline.
Results must be bit-identical to the device entry points (same kernels), hence within the oracle's gates."""
import numpy as np
import pytest
import torch

import parity
from paper_2209_10778_b200 import binding as nfad
from paper_2209_10778_b200 import workloads as W

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _host_run(kind, dtype, n, ws_bytes=None, want_d=True, pinned=True):
    x = W.normal(n, dtype, 61, 1.5)
    g = W.normal(n, dtype, 62, 1.0)
    mk = (lambda t: t.pin_memory()) if pinned else (lambda t: t)
    hx, hg = mk(x), mk(g)
    hy, hd, hgin = (mk(torch.empty_like(x)) for _ in range(3))
    nbytes = ws_bytes if ws_bytes is not None else nfad.nfad_host_step_workspace_bytes(W.TORCH_DTYPES[dtype], n)
    ws = torch.empty(nbytes, dtype=torch.uint8, device=DEV)
    nfad.nfad_host_step(kind, hx, hg, hy, hd if want_d else None, hgin, ws)
    torch.cuda.current_stream().synchronize()
    return x, g, hy, hd, hgin


@pytest.mark.parametrize("dtype", ["f32", "bf16", "f16"])
def test_host_step_equals_the_device_calls_and_the_oracle(dtype):
    n = 5 * (1 << 20) + 12345                       # several chunks and a ragged last one
    for kind in ("gelu_erf", "mish"):
        x, g, hy, hd, hgin = _host_run(kind, dtype, n)
        xd, gd = x.to(DEV), g.to(DEV)
        y, d, gin = parity.full_check(kind, dtype, xd, gd)          # device calls, checked against the oracle
        for a, b in ((hy, y), (hd, d), (hgin, gin)):
            assert np.array_equal(W.raw_numpy(a), W.raw_numpy(b))


def test_host_step_small_workspace_optional_outputs_and_pageable_memory():
    n = (1 << 18) + 77
    ref = _host_run("swish", "bf16", n)
    # the smallest workspace that holds one 2048-element chunk per slot: many tiny chunks, same bits
    small = _host_run("swish", "bf16", n, ws_bytes=4 * 5 * 2048 * 2)
    assert np.array_equal(W.raw_numpy(ref[2]), W.raw_numpy(small[2])) and np.array_equal(W.raw_numpy(ref[4]), W.raw_numpy(small[4]))
    nod = _host_run("swish", "bf16", n, want_d=False)
    assert np.array_equal(W.raw_numpy(ref[4]), W.raw_numpy(nod[4]))
    pageable = _host_run("swish", "bf16", n, pinned=False)
    assert np.array_equal(W.raw_numpy(ref[2]), W.raw_numpy(pageable[2])) and np.array_equal(W.raw_numpy(ref[4]), W.raw_numpy(pageable[4]))


def test_host_step_two_calls_back_to_back_and_later_stream_work_see_the_results():
    n = 3 * (1 << 20)
    x = W.normal(n, "bf16", 63, 1.0).pin_memory()
    g = W.normal(n, "bf16", 64, 1.0).pin_memory()
    outs = [[torch.empty_like(x).pin_memory() for _ in range(2)] for _ in range(2)]
    ws = torch.empty(nfad.nfad_host_step_workspace_bytes(torch.bfloat16, n), dtype=torch.uint8, device=DEV)
    back = torch.empty(n, dtype=torch.bfloat16, device=DEV)
    for k, kind in enumerate(("gelu_erf", "gelu_tanh")):
        # the same workspace, no sync in between, the second call free to run ahead into slots as they free up
        nfad.nfad_host_step(kind, x, g, outs[k][0], None, outs[k][1], ws, inputs_ready=True)
    back.copy_(outs[1][0], non_blocking=True)                                  # stream-ordered after the second call
    torch.cuda.synchronize()
    for k, kind in enumerate(("gelu_erf", "gelu_tanh")):
        y, d = torch.empty(n, dtype=torch.bfloat16, device=DEV), torch.empty(n, dtype=torch.bfloat16, device=DEV)
        nfad.nfad_act_forward(kind, x.to(DEV), y, d)
        assert torch.equal(y.cpu().view(torch.int16), outs[k][0].view(torch.int16))
    assert torch.equal(back.cpu().view(torch.int16), outs[1][0].view(torch.int16))


def test_host_step_refusals():
    lib = nfad.load()
    x = torch.zeros(4096).pin_memory()
    ws = torch.empty(1 << 20, dtype=torch.uint8, device=DEV)
    st = torch.cuda.current_stream().cuda_stream
    p = x.data_ptr()
    assert lib.nfad_host_step(7, 0, p, p, p, None, p, 4096, ws.data_ptr(), 1 << 20, 0, st) == 1
    assert lib.nfad_host_step(0, 3, p, p, p, None, p, 4096, ws.data_ptr(), 1 << 20, 0, st) == 2
    assert lib.nfad_host_step(0, 0, None, p, p, None, p, 4096, ws.data_ptr(), 1 << 20, 0, st) == 3
    assert lib.nfad_host_step(0, 0, p, p, p, None, p, 4096, None, 0, 0, st) == 3
    assert lib.nfad_host_step(0, 0, p, p, p, None, p, 4096, ws.data_ptr(), 1000, 0, st) == 7
    assert lib.nfad_host_step(0, 0, p, p, p, None, p, 4096, ws.data_ptr() + 4, 1 << 19, 0, st) == 6
    assert lib.nfad_host_step(0, 0, p, p, p, None, p, 0, None, 0, 0, st) == 0
    assert lib.nfad_host_step(0, 0, p, p, p, None, p, 4096, ws.data_ptr(), 1 << 20, 2, st) == 8
    assert nfad.nfad_host_step_workspace_bytes(torch.float32, 0) == 0


def test_host_step_inputs_ready_with_changing_workspaces():
    # consecutive calls that may run ahead (inputs ready) but use different workspaces and chunk sizes: the second
    # must not touch slots the first still uses, and each must give the device calls' bits
    n1, n2 = 3 * (1 << 20) + 5, (1 << 19) + 3
    x1, g1 = W.normal(n1, "bf16", 71, 1.0).pin_memory(), W.normal(n1, "bf16", 72, 1.0).pin_memory()
    x2, g2 = W.normal(n2, "f32", 73, 1.0).pin_memory(), W.normal(n2, "f32", 74, 1.0).pin_memory()
    y1, gi1 = torch.empty_like(x1).pin_memory(), torch.empty_like(x1).pin_memory()
    y2, gi2 = torch.empty_like(x2).pin_memory(), torch.empty_like(x2).pin_memory()
    ws1 = torch.empty(nfad.nfad_host_step_workspace_bytes(torch.bfloat16, n1), dtype=torch.uint8, device=DEV)
    ws2 = torch.empty(4 * 5 * 4096 * 4, dtype=torch.uint8, device=DEV)          # small: many chunks
    nfad.nfad_host_step("mish", x1, g1, y1, None, gi1, ws1, inputs_ready=True)
    nfad.nfad_host_step("swish", x2, g2, y2, None, gi2, ws2, inputs_ready=True)
    nfad.nfad_host_step("gelu_erf", x1, g1, y1, None, gi1, ws1, inputs_ready=True)   # back to the first layout
    torch.cuda.synchronize()
    for kind, x, g, y, gi in (("gelu_erf", x1, g1, y1, gi1), ("swish", x2, g2, y2, gi2)):
        xd, gd = x.to(DEV), g.to(DEV)
        yd, dd, gid = torch.empty_like(xd), torch.empty_like(xd), torch.empty_like(xd)
        nfad.nfad_act_forward(kind, xd, yd, dd)
        nfad.nfad_act_backward(kind, gd, dd, gid)
        assert np.array_equal(W.raw_numpy(y), W.raw_numpy(yd)) and np.array_equal(W.raw_numpy(gi), W.raw_numpy(gid))


def test_host_step_two_streams_sharing_one_workspace_with_different_cuts():
    # two callers on different streams hand the SAME workspace to calls that cut it differently (other dtype and size,
    # stream-ordered inputs): the second call must wait until the first has finished with its slots
    n1, n2 = 6 * (1 << 20) + 77, 2 * (1 << 20) + 9
    x1, g1 = W.normal(n1, "bf16", 81, 1.0).pin_memory(), W.normal(n1, "bf16", 82, 1.0).pin_memory()
    x2, g2 = W.normal(n2, "f32", 83, 1.0).pin_memory(), W.normal(n2, "f32", 84, 1.0).pin_memory()
    y1, gi1 = torch.empty_like(x1).pin_memory(), torch.empty_like(x1).pin_memory()
    y2, gi2 = torch.empty_like(x2).pin_memory(), torch.empty_like(x2).pin_memory()
    ws = torch.empty(nfad.nfad_host_step_workspace_bytes(torch.bfloat16, n1), dtype=torch.uint8, device=DEV)
    sa, sb = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    for _ in range(3):
        with torch.cuda.stream(sa):
            nfad.nfad_host_step("gelu_tanh", x1, g1, y1, None, gi1, ws)
        with torch.cuda.stream(sb):
            nfad.nfad_host_step("mish", x2, g2, y2, None, gi2, ws)
    torch.cuda.synchronize()
    for kind, x, g, y, gi in (("gelu_tanh", x1, g1, y1, gi1), ("mish", x2, g2, y2, gi2)):
        xd, gd = x.to(DEV), g.to(DEV)
        yd, dd, gid = torch.empty_like(xd), torch.empty_like(xd), torch.empty_like(xd)
        nfad.nfad_act_forward(kind, xd, yd, dd)
        nfad.nfad_act_backward(kind, gd, dd, gid)
        torch.cuda.synchronize()
        assert np.array_equal(W.raw_numpy(y), W.raw_numpy(yd)) and np.array_equal(W.raw_numpy(gi), W.raw_numpy(gid))
