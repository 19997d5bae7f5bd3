"""The traffic probes (a measurement aid): what each read/write mix leaves in memory, and its refusals."""
import numpy as np
import pytest
import torch

from paper_2209_10778_b200 import binding as nfad

pytestmark = pytest.mark.gpu
DEV = "cuda"


def test_probe_mixes_move_the_bits_they_claim():
    n = 4 * 1000 + 4 * 256 * 4 * 3                       # several tiles and a ragged last one, whole packets
    a = torch.randn(n, device=DEV)
    b = torch.randn(n, device=DEV)
    o0, o1 = torch.empty_like(a), torch.empty_like(a)
    nfad.nfad_probe_stream(1, 1, a, None, o0, None)
    assert torch.equal(o0.view(torch.int32), a.view(torch.int32))
    nfad.nfad_probe_stream(1, 2, a, None, o0, o1)
    assert torch.equal(o0.view(torch.int32), a.view(torch.int32))
    assert torch.equal(o1.view(torch.int32), ~a.view(torch.int32))
    nfad.nfad_probe_stream(2, 1, a, b, o0, None)
    assert torch.equal(o0.view(torch.int32), a.view(torch.int32) ^ b.view(torch.int32))
    # write only: packet k holds (k low, k high, 1.0f, 0)
    guard = torch.full((n + 8,), 7.0, device=DEV)
    nfad.nfad_probe_stream(0, 1, None, None, guard[4:4 + n], None)
    torch.cuda.synchronize()
    w = guard.view(torch.int32).cpu().numpy()
    body = w[4:4 + n].reshape(-1, 4)
    assert np.array_equal(body[:, 0], np.arange(n // 4, dtype=np.int32)) and (body[:, 1] == 0).all()
    assert (body[:, 2] == 0x3f800000).all() and (body[:, 3] == 0).all()
    assert (guard[:4] == 7.0).all() and (guard[4 + n:] == 7.0).all()
    # read only: nothing is written (the sink keeps its value unless a checksum matches a fixed constant)
    sink = torch.zeros(4, device=DEV)
    before = a.clone()
    nfad.nfad_probe_stream(1, 0, a, None, sink, None)
    torch.cuda.synchronize()
    assert torch.equal(a, before) and (sink == 0).all()


def test_probe_refusals():
    lib = nfad.load()
    a = torch.zeros(1024 + 4, device=DEV)
    o = torch.zeros(1024 + 4, device=DEV)
    st = torch.cuda.current_stream().cuda_stream
    assert lib.nfad_probe_stream(3, 1, a.data_ptr(), None, o.data_ptr(), None, 1024, st) == 8
    assert lib.nfad_probe_stream(0, 0, None, None, None, None, 1024, st) == 8
    assert lib.nfad_probe_stream(1, 0, a.data_ptr() + 4, None, o.data_ptr(), None, 1024, st) == 6      # not 16-byte aligned
    assert lib.nfad_probe_stream(0, 1, None, None, o.data_ptr(), None, 1022, st) == 6                 # not whole packets
    assert lib.nfad_probe_stream(1, 0, a.data_ptr(), None, None, None, 1024, st) == 3
    assert lib.nfad_probe_stream(1, 0, a.data_ptr(), None, a.data_ptr() + 16, None, 1024, st) == 4    # sink inside the input
    assert lib.nfad_probe_stream(1, 0, a.data_ptr(), None, o.data_ptr(), None, 0, st) == 0
    torch.cuda.synchronize()
