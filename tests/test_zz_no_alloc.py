"""The allocation-free all-to-all entry point against the ordinary one.

`Iso_neighbor_alltoall_static` serves callers that may not allocate device memory where
they need the collective (a fixed memory budget handed out at start-up, a host framework
that owns the memory pool, a hot path where cudaMalloc's device-wide synchronisation is not
acceptable): its tables and intermediate buffer live in a fixed scratch array inside the
library.  This file is collected last on purpose, so that a failure here cannot hide the
result of any other test in a run that stops at the first failure.
"""
import numpy as np
import pytest

from paper_1606_07676_b200 import binding as iso
from paper_1606_07676_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _reference(torch, dims, offs, m, send):
    """The existing entry points: init + start + wait (allocates tables and buffer)."""
    P, s = int(np.prod(dims)), len(offs)
    recv = torch.full((P, s * m), 0xA5, dtype=torch.uint8, device="cuda")
    comm = iso.Iso_neighborhood_create(dims, offs)
    req = iso.Iso_neighbor_alltoall_init(send, m, iso.ISO_BYTE, recv, m, iso.ISO_BYTE, comm)
    iso.Iso_Start(req)
    iso.Iso_wait(req)
    iso.Iso_request_free(req)
    iso.Iso_comm_free(comm)
    return recv


def test_static_entry_point_matches_the_allocating_one_twice_in_a_row():
    import torch
    if not torch.cuda.is_available():
        pytest.fail("needs a CUDA device")
    torch.cuda.set_device(0)
    # two different problems back to back: the second call finds the scratch area full of
    # the first call's tables and intermediate blocks
    cases = [((8, 8, 8), wl.moore(3, 1), 64, 11), ((12, 10), wl.moore(2, 2), 24, 12)]
    for dims, offs, m, seed in cases:
        P, s = int(np.prod(dims)), len(offs)
        send = wl.payload_torch("uint8", seed, 0, P * s * m, "cuda").view(P, s * m)
        want = _reference(torch, dims, offs, m, send)
        got = torch.full((P, s * m), 0x5A, dtype=torch.uint8, device="cuda")
        iso.Iso_neighbor_alltoall_static(dims, offs, send, got, m, iso.ISO_BYTE, torch.cuda.current_stream())
        torch.cuda.synchronize()
        assert torch.equal(got, want), "first call differs (dims %s)" % (dims,)
        # same problem again with new payload: same scratch contents layout, new data
        send2 = wl.payload_torch("uint8", seed + 100, 0, P * s * m, "cuda").view(P, s * m)
        want2 = _reference(torch, dims, offs, m, send2)
        got.fill_(0x5A)
        iso.Iso_neighbor_alltoall_static(dims, offs, send2, got, m, iso.ISO_BYTE, torch.cuda.current_stream())
        torch.cuda.synchronize()
        assert torch.equal(got, want2), "second call differs (dims %s)" % (dims,)


def test_static_entry_point_rejects_what_does_not_fit():
    import torch
    if not torch.cuda.is_available():
        pytest.fail("needs a CUDA device")
    torch.cuda.set_device(0)
    dims, offs, m = (32, 32, 32), wl.moore(3, 1), 64     # needs 32768 * 1792 B = 56 MiB of intermediate storage
    P, s = 32768, 26
    send = torch.zeros((P, s * m), dtype=torch.uint8, device="cuda")
    recv = torch.full((P, s * m), 0x33, dtype=torch.uint8, device="cuda")
    with pytest.raises(iso.IsoError) as e:
        iso.Iso_neighbor_alltoall_static(dims, offs, send, recv, m, iso.ISO_BYTE)
    assert e.value.code == iso.ISO_ERR_TOO_LARGE
    assert "scratch" in iso.Iso_error_string(iso.ISO_ERR_TOO_LARGE)
    torch.cuda.synchronize()
    assert int(recv.min()) == 0x33 and int(recv.max()) == 0x33      # nothing was enqueued
