"""The allocation-free all-to-all entry point against the CPU oracle and the ordinary path.

`Iso_neighbor_alltoall_static` serves callers that may not allocate device memory where
they need the collective (a fixed memory budget handed out at start-up, a host framework
that owns the memory pool, a hot path where cudaMalloc's device-wide synchronisation is not
acceptable): its tables and intermediate buffer live in a fixed scratch array inside the
library.  This file is collected last on purpose, so that a failure here cannot hide the
result of any other test in a run that stops at the first failure.
"""
import numpy as np
import pytest

import oracle
from paper_1606_07676_b200 import binding as iso
from paper_1606_07676_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _allocating(torch, dims, offs, m, send):
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


def _cases():
    odd = np.array([[0, 0, 0], [1, 0, -1], [1, 0, -1], [-5, 3, 2], [0, 1, 0], [2, 2, 2]], np.int32)  # zero vector, a repeat, |c| >= p
    return [((8, 8, 8), wl.moore(3, 1), 64, 11), ((12, 10), wl.moore(2, 2), 24, 12),
            ((7, 5), wl.moore(2, 1), 1, 13), ((6, 4, 3), wl.moore(3, 1), 2, 14), ((9, 11), wl.moore(2, 2), 20, 15),
            ((3, 1, 2), odd, 16, 16), ((2, 2), wl.moore(2, 1), 48, 17), ((5, 4, 3, 2), wl.moore(4, 1), 8, 18)]


def test_static_entry_point_matches_the_oracle_twice_in_a_row():
    import torch
    if not torch.cuda.is_available():
        pytest.fail("needs a CUDA device")
    torch.cuda.set_device(0)
    # different problems back to back: every call finds the scratch area full of the previous
    # call's tables and intermediate blocks
    for dims, offs, m, seed in _cases():
        P, s = int(np.prod(dims)), len(offs)
        got = torch.full((P, s * m), 0x5A, dtype=torch.uint8, device="cuda")
        for call in range(2):       # the same problem twice, with new contents the second time
            send_h = wl.payload_np("uint8", seed + 100 * call, 0, 0, P * s * m).reshape(P, s * m).copy()
            send = torch.from_numpy(send_h).cuda()
            want = oracle.alltoall(dims, offs, m, send_h)
            got.fill_(0x5A)
            iso.Iso_neighbor_alltoall_static(dims, offs, send, got, m, iso.ISO_BYTE, torch.cuda.current_stream())
            torch.cuda.synchronize()
            assert np.array_equal(got.cpu().numpy(), want), "call %d differs from the oracle (dims %s, m %d)" % (call, dims, m)
            # and the ordinary entry points give the same bytes
            assert torch.equal(got, _allocating(torch, dims, offs, m, send)), (dims, m, call)


def test_static_entry_point_allocates_no_device_memory():
    """What the entry point exists for: once the device has loaded the library's kernels
    (first call), a call leaves the amount of free device memory exactly as it found it."""
    import torch
    if not torch.cuda.is_available():
        pytest.fail("needs a CUDA device")
    torch.cuda.set_device(0)
    dims, offs, m = (8, 8, 8), wl.moore(3, 1), 64
    P, s = 512, 26
    send = wl.payload_torch("uint8", 3, 0, P * s * m, "cuda").view(P, s * m)
    recv = torch.empty((P, s * m), dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream()
    iso.Iso_neighbor_alltoall_static(dims, offs, send, recv, m, iso.ISO_BYTE, stream)      # warm-up: kernels get loaded
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    for _ in range(3):
        iso.Iso_neighbor_alltoall_static(dims, offs, send, recv, m, iso.ISO_BYTE, stream)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before


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
