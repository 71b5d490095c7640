"""Test-only helpers: run an exported schedule on host memory with numpy, and build the
expected result of a workload with the CPU oracle."""
import numpy as np

import oracle
from paper_1606_07676_b200 import binding as iso
from paper_1606_07676_b200 import workloads as wl

POISON = 0xA5


def simulate(parts, dims, stats, send, periodic=None):
    """Executes `parts` (Iso_request_get_parts) for all processes.

    Inside a phase every read sees the buffers as they were when the phase began, so an
    ordering hazard inside a phase shows up as a wrong result.  Returns the receive buffers
    as uint8 [P, recv_stride]; bytes never written keep the poison value.
    """
    dims = tuple(int(x) for x in dims)
    d = len(dims)
    P = int(np.prod(dims))
    periodic = [1] * d if periodic is None else list(periodic)
    bufs = {
        iso.ISO_BUF_SEND: np.ascontiguousarray(send).view(np.uint8).reshape(P, stats["send_stride"]) if stats["send_stride"] else np.zeros((P, 0), np.uint8),
        iso.ISO_BUF_RECV: np.full((P, stats["recv_stride"]), POISON, np.uint8),
        iso.ISO_BUF_INTER: np.full((P, stats["inter_stride"]), POISON, np.uint8),
    }
    coords = np.stack(np.unravel_index(np.arange(P), dims), axis=1) if P else np.zeros((0, d), np.int64)
    phases = sorted({p["phase"] for p in parts})
    last = -1
    for ph in phases:
        assert ph > last
        last = ph
        snap = {k: v.copy() for k, v in bufs.items()}
        for p in parts:
            if p["phase"] != ph:
                continue
            assert p["dst_buf"] != iso.ISO_BUF_SEND
            src = coords.copy()
            valid = np.ones(P, bool)
            for j in range(d):
                c = p["shift"][j]
                if periodic[j]:
                    src[:, j] = (src[:, j] - c) % dims[j]
                else:
                    y = coords[:, j] - p["check"][j]
                    valid &= (y >= 0) & (y < dims[j])
                    src[:, j] = src[:, j] - c
            src[~valid] = 0
            sr = np.ravel_multi_index(tuple(src.T), dims) if P else np.zeros(0, np.int64)
            so, do, n = p["src_off"], p["dst_off"], p["len"]
            data = snap[p["src_buf"]][sr, so:so + n]
            dst = bufs[p["dst_buf"]]
            dst[valid, do:do + n] = data[valid]
    return bufs[iso.ISO_BUF_RECV]


layout = wl.layout
send_buffer_np = wl.send_buffer_np


def oracle_result(w, send, r0=0, r1=None, fill=POISON, periodic=None):
    """Expected receive buffers of ranks [r0, r1) from the CPU oracle; with non-periodic
    dimensions, slots that are not delivered hold `fill`."""
    lens, sd, rd, ss, rs = layout(w)
    if w.collective == "alltoall":
        return oracle.alltoall(w.dims, w.offsets, w.block_bytes, send, r0, r1, periodic=periodic, fill=fill)
    if w.collective == "allgather":
        return oracle.allgather(w.dims, w.offsets, w.block_bytes, send, r0, r1, periodic=periodic, fill=fill)
    return oracle.alltoallv(w.dims, w.offsets, lens, sd, rd, ss, rs, send, r0, r1, fill=fill, periodic=periodic)


def make_request(w, sendbuf=None, recvbuf=None, periodic=None):
    """Creates (comm, request) for workload `w` through the C-ABI binding."""
    comm = iso.Iso_neighborhood_create(w.dims, w.offsets)
    if periodic is not None:
        iso.Iso_comm_set_periodic(comm, periodic)
    if w.collective == "alltoall":
        req = iso.Iso_neighbor_alltoall_init(sendbuf, w.block_bytes, iso.ISO_BYTE, recvbuf, w.block_bytes,
                                             iso.ISO_BYTE, comm)
    elif w.collective == "allgather":
        req = iso.Iso_neighbor_allgather_init(sendbuf, w.block_bytes, iso.ISO_BYTE, recvbuf, w.block_bytes,
                                              iso.ISO_BYTE, comm)
    else:
        lens, sd, rd, _, _ = layout(w)
        req = iso.Iso_neighbor_alltoallv_init(sendbuf, lens, sd, iso.ISO_BYTE, recvbuf, lens, rd, iso.ISO_BYTE, comm)
    return comm, req
