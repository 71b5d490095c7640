"""Pins for the CPU oracle: it is checked against things other than itself.

* values worked by hand from the definition (tests/golden/moore_4x4_alltoall.txt),
* the sender-side ("push") statement of the collective, enumerated in pure Python
  with coordinate arithmetic written here,
* special cases that reduce to numpy routines (roll, transpose, tile),
* mutants of the oracle source (a flipped sign, a transposed rank order, a dropped
  index ...) which these same pins must reject.
"""
import itertools
import os
import subprocess

import numpy as np
import pytest

import oracle

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
GOLDEN = os.path.join(ROOT, "tests", "golden")


# --------------------------------------------------------------- helpers written here
def coords_of(r, dims):
    out = []
    for p in reversed(dims):
        out.append(r % p)
        r //= p
    return list(reversed(out))


def rank_of(coords, dims):
    r = 0
    for c, p in zip(coords, dims):
        r = r * p + c
    return r


def push_alltoallv(dims, offsets, lens, sdispls, rdispls, sstride, rstride, send, fill=0):
    """Every process q writes its block i into the receive buffer of q (+) C^i."""
    P = int(np.prod(dims))
    recv = np.full((P, rstride), fill, dtype=np.uint8)
    written = np.zeros((P, rstride), dtype=np.int32)
    send = send.reshape(P, sstride)
    for q in range(P):
        Q = coords_of(q, dims)
        for i, C in enumerate(offsets):
            T = [(a + int(c)) % p for a, c, p in zip(Q, C, dims)]
            t = rank_of(T, dims)
            recv[t, rdispls[i]:rdispls[i] + lens[i]] = send[q, sdispls[i]:sdispls[i] + lens[i]]
            written[t, rdispls[i]:rdispls[i] + lens[i]] += 1
    return recv, written


def moore_list(d, r):
    return [v for v in itertools.product(range(-r, r + 1), repeat=d) if any(v)]


# ------------------------------------------------------------------ the pins, reusable
def pin_golden(lib):
    dims = (4, 4)
    offs = moore_list(2, 1)
    P, s = 16, 8
    send = np.array([[100 * q + i for i in range(s)] for q in range(P)], dtype=np.int32)
    recv = oracle.alltoall(dims, offs, 4, send, lib=lib).view(np.int32).reshape(P, s)
    n = 0
    for line in open(os.path.join(GOLDEN, "moore_4x4_alltoall.txt")):
        if line.startswith("#") or not line.strip():
            continue
        rank, vals = line.split(":")
        assert recv[int(rank)].tolist() == [int(v) for v in vals.split()], "rank " + rank
        n += 1
    assert n == 3


def pin_golden_allgather(lib):
    dims, offs = (4, 4), moore_list(2, 1)
    send = np.array([100 * q for q in range(16)], dtype=np.int32)
    recv = oracle.allgather(dims, offs, 4, send, lib=lib).view(np.int32).reshape(16, 8)
    n = 0
    for line in open(os.path.join(GOLDEN, "moore_4x4_allgather.txt")):
        if line.startswith("#") or not line.strip():
            continue
        rank, vals = line.split(":")
        assert recv[int(rank)].tolist() == [int(v) for v in vals.split()], "rank " + rank
        n += 1
    assert n == 2


def pin_push_equals_pull(lib):
    rng = np.random.default_rng(7)
    cases = [((1,), 3), ((2,), 4), ((4,), 5), ((3, 2), 6), ((2, 3, 4), 9), ((1, 4), 4), ((4, 3), 12)]
    for dims, s in cases:
        d = len(dims)
        P = int(np.prod(dims))
        offs = rng.integers(-5, 6, size=(s, d)).astype(np.int32)
        offs[0] = 0                      # a message to oneself
        if s > 2:
            offs[2] = offs[1]            # a repeated neighbour
        lens = rng.integers(0, 7, size=s).astype(np.int64)
        sd = np.concatenate([[0], np.cumsum(lens)[:-1]]).astype(np.int64)
        perm = rng.permutation(s)        # receive layout differs from the send layout
        rd = np.zeros(s, dtype=np.int64)
        cur = 1
        for i in perm:
            rd[i] = cur
            cur += lens[i] + 1
        sstride, rstride = int(lens.sum()) + 2, int(cur) + 3
        send = rng.integers(0, 256, size=(P, sstride), dtype=np.uint8)
        want, written = push_alltoallv(dims, offs, lens, sd, rd, sstride, rstride, send, fill=0xA5)
        covered = np.zeros(rstride, dtype=np.int32)
        for i in range(s):
            covered[rd[i]:rd[i] + lens[i]] += 1
        assert (written == covered[None, :]).all(), "every block arrives exactly once"
        got = oracle.alltoallv(dims, offs, lens, sd, rd, sstride, rstride, send, fill=0xA5, lib=lib)
        assert np.array_equal(got, want), (dims, s)
        # regular all-to-all and allgather, stated from the sender's side
        m = 3
        send2 = rng.integers(0, 256, size=(P, s * m), dtype=np.uint8)
        ld = np.full(s, m, dtype=np.int64)
        dd = np.arange(s, dtype=np.int64) * m
        want2, _ = push_alltoallv(dims, offs, ld, dd, dd, s * m, s * m, send2)
        assert np.array_equal(oracle.alltoall(dims, offs, m, send2, lib=lib), want2)
        send3 = rng.integers(0, 256, size=(P, m), dtype=np.uint8)
        want3, _ = push_alltoallv(dims, offs, ld, np.zeros(s, np.int64), dd, m, s * m, send3)
        assert np.array_equal(oracle.allgather(dims, offs, m, send3, lib=lib), want3)


def pin_numpy_special_cases(lib):
    rng = np.random.default_rng(11)
    # d=1, single offset +c: a cyclic rotation of the process axis
    p, m = 7, 5
    send = rng.integers(0, 256, size=(p, m), dtype=np.uint8)
    for c in (1, -2, 9):
        got = oracle.alltoall((p,), [[c]], m, send, lib=lib)
        assert np.array_equal(got, np.roll(send, c, axis=0))
    # 3-D torus, one offset vector: np.roll over the reshaped process axes pins the
    # row-major (last dimension fastest) rank order
    dims = (3, 4, 5)
    P = 60
    send = rng.integers(0, 256, size=(P, m), dtype=np.uint8)
    C = (1, -1, 2)
    want = np.roll(send.reshape(*dims, m), C, axis=(0, 1, 2)).reshape(P, m)
    assert np.array_equal(oracle.alltoall(dims, [C], m, send, lib=lib), want)
    assert np.array_equal(oracle.allgather(dims, [C], m, send, lib=lib), want)
    # d=1, offsets 1..p-1: the dense all-to-all; recv[r][i] = send[r-(i+1)][i]
    p, m = 6, 2
    offs = [[k] for k in range(1, p)]
    send = rng.integers(0, 256, size=(p, p - 1, m), dtype=np.uint8)
    got = oracle.alltoall((p,), offs, m, send, lib=lib).reshape(p, p - 1, m)
    want = np.stack([np.roll(send[:, i], i + 1, axis=0) for i in range(p - 1)], axis=1)
    assert np.array_equal(got, want)
    # dense allgather: everybody ends with everybody else's block, in ring order
    blk = rng.integers(0, 256, size=(p, m), dtype=np.uint8)
    got = oracle.allgather((p,), offs, m, blk, lib=lib).reshape(p, p - 1, m)
    want = np.stack([np.roll(blk, i + 1, axis=0) for i in range(p - 1)], axis=1)
    assert np.array_equal(got, want)
    # the zero vector alone is a copy
    send = rng.integers(0, 256, size=(12, 4), dtype=np.uint8)
    assert np.array_equal(oracle.alltoall((3, 4), [[0, 0]], 4, send, lib=lib), send)
    # irregular with equal lengths and packed displacements is the regular collective
    dims, s, m = (3, 3), 8, 4
    offs = moore_list(2, 1)
    send = rng.integers(0, 256, size=(9, s * m), dtype=np.uint8)
    dd = np.arange(s) * m
    a = oracle.alltoall(dims, offs, m, send, lib=lib)
    b = oracle.alltoallv(dims, offs, [m] * s, dd, dd, s * m, s * m, send, lib=lib)
    assert np.array_equal(a, b)
    # swapping send and receive displacements is visible when they differ
    sd = np.array([0, 4, 8]); rd = np.array([8, 0, 4])
    send = np.arange(5 * 12, dtype=np.uint8).reshape(5, 12)
    got = oracle.alltoallv((5,), [[0], [0], [0]], [4, 4, 4], sd, rd, 12, 12, send, lib=lib)
    want = np.concatenate([send[:, 4:8], send[:, 8:12], send[:, 0:4]], axis=1)
    assert np.array_equal(got, want)


def pin_rank_helpers(lib):
    dims = (2, 3, 4)
    for r in range(24):
        R = coords_of(r, dims)
        for C in [(0, 0, 0), (1, 0, 0), (0, -1, 0), (0, 0, 5), (-3, 4, -9)]:
            src = rank_of([(a - c) % p for a, c, p in zip(R, C, dims)], dims)
            dst = rank_of([(a + c) % p for a, c, p in zip(R, C, dims)], dims)
            assert oracle.source_rank(dims, r, C, lib=lib) == src
            assert oracle.target_rank(dims, r, C, lib=lib) == dst


def pin_chunks(lib):
    rng = np.random.default_rng(3)
    dims, m = (4, 5), 3
    offs = moore_list(2, 1)
    send = rng.integers(0, 256, size=(20, 8 * m), dtype=np.uint8)
    full = oracle.alltoall(dims, offs, m, send, lib=lib)
    parts = [oracle.alltoall(dims, offs, m, send, r0, r1, lib=lib) for r0, r1 in ((0, 7), (7, 8), (8, 20))]
    assert np.array_equal(np.concatenate(parts), full)


def _padded(rows, width, dtype=np.uint8, rng=None):
    """`rows` x `width` array that is a view into a larger allocation, so that a planted
    off-by-one in a mesh bound reads defined memory instead of running off the array."""
    backing = np.zeros((rows + 16, width), dtype=dtype) if rng is None else \
        rng.integers(0, 256, size=(rows + 16, width)).astype(dtype)
    return backing[:rows]


def pin_golden_mesh(lib):
    dims, periodic, offs = (3, 4), (0, 0), moore_list(2, 1)
    P, s = 12, 8
    send = _padded(P, s, np.int32)
    send[:] = [[100 * q + i for i in range(s)] for q in range(P)]
    KEEP = 0x77
    recv = oracle.alltoall(dims, offs, 4, send, lib=lib, periodic=periodic, fill=KEEP).view(np.int32).reshape(P, s)
    kept = int(np.array([KEEP] * 4, np.uint8).view(np.int32)[0])
    n = 0
    for line in open(os.path.join(GOLDEN, "mesh_3x4_alltoall.txt")):
        if line.startswith("#") or not line.strip():
            continue
        rank, vals = line.split(":")
        want = [kept if v == "-" else int(v) for v in vals.split()]
        assert recv[int(rank)].tolist() == want, "rank " + rank
        n += 1
    assert n == 4
    # the same geometry as an allgather: slot i holds the source's single value or is kept
    blk = _padded(P, 1, np.int32)
    blk[:, 0] = [100 * q for q in range(P)]
    got = oracle.allgather(dims, offs, 4, blk, lib=lib, periodic=periodic, fill=KEEP).view(np.int32).reshape(P, s)
    assert got[0].tolist() == [500, 400, kept, 100, kept, kept, kept, kept]
    assert got[11].tolist() == [kept, kept, kept, kept, 1000, kept, 700, 600]


def push_mesh(dims, periodic, offsets, lens, sdispls, rdispls, sstride, rstride, send, fill):
    """Sender's side on a mesh: q sends block i to q + C^i if that process exists."""
    P = int(np.prod(dims))
    recv = np.full((P, rstride), fill, dtype=np.uint8)
    for q in range(P):
        Q = coords_of(q, dims)
        for i, C in enumerate(offsets):
            T = []
            for a, c, p, per in zip(Q, C, dims, periodic):
                t = a + int(c)
                if per:
                    t %= p
                elif not 0 <= t < p:
                    T = None
                    break
                T.append(t)
            if T is None:
                continue
            t = rank_of(T, dims)
            recv[t, rdispls[i]:rdispls[i] + lens[i]] = send[q, sdispls[i]:sdispls[i] + lens[i]]
    return recv


def pin_mesh_push_equals_pull(lib):
    rng = np.random.default_rng(19)
    for dims, periodic in [((5,), (0,)), ((3, 4), (0, 1)), ((3, 4), (1, 0)), ((2, 3, 4), (0, 1, 0)), ((4, 1, 3), (0, 0, 0)),
                           ((3, 3), (1, 1))]:
        d, P = len(dims), int(np.prod(dims))
        s = 9
        offs = rng.integers(-4, 5, size=(s, d)).astype(np.int32)
        offs[0] = 0
        offs[3] = offs[2]
        m = 3
        ld, dd = np.full(s, m, np.int64), np.arange(s, dtype=np.int64) * m
        send = _padded(P, s * m, rng=rng)
        want = push_mesh(dims, periodic, offs, ld, dd, dd, s * m, s * m, send, 0xA5)
        assert np.array_equal(oracle.alltoall(dims, offs, m, send, lib=lib, periodic=periodic, fill=0xA5), want), (dims, periodic)
        got = oracle.alltoallv(dims, offs, ld, dd, dd[::-1].copy(), s * m, s * m, send, fill=0xA5, lib=lib, periodic=periodic)
        assert np.array_equal(got, push_mesh(dims, periodic, offs, ld, dd, dd[::-1], s * m, s * m, send, 0xA5)), (dims, periodic)
        blk = _padded(P, m, rng=rng)
        want = push_mesh(dims, periodic, offs, ld, np.zeros(s, np.int64), dd, m, s * m, blk, 0xA5)
        assert np.array_equal(oracle.allgather(dims, offs, m, blk, lib=lib, periodic=periodic, fill=0xA5), want), (dims, periodic)
        for r in range(P):
            R = coords_of(r, dims)
            for C in offs:
                src = [a - int(c) for a, c in zip(R, C)]
                inside = all(per or 0 <= y < p for y, p, per in zip(src, dims, periodic))
                q = oracle.source_rank_mesh(dims, periodic, r, C, lib=lib)
                assert (q >= 0) == inside
                if inside:
                    assert q == rank_of([y % p for y, p in zip(src, dims)], dims)


PINS = [pin_golden_mesh, pin_mesh_push_equals_pull, pin_golden, pin_golden_allgather, pin_push_equals_pull, pin_numpy_special_cases, pin_rank_helpers, pin_chunks]


@pytest.mark.parametrize("pin", PINS, ids=lambda f: f.__name__)
def test_oracle_pin(pin, oracle_lib):
    pin(oracle_lib)


# ------------------------------------------------------------------------------ mutants
MUTANTS = {
    "adds_instead_of_subtracts": ("(coord[j] - (int64_t)C[j]) % p", "(coord[j] + (int64_t)C[j]) % p"),
    "no_wrap_of_negative": ("        if (x < 0)\n            x += p;\n", ""),
    "first_dimension_fastest": ("    for (j = d - 1; j >= 0; j--) {\n        coord[j] = rest % dims[j];",
                                "    for (j = 0; j < d; j++) {\n        coord[j] = rest % dims[j];"),
    "recompose_reversed": ("    for (j = 0; j < d; j++)\n        rest = rest * dims[j] + coord[j];",
                           "    for (j = d - 1; j >= 0; j--)\n        rest = rest * dims[j] + coord[j];"),
    "alltoall_drops_block_index": ("send + (q * s + i) * m", "send + (q * s) * m"),
    "alltoall_reads_own_block": ("send + (q * s + i) * m", "send + (r * s + i) * m"),
    "allgather_reads_own_block": ("send + q * m, (size_t)m", "send + r * m, (size_t)m"),
    "alltoallv_swaps_displacements": ("recv + (r - r0) * recv_stride + rdispl[i],\n                   send + q * send_stride + sdispl[i]",
                                      "recv + (r - r0) * recv_stride + sdispl[i],\n                   send + q * send_stride + rdispl[i]"),
    "alltoallv_wrong_stride": ("send + q * send_stride + sdispl[i]", "send + q * recv_stride + sdispl[i]"),
    "mesh_checks_the_receiver_side": ("int64_t y = coord[j] - (int64_t)C[j];", "int64_t y = coord[j] + (int64_t)C[j];"),
    "mesh_upper_edge_inclusive": ("} else if (y < 0 || y >= p) {", "} else if (y < 0 || y > p) {"),
    "mesh_flags_ignored": ("        if (periodic[j]) {\n            y = y % p;", "        if (1) {\n            y = y % p;"),
    "mesh_allgather_reads_own_block": ("            memcpy(recv + ((r - r0) * s + i) * m, send + q * m, (size_t)m);\n        }\n    }\n    return 0;\n}\n\n/* Irregular all-to-all on a mesh",
                                       "            memcpy(recv + ((r - r0) * s + i) * m, send + r * m, (size_t)m);\n        }\n    }\n    return 0;\n}\n\n/* Irregular all-to-all on a mesh"),
    "offset_row_ignored": ("offsets + (int64_t)i * d);\n            memcpy(recv + ((r - r0) * s + i) * m, send + (q * s + i) * m",
                           "offsets + (int64_t)0 * d);\n            memcpy(recv + ((r - r0) * s + i) * m, send + (q * s + i) * m"),
}


@pytest.mark.parametrize("name", sorted(MUTANTS))
def test_pins_reject_mutant(name, tmp_path):
    old, new = MUTANTS[name]
    src = open(os.path.join(ROOT, "oracle", "iso_oracle.c")).read()
    assert src.count(old) >= 1, "mutation site not found: " + name
    mutated = src.replace(old, new, 1)
    cfile = tmp_path / "mutant.c"
    cfile.write_text(mutated)
    so = tmp_path / "mutant.so"
    subprocess.check_call(["gcc", "-O1", "-std=c99", "-fPIC", "-shared", "-o", str(so), str(cfile)])
    lib = oracle.load(str(so))
    failed = []
    for pin in PINS:
        try:
            pin(lib)
        except (AssertionError, ValueError):
            failed.append(pin.__name__)
    assert failed, "no pin noticed the planted mistake '%s'" % name
