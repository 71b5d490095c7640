"""Seeded synthetic workloads: neighbourhood lists and buffer contents.

This module holds input generators only, none of the collective's arithmetic, so
that the CUDA library's tests, the benchmark and the CPU oracle's tests can all
draw the same inputs from it.  Buffer contents are counter based: the 32-bit word
at word index g of a buffer is a fixed function of (seed, stream, g), so any slice
of a buffer can be produced on its own, on the host (numpy) or on the device
(torch), without generating the rest.

The neighbourhoods are the ones the paper benchmarks (Section IV): Moore
neighbourhoods of radius r in d dimensions, listed in lexicographic order with the
last coordinate varying fastest and the origin left out; the positive-octant
variant; and two Chebyshev shells.
"""
from __future__ import annotations

import itertools
from dataclasses import dataclass, field

import numpy as np

DEFAULT_SEED = 20160707
_MASK64 = (1 << 64) - 1
_GOLDEN = 0x9E3779B97F4A7C15
_M1 = 0xBF58476D1CE4E5B9
_M2 = 0x94D049BB133111EB


# --------------------------------------------------------------------------- mixer
def mix64(x: int) -> int:
    """splitmix64 output function on a Python integer."""
    z = (x + _GOLDEN) & _MASK64
    z = ((z ^ (z >> 30)) * _M1) & _MASK64
    z = ((z ^ (z >> 27)) * _M2) & _MASK64
    return z ^ (z >> 31)


def _mix64_np(x: np.ndarray) -> np.ndarray:
    z = x + np.uint64(_GOLDEN)
    z = (z ^ (z >> np.uint64(30))) * np.uint64(_M1)
    z = (z ^ (z >> np.uint64(27))) * np.uint64(_M2)
    return z ^ (z >> np.uint64(31))


def _signed(v: int) -> int:
    v &= _MASK64
    return v - (1 << 64) if v >> 63 else v


def _lsr_torch(z, k: int):
    # logical shift right of an int64 tensor
    return (z >> k) & ((1 << (64 - k)) - 1)


def _mix64_torch(x):
    z = x + _signed(_GOLDEN)
    z = (z ^ _lsr_torch(z, 30)) * _signed(_M1)
    z = (z ^ _lsr_torch(z, 27)) * _signed(_M2)
    return z ^ _lsr_torch(z, 31)


def _base(seed: int, stream: int) -> int:
    return mix64((seed * 2654435761 + stream) & _MASK64)


def words_np(seed: int, stream: int, start: int, n: int) -> np.ndarray:
    """uint32 words [start, start+n) of buffer `stream` (numpy, host)."""
    g = np.arange(start, start + n, dtype=np.uint64)
    with np.errstate(over="ignore"):
        z = _mix64_np(np.uint64(_base(seed, stream)) + g * np.uint64(_GOLDEN))
    return (z >> np.uint64(32)).astype(np.uint32)


def words_torch(seed: int, stream: int, start: int, n: int, device, chunk: int = 1 << 26):
    """The same words as `words_np`, produced on `device` as an int32 tensor."""
    import torch

    out = torch.empty(n, dtype=torch.int32, device=device)
    base = _signed(_base(seed, stream))
    for lo in range(0, n, chunk):
        hi = min(n, lo + chunk)
        g = torch.arange(start + lo, start + hi, dtype=torch.int64, device=device)
        z = _mix64_torch(g * _signed(_GOLDEN) + base)
        out[lo:hi] = _lsr_torch(z, 32).to(torch.int32)
    return out


KINDS = ("int32", "fp32", "uint8")


def payload_np(kind: str, seed: int, stream: int, start_byte: int, nbytes: int) -> np.ndarray:
    """Bytes [start_byte, start_byte+nbytes) of a buffer, as uint8.

    kind: "int32" (all bit patterns), "fp32" (uniform in [-1, 1), exact multiples of
    2^-23), "uint8" (the bytes of the words).  Offsets are in bytes of the buffer.
    """
    w0 = start_byte // 4
    w1 = (start_byte + nbytes + 3) // 4
    w = words_np(seed, stream, w0, w1 - w0)
    if kind == "fp32":
        f = (w >> np.uint32(8)).astype(np.float32) * np.float32(2.0 ** -23) - np.float32(1.0)
        raw = f.view(np.uint8)
    elif kind in ("int32", "uint8"):
        raw = w.view(np.uint8)
    else:
        raise ValueError(kind)
    lo = start_byte - 4 * w0
    return raw[lo:lo + nbytes]


def payload_torch(kind: str, seed: int, stream: int, nbytes: int, device):
    """A whole buffer of `nbytes` bytes on `device`, as a uint8 tensor (nbytes % 4 == 0)."""
    import torch

    if nbytes % 4:
        raise ValueError("buffer sizes are multiples of 4 bytes")
    w = words_torch(seed, stream, 0, nbytes // 4, device)
    if kind == "fp32":
        f = ((w >> 8) & 0xFFFFFF).to(torch.float32) * (2.0 ** -23) - 1.0
        return f.view(torch.uint8)
    if kind in ("int32", "uint8"):
        return w.view(torch.uint8)
    raise ValueError(kind)


class Stream:
    """Sequential splitmix64 stream for the few scalar draws of a recipe."""

    def __init__(self, seed: int):
        self.state = seed & _MASK64

    def next(self) -> int:
        v = mix64(self.state)
        self.state = (self.state + _GOLDEN) & _MASK64
        return v

    def below(self, n: int) -> int:
        return self.next() % n


# ------------------------------------------------------------------ neighbourhoods
def moore(d: int, r: int) -> np.ndarray:
    """All vectors of {-r..r}^d but the origin, lexicographic, last coordinate fastest."""
    rows = [v for v in itertools.product(range(-r, r + 1), repeat=d) if any(v)]
    return np.asarray(rows, dtype=np.int32).reshape(-1, d)


def positive_octant(d: int, r: int) -> np.ndarray:
    """The vectors of {0..r}^d but the origin (the paper's asymmetric neighbourhood)."""
    rows = [v for v in itertools.product(range(0, r + 1), repeat=d) if any(v)]
    return np.asarray(rows, dtype=np.int32).reshape(-1, d)


def shells(d: int, radii) -> np.ndarray:
    """The vectors whose Chebyshev norm is one of `radii` ("shales" in the paper)."""
    radii = set(radii)
    rmax = max(radii)
    rows = [v for v in itertools.product(range(-rmax, rmax + 1), repeat=d)
            if max(abs(c) for c in v) in radii]
    return np.asarray(rows, dtype=np.int32).reshape(-1, d)


def random_offsets(seed: int, d: int, s: int, lo: int, hi: int) -> np.ndarray:
    """s distinct non-zero vectors, every coordinate drawn uniformly in [lo, hi]."""
    st = Stream(seed + 1)
    span = hi - lo + 1
    if s > span ** d - (1 if lo <= 0 <= hi else 0):
        raise ValueError("not that many distinct vectors")
    seen, rows = set(), []
    while len(rows) < s:
        v = tuple(lo + st.below(span) for _ in range(d))
        if not any(v) or v in seen:
            continue
        seen.add(v)
        rows.append(v)
    return np.asarray(rows, dtype=np.int32).reshape(-1, d)


def random_sizes(seed: int, s: int, choices=(4, 16, 64, 256, 1024)) -> np.ndarray:
    """One block length per neighbour, uniform over `choices`."""
    st = Stream(seed + 2)
    return np.asarray([choices[st.below(len(choices))] for _ in range(s)], dtype=np.int64)


def packed_displacements(lens) -> np.ndarray:
    """Exclusive prefix sums of the lengths (blocks stored back to back)."""
    lens = np.asarray(lens, dtype=np.int64)
    out = np.zeros_like(lens)
    if lens.size:
        out[1:] = np.cumsum(lens)[:-1]
    return out


# -------------------------------------------------------------------------- configs
@dataclass
class Workload:
    """One benchmark / parity configuration."""
    name: str
    collective: str            # "alltoall" | "allgather" | "alltoallv"
    dims: tuple
    offsets: np.ndarray        # [s, d]
    block_bytes: int = 0       # regular collectives
    lens: np.ndarray | None = None   # alltoallv
    kind: str = "uint8"        # payload kind
    seed: int = DEFAULT_SEED
    extra: dict = field(default_factory=dict)

    @property
    def P(self) -> int:
        return int(np.prod(self.dims, dtype=np.int64))

    @property
    def s(self) -> int:
        return int(self.offsets.shape[0])

    @property
    def d(self) -> int:
        return len(self.dims)


def config(name: str, seed: int = DEFAULT_SEED) -> Workload:
    """The named workloads.

    cfg1           all-to-all, 8x8, Moore r=1, 2 int32 per block
    cfg2_alltoall  all-to-all, 32^3, Moore r=1, 64 B of fp32 in [-1,1)
    cfg2_allgather allgather,  same torus and neighbourhood
    cfg3_m<M>      all-to-all, 256^2, Moore r=2, M in {4,64,512,4096} uint8 bytes
                   (cfg3_m<M>_<a>x<b>: the same on an a x b torus)
    cfg4           all-to-all, 8^5, Moore r=1, 16 B of fp32
    cfg5           irregular all-to-all, 64x64x32, 30 random offsets in [-3,3]^3,
                   lengths uniform over {4,16,64,256,1024} B, packed displacements
                   (cfg5_32x32x32: the same on a 32^3 torus)
    <nbh>_alltoall / <nbh>_allgather with nbh in moore_d3r3 (342 neighbours), octant_d3r3
                   (63), shells_d3 (1396, Chebyshev distances 3 and 7) on 32^3 and moore_d4r1
                   (80) on 16^4: the paper's larger neighbourhoods, 64-byte blocks
    """
    if name == "cfg1":
        return Workload(name, "alltoall", (8, 8), moore(2, 1), 8, kind="int32", seed=seed)
    if name == "cfg2_alltoall":
        return Workload(name, "alltoall", (32, 32, 32), moore(3, 1), 64, kind="fp32", seed=seed)
    if name == "cfg2_allgather":
        return Workload(name, "allgather", (32, 32, 32), moore(3, 1), 64, kind="fp32", seed=seed)
    if name.startswith("cfg3_m"):
        # cfg3_m<M>_<a>x<b>: the same neighbourhood and block size on an a x b torus (fewer rows,
        # same row length: the case profiler captures with many passes are taken on)
        size, _, shape = name[len("cfg3_m"):].partition("_")
        dims = tuple(int(x) for x in shape.split("x")) if shape else (256, 256)
        return Workload(name, "alltoall", dims, moore(2, 2), int(size), kind="uint8", seed=seed)
    if name == "cfg4":
        return Workload(name, "alltoall", (8, 8, 8, 8, 8), moore(5, 1), 16, kind="fp32", seed=seed)
    if name in ("cfg5", "cfg5_32x32x32"):
        # cfg5_32x32x32: the same draws on a quarter of the processes (1.3 GB instead of 5.2 GB on
        # the device), the case profiler captures with many passes are taken on
        offs = random_offsets(seed, 3, 30, -3, 3)
        lens = random_sizes(seed, 30)
        dims = (64, 64, 32) if name == "cfg5" else (32, 32, 32)
        return Workload(name, "alltoallv", dims, offs, 0, lens=lens, kind="uint8", seed=seed)
    if name.startswith("stencil_d3_m"):
        # the paper's irregular experiment (Section IV): block to neighbour i has mhat^(d - ||C^i||_1)
        # bytes, so corners get 1 byte, edges mhat, faces mhat^2; packed displacements
        mhat = int(name[len("stencil_d3_m"):])
        offs = moore(3, 1)
        lens = np.asarray([mhat ** (3 - int(np.abs(v).sum())) for v in offs], dtype=np.int64)
        return Workload(name, "alltoallv", (32, 32, 32), offs, 0, lens=lens, kind="uint8", seed=seed)
    # neighbourhoods of the paper's second set of experiments (Sections IV and VI), 64-byte blocks
    paper = {"moore_d3r3": ((32, 32, 32), lambda: moore(3, 3)), "octant_d3r3": ((32, 32, 32), lambda: positive_octant(3, 3)),
             "shells_d3": ((32, 32, 32), lambda: shells(3, (3, 7))), "moore_d4r1": ((16, 16, 16, 16), lambda: moore(4, 1))}
    for key, (dims, make) in paper.items():
        for coll in ("alltoall", "allgather"):
            if name == "%s_%s" % (key, coll):
                return Workload(name, coll, dims, make(), 64, kind="fp32", seed=seed)
    raise KeyError(name)


def layout(w: Workload):
    """(lens, send displacements, receive displacements, send stride, receive stride), in
    bytes, of a workload's buffers under the interface's layout rules: regular blocks back
    to back; irregular blocks packed, process stride rounded up to 16 bytes."""
    s = w.s
    if w.collective == "alltoall":
        m = w.block_bytes
        dd = np.arange(s, dtype=np.int64) * m
        return np.full(s, m, np.int64), dd, dd, s * m, s * m
    if w.collective == "allgather":
        m = w.block_bytes
        return np.full(s, m, np.int64), np.zeros(s, np.int64), np.arange(s, dtype=np.int64) * m, m, s * m
    lens = np.asarray(w.lens, np.int64)
    dd = packed_displacements(lens)
    stride = (int(lens.sum()) + 15) // 16 * 16
    return lens, dd, dd, stride, stride


def send_buffer_np(w: Workload, send_stride: int) -> np.ndarray:
    """Host copy of the seeded send buffers of a workload (uint8 [P, send_stride])."""
    return payload_np(w.kind, w.seed, 0, 0, w.P * send_stride).reshape(w.P, send_stride).copy()


PAPER_NAMES = tuple("%s_%s" % (k, c) for k in ("moore_d3r3", "octant_d3r3", "shells_d3", "moore_d4r1")
                    for c in ("alltoall", "allgather")) + ("stencil_d3_m32", "stencil_d3_m512")

CONFIG_NAMES = ("cfg1", "cfg2_alltoall", "cfg2_allgather", "cfg3_m4", "cfg3_m64", "cfg3_m512",
                "cfg3_m4096", "cfg4", "cfg5")
