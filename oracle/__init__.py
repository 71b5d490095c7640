"""CPU oracle for the isomorphic neighbourhood collectives (TEST INFRASTRUCTURE ONLY).

The arithmetic lives in ``iso_oracle.c`` (plain C, the direct definition of the
result from Section II of the paper) and in ``counters.py`` (the paper's round and
volume formulas).  This module only compiles the C file with gcc and marshals numpy
arrays into it.  Nothing here is shared with, imported by, or imports the CUDA
library; only tests, the smoke check and the benchmark's CPU-baseline leg use it.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "iso_oracle.c")
_LIB = os.path.join(_HERE, "libiso_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle (gcc -O2, no OpenMP) and return the library path."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c99", "-fPIC", "-shared", "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


def load(path: str | None = None) -> ctypes.CDLL:
    """Load the compiled oracle (building it first when needed)."""
    global _lib
    with _lock:
        if path is not None:
            return _declare(ctypes.CDLL(path))
        if _lib is None:
            _lib = _declare(ctypes.CDLL(build()))
        return _lib


def _declare(lib: ctypes.CDLL) -> ctypes.CDLL:
    i64, ci, vp = ctypes.c_int64, ctypes.c_int, ctypes.c_void_p
    lib.iso_oracle_source_rank.restype = i64
    lib.iso_oracle_source_rank.argtypes = [ci, vp, i64, vp]
    lib.iso_oracle_target_rank.restype = i64
    lib.iso_oracle_target_rank.argtypes = [ci, vp, i64, vp]
    for name in ("iso_oracle_alltoall", "iso_oracle_allgather"):
        f = getattr(lib, name)
        f.restype = ci
        f.argtypes = [ci, vp, ci, vp, i64, vp, vp, i64, i64]
    lib.iso_oracle_alltoallv.restype = ci
    lib.iso_oracle_alltoallv.argtypes = [ci, vp, ci, vp, vp, vp, vp, i64, i64, vp, vp, i64, i64]
    lib.iso_oracle_source_rank_mesh.restype = i64
    lib.iso_oracle_source_rank_mesh.argtypes = [ci, vp, vp, i64, vp]
    for name in ("iso_oracle_alltoall_mesh", "iso_oracle_allgather_mesh"):
        f = getattr(lib, name)
        f.restype = ci
        f.argtypes = [ci, vp, vp, ci, vp, i64, vp, vp, i64, i64]
    lib.iso_oracle_alltoallv_mesh.restype = ci
    lib.iso_oracle_alltoallv_mesh.argtypes = [ci, vp, vp, ci, vp, vp, vp, vp, i64, i64, vp, vp, i64, i64]
    return lib


def _ints(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32).reshape(-1))


def _i64s(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.int64).reshape(-1))


def _ptr(a: np.ndarray) -> int:
    return a.ctypes.data


def _geometry(dims, offsets):
    dims = _ints(dims)
    d = int(dims.size)
    offs = _ints(offsets)
    if d == 0 or offs.size % d:
        raise ValueError("offsets must hold s*d integers")
    return dims, d, offs, offs.size // d


def _bytes_view(a: np.ndarray) -> np.ndarray:
    a = np.ascontiguousarray(a)
    return a.view(np.uint8).reshape(-1)


def source_rank(dims, r: int, C, lib=None) -> int:
    """rank(R (-) C) for the process of rank r (Section II)."""
    lib = lib or load()
    dims = _ints(dims)
    C = _ints(C)
    return int(lib.iso_oracle_source_rank(dims.size, _ptr(dims), int(r), _ptr(C)))


def target_rank(dims, r: int, C, lib=None) -> int:
    """rank(R (+) C) for the process of rank r (Section II)."""
    lib = lib or load()
    dims = _ints(dims)
    C = _ints(C)
    return int(lib.iso_oracle_target_rank(dims.size, _ptr(dims), int(r), _ptr(C)))


def source_rank_mesh(dims, periodic, r: int, C, lib=None) -> int:
    """rank(R - C) on a torus whose dimensions with periodic[j] == 0 do not wrap; -1 when
    that process does not exist (Section VII)."""
    lib = lib or load()
    dims, periodic, C = _ints(dims), _ints(periodic), _ints(C)
    return int(lib.iso_oracle_source_rank_mesh(dims.size, _ptr(dims), _ptr(periodic), int(r), _ptr(C)))


def _mesh_flags(periodic, d):
    """None when every dimension wraps (the plain functions apply), else the flags."""
    if periodic is None:
        return None
    flags = _ints(periodic)
    if flags.size != d:
        raise ValueError("periodic must hold d flags")
    return None if bool(flags.all()) else flags


def alltoall(dims, offsets, m: int, send: np.ndarray, r0: int = 0, r1: int | None = None,
             lib=None, periodic=None, fill: int = 0) -> np.ndarray:
    """Receive buffers (uint8, shape [r1-r0, s*m]) of a regular all-to-all.

    With non-periodic dimensions (`periodic`), slots whose source lies outside the mesh
    keep the value ``fill``."""
    lib = lib or load()
    dims, d, offs, s = _geometry(dims, offsets)
    P = int(np.prod(dims, dtype=np.int64))
    r1 = P if r1 is None else r1
    sb = _bytes_view(send)
    if sb.size != P * s * m:
        raise ValueError("send buffer must hold P*s*m bytes")
    flags = _mesh_flags(periodic, d)
    if flags is not None:
        out = np.full((r1 - r0, s * m), fill, dtype=np.uint8)
        rc = lib.iso_oracle_alltoall_mesh(d, _ptr(dims), _ptr(flags), s, _ptr(offs), m, _ptr(sb), _ptr(out), r0, r1)
        if rc:
            raise ValueError("oracle rejected the arguments")
        return out
    out = np.empty((r1 - r0, s * m), dtype=np.uint8)
    rc = lib.iso_oracle_alltoall(d, _ptr(dims), s, _ptr(offs), m, _ptr(sb), _ptr(out), r0, r1)
    if rc:
        raise ValueError("oracle rejected the arguments")
    return out


def allgather(dims, offsets, m: int, send: np.ndarray, r0: int = 0, r1: int | None = None,
              lib=None, periodic=None, fill: int = 0) -> np.ndarray:
    """Receive buffers (uint8, shape [r1-r0, s*m]) of an allgather (`periodic`, `fill`: as
    for `alltoall`)."""
    lib = lib or load()
    dims, d, offs, s = _geometry(dims, offsets)
    P = int(np.prod(dims, dtype=np.int64))
    r1 = P if r1 is None else r1
    sb = _bytes_view(send)
    if sb.size != P * m:
        raise ValueError("send buffer must hold P*m bytes")
    flags = _mesh_flags(periodic, d)
    if flags is not None:
        out = np.full((r1 - r0, s * m), fill, dtype=np.uint8)
        rc = lib.iso_oracle_allgather_mesh(d, _ptr(dims), _ptr(flags), s, _ptr(offs), m, _ptr(sb), _ptr(out), r0, r1)
        if rc:
            raise ValueError("oracle rejected the arguments")
        return out
    out = np.empty((r1 - r0, s * m), dtype=np.uint8)
    rc = lib.iso_oracle_allgather(d, _ptr(dims), s, _ptr(offs), m, _ptr(sb), _ptr(out), r0, r1)
    if rc:
        raise ValueError("oracle rejected the arguments")
    return out


def alltoallv(dims, offsets, lens, sdispls, rdispls, send_stride: int, recv_stride: int,
              send: np.ndarray, r0: int = 0, r1: int | None = None, fill: int = 0,
              lib=None, periodic=None) -> np.ndarray:
    """Receive buffers (uint8, shape [r1-r0, recv_stride]) of an irregular all-to-all.

    Bytes of the receive buffer that no block covers keep the value ``fill``.
    """
    lib = lib or load()
    dims, d, offs, s = _geometry(dims, offsets)
    P = int(np.prod(dims, dtype=np.int64))
    r1 = P if r1 is None else r1
    lens, sdispls, rdispls = _i64s(lens), _i64s(sdispls), _i64s(rdispls)
    if not (lens.size == sdispls.size == rdispls.size == s):
        raise ValueError("lens / displacements must have s entries")
    if s and (int((sdispls + lens).max()) > send_stride or int((rdispls + lens).max()) > recv_stride):
        raise ValueError("a block reaches past the process stride")
    sb = _bytes_view(send)
    if sb.size != P * send_stride:
        raise ValueError("send buffer must hold P*send_stride bytes")
    out = np.full((r1 - r0, recv_stride), fill, dtype=np.uint8)
    flags = _mesh_flags(periodic, d)
    if flags is not None:
        rc = lib.iso_oracle_alltoallv_mesh(d, _ptr(dims), _ptr(flags), s, _ptr(offs), _ptr(lens), _ptr(sdispls),
                                           _ptr(rdispls), send_stride, recv_stride, _ptr(sb), _ptr(out), r0, r1)
        if rc:
            raise ValueError("oracle rejected the arguments")
        return out
    rc = lib.iso_oracle_alltoallv(d, _ptr(dims), s, _ptr(offs), _ptr(lens), _ptr(sdispls),
                                  _ptr(rdispls), send_stride, recv_stride, _ptr(sb), _ptr(out),
                                  r0, r1)
    if rc:
        raise ValueError("oracle rejected the arguments")
    return out
