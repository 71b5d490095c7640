"""ctypes binding of the C-ABI library (``include/iso.h``): argument marshalling only.

Every function has the name of the C entry point it calls, takes numpy arrays / torch
tensors / plain integers, and raises `IsoError` when the library returns a non-zero code.
Device buffers are passed as integer addresses (``tensor.data_ptr()``) or as torch tensors;
streams as ``torch.cuda.Stream`` objects, raw ``cudaStream_t`` integers or None.
There is no fallback: if the compiled library is missing, loading raises.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np

ISO_MAX_DIMS = 8
ISO_ALG_COMBINING, ISO_ALG_DIRECT, ISO_ALG_TORUS = 0, 1, 2
ISO_KIND_ALLTOALL, ISO_KIND_ALLGATHER, ISO_KIND_ALLTOALLV = 0, 1, 2
ISO_BUF_SEND, ISO_BUF_RECV, ISO_BUF_INTER = 0, 1, 2
ISO_LAYOUT_PACKED, ISO_LAYOUT_ALTERNATING = 0, 1
ISO_BYTE, ISO_INT32, ISO_FLOAT, ISO_DOUBLE = 1, 4, 4, 8
(ISO_SUCCESS, ISO_ERR_ARG, ISO_ERR_DIMS, ISO_ERR_COUNT, ISO_ERR_ALIGN, ISO_ERR_NOMEM, ISO_ERR_CUDA,
 ISO_ERR_OVERLAP, ISO_ERR_STATE, ISO_ERR_TIMEOUT, ISO_ERR_TOO_LARGE) = range(11)
ISO_STATIC_SCRATCH_BYTES = 8 << 20

LIB_NAME = "libiso_b200.so"
LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), LIB_NAME)

# every symbol include/iso.h declares
EXPORTS = (
    "Iso_neighborhood_create", "Iso_comm_free", "Iso_comm_set_periodic",
    "Iso_neighbor_alltoall_init", "Iso_neighbor_allgather_init", "Iso_neighbor_alltoallv_init",
    "Iso_neighbor_allgatherv_init", "Iso_request_set_algorithm", "Iso_request_set_layout", "Iso_request_set_single_launch", "Iso_request_set_slabs", "Iso_request_set_pipeline", "Iso_request_set_chains", "Iso_request_set_graph", "Iso_request_tune", "Iso_request_get_execution", "Iso_request_set_bulk_threshold",
    "Iso_request_set_hybrid", "Iso_request_set_sender_side", "Iso_request_set_dimension_order", "Iso_request_get_dimension_order", "Iso_request_check_guards", "Iso_request_get_host_transfer_ms", "Iso_request_set_wait_limit", "Iso_request_test_skew_arrivals", "Iso_measure_launch_floor",
    "Iso_Start", "Iso_Start_host", "Iso_wait", "Iso_request_get_stats", "Iso_request_get_parts",
    "Iso_neighbor_alltoall_static", "Iso_request_free", "Iso_error_string", "Iso_last_cuda_error", "Iso_selftest",
)


class IsoError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__("%s failed: %s (code %d, cuda error %d)" %
                         (where, Iso_error_string(code), code, Iso_last_cuda_error()))


class Iso_stats(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in
                ("kind", "algorithm", "fusion_level", "d", "s", "rounds", "max_rounds_per_dim", "phases",
                 "launches", "parts", "local_copies")] + \
               [(n, ctypes.c_int64) for n in
                ("P", "send_stride", "recv_stride", "inter_stride", "bytes_min", "bytes_moved", "bulk_bytes")]

    def as_dict(self) -> dict:
        return {n: int(getattr(self, n)) for n, _ in self._fields_}


class Iso_part(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in
                ("phase", "round", "slot", "src_buf", "dst_buf", "kernel", "width", "reserved")] + \
               [(n, ctypes.c_int64) for n in ("src_off", "dst_off", "len")] + \
               [("shift", ctypes.c_int * ISO_MAX_DIMS), ("check", ctypes.c_int * ISO_MAX_DIMS)]

    def as_dict(self) -> dict:
        d = {n: int(getattr(self, n)) for n, _ in self._fields_ if n not in ("shift", "check", "reserved")}
        d["shift"] = list(self.shift)
        d["check"] = list(self.check)
        return d


_lib = None


def load_library() -> ctypes.CDLL:
    """Loads libiso_b200.so from the package directory; raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(
            "%s is missing: build it with `python -m paper_1606_07676_b200.build` "
            "(there is no fallback implementation)" % LIB_PATH)
    lib = ctypes.CDLL(LIB_PATH)
    vp, ci, i64 = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64
    pp = ctypes.POINTER(vp)
    sig = {
        "Iso_neighborhood_create": [ci, vp, ci, vp, pp],
        "Iso_comm_free": [pp],
        "Iso_comm_set_periodic": [vp, vp],
        "Iso_neighbor_alltoall_init": [vp, ci, ci, vp, ci, ci, vp, pp],
        "Iso_neighbor_allgather_init": [vp, ci, ci, vp, ci, ci, vp, pp],
        "Iso_neighbor_alltoallv_init": [vp, vp, vp, ci, vp, vp, vp, ci, vp, pp],
        "Iso_neighbor_allgatherv_init": [vp, ci, ci, vp, vp, vp, ci, vp, pp],
        "Iso_request_set_algorithm": [vp, ci, ci],
        "Iso_request_set_layout": [vp, ci],
        "Iso_request_set_single_launch": [vp, ci],
        "Iso_request_set_slabs": [vp, ci],
        "Iso_request_set_pipeline": [vp, ci],
        "Iso_request_set_chains": [vp, ci],
        "Iso_request_set_graph": [vp, ci],
        "Iso_request_tune": [vp, vp, ci],
        "Iso_request_get_execution": [vp, ctypes.POINTER(ci), ctypes.POINTER(ci), ctypes.POINTER(ci)],
        "Iso_request_set_bulk_threshold": [vp, i64],
        "Iso_request_set_hybrid": [vp, ci],
        "Iso_request_set_sender_side": [vp, ci],
        "Iso_request_set_dimension_order": [vp, ctypes.POINTER(ci)],
        "Iso_request_get_dimension_order": [vp, ctypes.POINTER(ci)],
        "Iso_request_check_guards": [vp, ctypes.POINTER(i64)],
        "Iso_request_get_host_transfer_ms": [vp, ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_float),
                                             ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ci)],
        "Iso_request_set_wait_limit": [vp, ctypes.c_uint],
        "Iso_request_test_skew_arrivals": [vp, ci],
        "Iso_measure_launch_floor": [vp, ci, ci, ctypes.POINTER(ctypes.c_float)],
        "Iso_Start": [vp, vp],
        "Iso_Start_host": [vp, vp, vp, vp],
        "Iso_wait": [vp],
        "Iso_request_get_stats": [vp, ctypes.POINTER(Iso_stats)],
        "Iso_request_get_parts": [vp, ctypes.POINTER(Iso_part), ci, ctypes.POINTER(ci)],
        "Iso_neighbor_alltoall_static": [ci, vp, ci, vp, vp, vp, ci, ci, vp],
        "Iso_request_free": [pp],
        "Iso_last_cuda_error": [],
        "Iso_selftest": [],
    }
    for name, args in sig.items():
        f = getattr(lib, name)
        f.argtypes = args
        f.restype = ci
    lib.Iso_error_string.argtypes = [ci]
    lib.Iso_error_string.restype = ctypes.c_char_p
    _lib = lib
    return lib


# ------------------------------------------------------------------------ marshalling
def _addr(buf) -> int:
    """Address of a device tensor / pinned host tensor / numpy array / raw integer."""
    if buf is None:
        return 0
    if isinstance(buf, int):
        return buf
    if hasattr(buf, "data_ptr"):
        return int(buf.data_ptr())
    if isinstance(buf, np.ndarray):
        return int(buf.ctypes.data)
    raise TypeError("cannot take the address of %r" % type(buf))


def _stream(stream) -> int:
    if stream is None:
        return 0
    if isinstance(stream, int):
        return stream
    return int(stream.cuda_stream)


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32).reshape(-1))


def _i64(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.int64).reshape(-1))


def _check(code: int, where: str) -> None:
    if code != ISO_SUCCESS:
        raise IsoError(code, where)


# --------------------------------------------------------------------- the entry points
def Iso_error_string(code: int) -> str:
    return load_library().Iso_error_string(int(code)).decode()


def Iso_last_cuda_error() -> int:
    return int(load_library().Iso_last_cuda_error())


def Iso_selftest() -> None:
    _check(load_library().Iso_selftest(), "Iso_selftest")


def Iso_neighborhood_create(dims, relative_coordinates) -> int:
    """dims: d torus sizes; relative_coordinates: [s, d] integers.  Returns the comm handle."""
    lib = load_library()
    dims = _i32(dims)
    coords = _i32(relative_coordinates)
    d = int(dims.size)
    if d == 0 or coords.size % d:
        raise ValueError("relative_coordinates must hold s*d integers")
    comm = ctypes.c_void_p()
    _check(lib.Iso_neighborhood_create(d, dims.ctypes.data, coords.size // d, coords.ctypes.data,
                                       ctypes.byref(comm)), "Iso_neighborhood_create")
    return comm.value


def Iso_comm_set_periodic(comm: int, periodic) -> None:
    p = _i32(periodic)
    _check(load_library().Iso_comm_set_periodic(comm, p.ctypes.data), "Iso_comm_set_periodic")


def Iso_comm_free(comm: int) -> None:
    h = ctypes.c_void_p(comm)
    _check(load_library().Iso_comm_free(ctypes.byref(h)), "Iso_comm_free")


def Iso_neighbor_alltoall_init(sendbuf, sendcount: int, sendtype: int, recvbuf, recvcount: int,
                               recvtype: int, comm: int) -> int:
    req = ctypes.c_void_p()
    _check(load_library().Iso_neighbor_alltoall_init(_addr(sendbuf), sendcount, sendtype, _addr(recvbuf),
                                                     recvcount, recvtype, comm, ctypes.byref(req)),
           "Iso_neighbor_alltoall_init")
    return req.value


def Iso_neighbor_allgather_init(sendbuf, sendcount: int, sendtype: int, recvbuf, recvcount: int,
                                recvtype: int, comm: int) -> int:
    req = ctypes.c_void_p()
    _check(load_library().Iso_neighbor_allgather_init(_addr(sendbuf), sendcount, sendtype, _addr(recvbuf),
                                                      recvcount, recvtype, comm, ctypes.byref(req)),
           "Iso_neighbor_allgather_init")
    return req.value


def Iso_neighbor_alltoallv_init(sendbuf, sendcounts, senddispls, sendtype: int, recvbuf, recvcounts,
                                recvdispls, recvtype: int, comm: int) -> int:
    sc, sd, rc, rd = _i32(sendcounts), _i64(senddispls), _i32(recvcounts), _i64(recvdispls)
    req = ctypes.c_void_p()
    _check(load_library().Iso_neighbor_alltoallv_init(_addr(sendbuf), sc.ctypes.data, sd.ctypes.data, sendtype,
                                                      _addr(recvbuf), rc.ctypes.data, rd.ctypes.data, recvtype,
                                                      comm, ctypes.byref(req)),
           "Iso_neighbor_alltoallv_init")
    return req.value


def Iso_neighbor_allgatherv_init(sendbuf, sendcount: int, sendtype: int, recvbuf, recvcounts, recvdispls,
                                 recvtype: int, comm: int) -> int:
    rc, rd = _i32(recvcounts), _i64(recvdispls)
    req = ctypes.c_void_p()
    _check(load_library().Iso_neighbor_allgatherv_init(_addr(sendbuf), sendcount, sendtype, _addr(recvbuf),
                                                       rc.ctypes.data, rd.ctypes.data, recvtype, comm,
                                                       ctypes.byref(req)),
           "Iso_neighbor_allgatherv_init")
    return req.value


def Iso_request_set_algorithm(request: int, alg: int, fusion_level: int = 1) -> None:
    _check(load_library().Iso_request_set_algorithm(request, alg, fusion_level), "Iso_request_set_algorithm")


def Iso_request_set_layout(request: int, layout: int) -> None:
    _check(load_library().Iso_request_set_layout(request, layout), "Iso_request_set_layout")


def Iso_request_set_single_launch(request: int, enable: bool) -> None:
    _check(load_library().Iso_request_set_single_launch(request, 1 if enable else 0), "Iso_request_set_single_launch")


def Iso_request_set_pipeline(request: int, slabs: int) -> None:
    _check(load_library().Iso_request_set_pipeline(request, slabs), "Iso_request_set_pipeline")


def Iso_request_set_slabs(request: int, slabs: int) -> None:
    _check(load_library().Iso_request_set_slabs(request, slabs), "Iso_request_set_slabs")


def Iso_request_set_chains(request: int, chains: int) -> None:
    _check(load_library().Iso_request_set_chains(request, chains), "Iso_request_set_chains")


def Iso_request_set_graph(request: int, enable: bool) -> None:
    _check(load_library().Iso_request_set_graph(request, 1 if enable else 0), "Iso_request_set_graph")


ISO_TUNE_COLD, ISO_TUNE_SCHEDULE = 1, 2


def Iso_request_tune(request: int, cuda_stream=None, cold: bool = False, schedule: bool = False) -> dict:
    """Times the execution variants (and, with `schedule`, the schedules) on the device and
    keeps the fastest; returns the execution plan."""
    flags = (ISO_TUNE_COLD if cold else 0) | (ISO_TUNE_SCHEDULE if schedule else 0)
    _check(load_library().Iso_request_tune(request, _stream(cuda_stream), flags), "Iso_request_tune")
    return Iso_request_get_execution(request)


def Iso_request_get_execution(request: int) -> dict:
    slabs, chains, graph = ctypes.c_int(0), ctypes.c_int(0), ctypes.c_int(0)
    _check(load_library().Iso_request_get_execution(request, ctypes.byref(slabs), ctypes.byref(chains),
                                                    ctypes.byref(graph)), "Iso_request_get_execution")
    return {"slabs": slabs.value, "chains": chains.value, "graph": graph.value}


def Iso_request_set_bulk_threshold(request: int, nbytes: int) -> None:
    _check(load_library().Iso_request_set_bulk_threshold(request, nbytes), "Iso_request_set_bulk_threshold")


def Iso_request_get_host_transfer_ms(request: int) -> dict:
    """Link-busy times of the last pipelined Iso_Start_host (milliseconds) and its slab count."""
    up, down, total, slabs = ctypes.c_float(0), ctypes.c_float(0), ctypes.c_float(0), ctypes.c_int(0)
    _check(load_library().Iso_request_get_host_transfer_ms(request, ctypes.byref(up), ctypes.byref(down),
                                                           ctypes.byref(total), ctypes.byref(slabs)),
           "Iso_request_get_host_transfer_ms")
    return {"upload_ms": up.value, "download_ms": down.value, "total_ms": total.value, "slabs": slabs.value}


def Iso_request_set_hybrid(request: int, enable: bool) -> None:
    _check(load_library().Iso_request_set_hybrid(request, 1 if enable else 0), "Iso_request_set_hybrid")


def Iso_request_set_sender_side(request: int, mode: int) -> None:
    _check(load_library().Iso_request_set_sender_side(request, mode), "Iso_request_set_sender_side")


def Iso_request_set_dimension_order(request: int, order) -> None:
    arr = (ctypes.c_int * len(order))(*[int(x) for x in order])
    _check(load_library().Iso_request_set_dimension_order(request, arr), "Iso_request_set_dimension_order")


def Iso_request_get_dimension_order(request: int, d: int):
    arr = (ctypes.c_int * d)()
    _check(load_library().Iso_request_get_dimension_order(request, arr), "Iso_request_get_dimension_order")
    return [int(x) for x in arr]


def Iso_request_check_guards(request: int) -> int:
    """Bytes of the guard bands around the intermediate buffer that were overwritten."""
    bad = ctypes.c_int64(-1)
    _check(load_library().Iso_request_check_guards(request, ctypes.byref(bad)), "Iso_request_check_guards")
    return int(bad.value)


def Iso_request_set_wait_limit(request: int, polls: int) -> None:
    _check(load_library().Iso_request_set_wait_limit(request, polls), "Iso_request_set_wait_limit")


def Iso_request_test_skew_arrivals(request: int, extra: int) -> None:
    _check(load_library().Iso_request_test_skew_arrivals(request, extra), "Iso_request_test_skew_arrivals")


def Iso_measure_launch_floor(stream=None, launches: int = 1000, dependent: bool = True) -> float:
    """Device time per launch of an empty kernel, in microseconds."""
    us = ctypes.c_float(0.0)
    _check(load_library().Iso_measure_launch_floor(_stream(stream), launches, 1 if dependent else 0,
                                                   ctypes.byref(us)), "Iso_measure_launch_floor")
    return float(us.value)


def Iso_Start(request: int, stream=None) -> None:
    _check(load_library().Iso_Start(request, _stream(stream)), "Iso_Start")


def Iso_Start_host(request: int, host_sendbuf, host_recvbuf, stream=None) -> None:
    _check(load_library().Iso_Start_host(request, _addr(host_sendbuf), _addr(host_recvbuf), _stream(stream)),
           "Iso_Start_host")


def Iso_wait(request: int) -> None:
    _check(load_library().Iso_wait(request), "Iso_wait")


def Iso_request_get_stats(request: int) -> dict:
    st = Iso_stats()
    _check(load_library().Iso_request_get_stats(request, ctypes.byref(st)), "Iso_request_get_stats")
    return st.as_dict()


def Iso_request_get_parts(request: int) -> list:
    lib = load_library()
    n = ctypes.c_int(0)
    _check(lib.Iso_request_get_parts(request, None, 0, ctypes.byref(n)), "Iso_request_get_parts")
    arr = (Iso_part * max(1, n.value))()
    _check(lib.Iso_request_get_parts(request, arr, n.value, ctypes.byref(n)), "Iso_request_get_parts")
    return [arr[k].as_dict() for k in range(n.value)]


def Iso_neighbor_alltoall_static(dims, relative_coordinates, sendbuf, recvbuf, count: int, datatype: int,
                                 stream=None) -> None:
    """All-to-all through the entry point that allocates no device memory: tables and
    intermediate buffer live in the library's fixed scratch array (see include/iso.h)."""
    dims = _i32(dims)
    coords = _i32(relative_coordinates)
    d = int(dims.size)
    if d == 0 or coords.size % d:
        raise ValueError("relative_coordinates must hold s*d integers")
    _check(load_library().Iso_neighbor_alltoall_static(d, dims.ctypes.data, coords.size // d, coords.ctypes.data,
                                                       _addr(sendbuf), _addr(recvbuf), count, datatype,
                                                       _stream(stream)), "Iso_neighbor_alltoall_static")


def Iso_request_free(request: int) -> None:
    h = ctypes.c_void_p(request)
    _check(load_library().Iso_request_free(ctypes.byref(h)), "Iso_request_free")
