"""Failure detection and race detection on the device, without faulting it: a bounded wait
that is made to run out, guard bands around every buffer a schedule touches, and the
library driven from a plain C program."""
import os
import subprocess

import numpy as np
import pytest

from paper_1606_07676_b200 import binding as iso
from paper_1606_07676_b200 import workloads as wl
from schedule_sim import POISON, layout, make_request, oracle_result, send_buffer_np

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def torch_cuda():
    import torch
    if not torch.cuda.is_available():
        pytest.fail("these tests need a CUDA device")
    iso.load_library()
    torch.cuda.set_device(0)
    return torch


@pytest.mark.parametrize("mode", ["grid_barrier", "item_counters"])
def test_a_bounded_wait_runs_out_and_the_request_recovers(torch_cuda, mode):
    """The one-launch modes make thread blocks wait for each other.  Here the next start is
    told to expect one arrival more than there are thread blocks, with a poll limit of 2^10:
    the first wait cannot be met, every block gives up after about 50 microseconds, the
    kernel returns by itself and Iso_wait says ISO_ERR_TIMEOUT.  The request is then usable
    again: the following ordinary starts give the oracle's bytes."""
    torch = torch_cuda
    w = wl.Workload("t", "alltoall", (16, 16, 8), wl.moore(3, 1), 64, kind="fp32", seed=23)
    lens, sd, rd, ss, rs = layout(w)
    send_h = send_buffer_np(w, ss)
    send = torch.from_numpy(send_h).cuda()
    recv = torch.full((w.P, rs), POISON, dtype=torch.uint8, device="cuda")
    comm, req = make_request(w, send, recv)
    want = oracle_result(w, send_h)
    try:
        if mode == "grid_barrier":
            iso.Iso_request_set_single_launch(req, True)
        else:
            iso.Iso_request_set_pipeline(req, 2)
        iso.Iso_Start(req)
        iso.Iso_wait(req)
        assert iso.Iso_request_get_stats(req)["launches"] == 1      # the mode is in use
        assert np.array_equal(recv.cpu().numpy(), want)
        for _ in range(2):
            iso.Iso_request_set_wait_limit(req, 1 << 10)
            iso.Iso_request_test_skew_arrivals(req, 1)
            recv.fill_(POISON)
            iso.Iso_Start(req)
            with pytest.raises(iso.IsoError) as e:
                iso.Iso_wait(req)
            assert e.value.code == iso.ISO_ERR_TIMEOUT
            assert not np.array_equal(recv.cpu().numpy(), want)      # later phases never ran
            iso.Iso_wait(req)                                         # the error was consumed
            iso.Iso_request_set_wait_limit(req, 1 << 22)
            for _ in range(2):                                        # counters start afresh
                recv.fill_(POISON)
                iso.Iso_Start(req)
                iso.Iso_wait(req)
                assert np.array_equal(recv.cpu().numpy(), want)
        assert iso.Iso_request_check_guards(req) == 0
    finally:
        iso.Iso_request_free(req)
        iso.Iso_comm_free(comm)


BAND = 4096


def _banded(torch, nbytes, fill):
    """A device buffer of `nbytes` with a band of 0xC3 bytes before and after it."""
    whole = torch.full((nbytes + 2 * BAND,), 0xC3, dtype=torch.uint8, device="cuda")
    inner = whole[BAND:BAND + nbytes]
    inner.fill_(fill)
    return whole, inner


def _bands_intact(whole, nbytes):
    return bool((whole[:BAND] == 0xC3).all()) and bool((whole[BAND + nbytes:] == 0xC3).all())


@pytest.mark.parametrize("name", ["cfg2_alltoall", "cfg2_allgather", "cfg5_32x32x32", "cfg4", "ragged", "bulk"])
def test_no_schedule_writes_outside_its_buffers(torch_cuda, name):
    """Canary bands before and after the send and receive buffers (caller side) and around
    the library's intermediate buffer: untouched after every schedule and execution plan,
    while the result is the oracle's."""
    torch = torch_cuda
    if name == "ragged":
        w = wl.Workload("ragged", "alltoallv", (37, 53), wl.moore(2, 1), 0,
                        lens=np.array([1024, 4, 2064, 16, 1040, 8, 3072, 64]), seed=8)
    elif name == "bulk":
        w = wl.Workload("bulk", "alltoall", (24, 20), wl.moore(2, 2), 2048, seed=9)
    else:
        w = wl.config(name)
    lens, sd, rd, ss, rs = layout(w)
    send_h = send_buffer_np(w, ss)
    send_whole, send = _banded(torch, w.P * ss, 0)
    send.copy_(torch.from_numpy(send_h).reshape(-1))
    recv_whole, recv = _banded(torch, w.P * rs, POISON)
    comm, req = make_request(w, send, recv)
    want = oracle_result(w, send_h)
    plans = [dict(alg=iso.ISO_ALG_COMBINING, fusion=1), dict(alg=iso.ISO_ALG_COMBINING, fusion=0),
             dict(alg=iso.ISO_ALG_COMBINING, fusion=2), dict(alg=iso.ISO_ALG_DIRECT, fusion=1),
             dict(alg=iso.ISO_ALG_COMBINING, fusion=1, slabs=4), dict(alg=iso.ISO_ALG_COMBINING, fusion=1, slabs=8, chains=2),
             dict(alg=iso.ISO_ALG_COMBINING, fusion=1, single=True), dict(alg=iso.ISO_ALG_COMBINING, fusion=1, pipeline=3)]
    if w.collective != "allgather":
        plans.append(dict(alg=iso.ISO_ALG_TORUS, fusion=1))
    try:
        for plan in plans:
            iso.Iso_request_set_single_launch(req, plan.get("single", False))
            iso.Iso_request_set_pipeline(req, plan.get("pipeline", 0))
            iso.Iso_request_set_slabs(req, plan.get("slabs", 0))
            iso.Iso_request_set_chains(req, plan.get("chains", 1))
            iso.Iso_request_set_algorithm(req, plan["alg"], plan["fusion"])
            recv.fill_(POISON)
            iso.Iso_Start(req)
            iso.Iso_wait(req)
            assert np.array_equal(recv.cpu().numpy().reshape(want.shape), want), (name, plan)
            assert iso.Iso_request_check_guards(req) == 0, (name, plan)
            assert _bands_intact(send_whole, w.P * ss) and _bands_intact(recv_whole, w.P * rs), (name, plan)
        assert np.array_equal(send.cpu().numpy().reshape(send_h.shape), send_h)     # the send buffer is never written
    finally:
        iso.Iso_request_free(req)
        iso.Iso_comm_free(comm)


def test_plain_c_program_runs_a_collective_on_the_device(torch_cuda, tmp_path):
    """tests/c_abi_gpu.c: cudaMalloc'd buffers, Iso_Start and Iso_wait from C, compared with
    the hand-worked rows of the 4x4 example."""
    exe = tmp_path / "c_abi_gpu"
    libdir = os.path.dirname(iso.LIB_PATH)
    cuda = os.environ.get("CUDA_HOME", "/usr/local/cuda")
    subprocess.check_call(["gcc", "-std=c99", "-Wall", "-Werror", "-I", os.path.join(ROOT, "include"),
                           "-I", os.path.join(cuda, "include"), os.path.join(ROOT, "tests", "c_abi_gpu.c"),
                           "-o", str(exe), "-L", libdir, "-l:" + iso.LIB_NAME, "-L", os.path.join(cuda, "lib64"),
                           "-lcudart", "-Wl,-rpath," + libdir, "-Wl,-rpath," + os.path.join(cuda, "lib64")])
    out = subprocess.run([str(exe)], capture_output=True, text=True, timeout=300)
    assert out.returncode == 0 and "c abi gpu ok" in out.stdout, out.stdout + out.stderr
