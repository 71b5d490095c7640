"""GPU parity: the CUDA library, called through its C-ABI binding, against the CPU oracle,
bit for bit, on the same seeded inputs."""
import numpy as np
import pytest

import oracle
from oracle import counters
from paper_1606_07676_b200 import binding as iso
from paper_1606_07676_b200 import workloads as wl
from schedule_sim import POISON, layout, make_request, oracle_result, send_buffer_np

pytestmark = pytest.mark.gpu

COMB0, COMB1, COMB2, COMBD = ((iso.ISO_ALG_COMBINING, g) for g in (0, 1, 2, 8))
ALT0, ALT1 = ((iso.ISO_ALG_COMBINING, 100 + g) for g in (0, 1))   # Algorithm 1's alternating layout
DIRECT = (iso.ISO_ALG_DIRECT, 1)
TORUS = (iso.ISO_ALG_TORUS, 1)


@pytest.fixture(scope="module")
def torch_cuda():
    import torch
    if not torch.cuda.is_available():
        pytest.fail("these tests need a CUDA device")
    iso.load_library()          # no fallback: a missing library is an error
    torch.cuda.set_device(0)
    return torch


class Run:
    """A workload bound to device buffers; `result(alg, fusion)` runs it and returns the
    receive buffers as a numpy array."""

    def __init__(self, torch, w, stream=None, periodic=None):
        self.torch, self.w = torch, w
        self.periodic = periodic
        lens, sd, rd, ss, rs = layout(w)
        self.ss, self.rs = ss, rs
        self.send_host = send_buffer_np(w, ss)
        self.send = torch.from_numpy(self.send_host).cuda()
        self.recv = torch.empty((w.P, rs), dtype=torch.uint8, device="cuda")
        self.comm, self.req = make_request(w, self.send, self.recv, periodic)
        self.stream = stream
        st = iso.Iso_request_get_stats(self.req)
        assert (st["send_stride"], st["recv_stride"]) == (ss, rs)

    def result(self, alg, fusion, bulk=None, single=False):
        iso.Iso_request_set_single_launch(self.req, single)
        if fusion >= 100:
            iso.Iso_request_set_layout(self.req, iso.ISO_LAYOUT_ALTERNATING)
            fusion -= 100
        else:
            iso.Iso_request_set_layout(self.req, iso.ISO_LAYOUT_PACKED)
        iso.Iso_request_set_algorithm(self.req, alg, fusion)
        if bulk is not None:
            iso.Iso_request_set_bulk_threshold(self.req, bulk)
        self.recv.fill_(POISON)
        self.torch.cuda.synchronize()
        iso.Iso_Start(self.req, self.stream)
        iso.Iso_wait(self.req)
        return self.recv.cpu().numpy()

    def close(self):
        iso.Iso_request_free(self.req)
        iso.Iso_comm_free(self.comm)


def check(torch, w, algs, bulk=None, single=False):
    run = Run(torch, w)
    try:
        want = oracle_result(w, run.send_host)
        for alg, fusion in algs:
            got = run.result(alg, fusion, bulk, single)
            bad = np.argwhere(got != want)
            assert bad.size == 0, "alg %d fusion %d: first mismatch at (rank, byte) %s" % (alg, fusion, bad[0])
    finally:
        run.close()


# ------------------------------------------------------------------- the five configs
def test_cfg1(torch_cuda):
    check(torch_cuda, wl.config("cfg1"), [COMB0, COMB1, COMB2, ALT0, ALT1, DIRECT, TORUS])


def test_cfg2_alltoall(torch_cuda):
    check(torch_cuda, wl.config("cfg2_alltoall"), [COMB0, COMB1, COMB2, COMBD, ALT0, ALT1, DIRECT, TORUS])


def test_all_phases_in_one_cooperative_launch(torch_cuda):
    # opt-in execution mode: one cooperative launch with grid barriers between the phases
    check(torch_cuda, wl.config("cfg2_alltoall"), [COMB0, COMB1, COMB2, ALT1, TORUS], single=True)
    check(torch_cuda, wl.config("cfg2_allgather"), [COMB0, COMB1], single=True)
    check(torch_cuda, wl.config("cfg3_m64"), [COMB0, COMB1, TORUS], single=True)
    check(torch_cuda, wl.config("cfg4"), [COMB1], single=True)
    check(torch_cuda, wl.Workload("ragged", "alltoall", (37, 53), wl.moore(2, 2), 48, seed=7), [COMB0, COMB1], single=True)
    run = Run(torch_cuda, wl.config("cfg2_alltoall"))
    run.result(*COMB1, single=True)
    assert iso.Iso_request_get_stats(run.req)["launches"] == 1
    run.result(*COMB1, single=False)
    assert iso.Iso_request_get_stats(run.req)["launches"] == 3
    run.close()


def test_slab_execution(torch_cuda):
    """Slab after slab along dimension 0 with a one-slab intermediate buffer: same result for
    any slab count, and the intermediate buffer shrinks accordingly."""
    torch = torch_cuda
    for name, algs in [("cfg2_alltoall", [COMB1, COMB0, COMB2, ALT1, DIRECT]), ("cfg3_m64", [COMB1]),
                       ("cfg2_allgather", [COMB1]), ("octant_d3r3_allgather", [COMB1])]:
        w = wl.config(name)
        run = Run(torch, w)
        want = oracle_result(w, run.send_host)
        for slabs in (2, 5, 32, 1, 0):
            iso.Iso_request_set_slabs(run.req, slabs)
            for alg, fusion in algs:
                got = run.result(alg, fusion)
                assert np.array_equal(got, want), (name, slabs, alg, fusion)
                if slabs == 5 and (alg, fusion) == COMB1 and w.collective == "alltoall":
                    assert iso.Iso_request_get_stats(run.req)["launches"] % 5 == 0
        run.close()


def test_chains_graph_replay_and_tuning(torch_cuda):
    """Slabs side by side inside a captured graph, plain graph replay, and the measuring
    tuner: the result is the oracle's whatever the execution plan, also after the plan is
    changed on a request that has already run, and on repeated starts of one graph."""
    torch = torch_cuda
    for name, algs in [("cfg2_alltoall", [COMB1, COMB0, DIRECT]), ("cfg3_m64", [COMB1]), ("stencil_d3_m16", [COMB1]),
                       ("cfg2_allgather", [COMB1]), ("cfg1", [COMB1, TORUS])]:
        w = wl.config(name)
        run = Run(torch, w)
        want = oracle_result(w, run.send_host)
        for slabs, chains, graph in [(0, 1, True), (4, 2, False), (8, 4, True), (6, 3, True), (2, 1, True), (0, 1, False)]:
            iso.Iso_request_set_slabs(run.req, slabs)
            iso.Iso_request_set_chains(run.req, chains)
            iso.Iso_request_set_graph(run.req, graph)
            for alg, fusion in algs:
                got = run.result(alg, fusion)
                assert np.array_equal(got, want), (name, slabs, chains, graph, alg, fusion)
                ex = iso.Iso_request_get_execution(run.req)
                assert ex["chains"] in (1, chains) and (ex["chains"] == 1 or ex["graph"] == 1)
                if graph:
                    assert ex["graph"] == 1
                    # the same graph again, on poisoned receive buffers
                    run.recv.fill_(0xA5)
                    iso.Iso_Start(run.req, torch.cuda.current_stream())
                    iso.Iso_wait(run.req)
                    assert np.array_equal(run.recv.cpu().numpy().reshape(want.shape), want), (name, "replay")
        for cold in (False, True):
            chosen = iso.Iso_request_tune(run.req, torch.cuda.current_stream(), cold)
            assert chosen["slabs"] >= 1 and chosen["chains"] in (1, 2, 4) and chosen["graph"] in (0, 1)
            run.recv.fill_(0xA5)
            iso.Iso_Start(run.req, torch.cuda.current_stream())
            iso.Iso_wait(run.req)
            assert np.array_equal(run.recv.cpu().numpy().reshape(want.shape), want), (name, "tuned", chosen)
            assert iso.Iso_request_get_execution(run.req) == chosen
        # the tuner may choose the schedule as well: whatever it keeps gives the oracle's bytes
        chosen = iso.Iso_request_tune(run.req, torch.cuda.current_stream(), cold=False, schedule=True)
        st = iso.Iso_request_get_stats(run.req)
        assert (st["algorithm"], st["fusion_level"]) in [(iso.ISO_ALG_COMBINING, 1), (iso.ISO_ALG_COMBINING, 2), (iso.ISO_ALG_DIRECT, 1)]
        run.recv.fill_(0xA5)
        iso.Iso_Start(run.req, torch.cuda.current_stream())
        iso.Iso_wait(run.req)
        assert np.array_equal(run.recv.cpu().numpy().reshape(want.shape), want), (name, "tuned schedule", chosen, st["algorithm"])
        run.close()


def test_pipelined_one_launch_execution(torch_cuda):
    """One cooperative launch over (slab, launch) items with per-item completion counters:
    the oracle's result for any slab count, on repeated starts (the counters carry over),
    for schedules with compact descriptors (cfg4) and wide rows (342 neighbours), and the
    plain execution again after it is switched off."""
    torch = torch_cuda
    for name, algs in [("cfg2_alltoall", [COMB1, COMB0, COMB2, ALT1, DIRECT, TORUS]), ("cfg3_m64", [COMB1, TORUS]),
                       ("cfg4", [COMB1]), ("cfg2_allgather", [COMB1, COMB0]), ("moore_d3r3_alltoall", [COMB1]),
                       ("cfg1", [COMB1])]:
        w = wl.config(name)
        run = Run(torch, w)
        want = oracle_result(w, run.send_host)
        for slabs in (1, 2, 3, 8, 5, 0):
            iso.Iso_request_set_pipeline(run.req, slabs)
            for alg, fusion in algs:
                got = run.result(alg, fusion)
                assert np.array_equal(got, want), (name, slabs, alg, fusion)
                st = iso.Iso_request_get_stats(run.req)
                if slabs > 0 and w.block_bytes % 16 == 0:   # cfg1's 8-byte blocks run as if it were off
                    assert st["launches"] == 1, (name, slabs, st["launches"])
                for _ in range(2):   # again, on poisoned receive buffers
                    run.recv.fill_(0xA5)
                    iso.Iso_Start(run.req, torch.cuda.current_stream())
                iso.Iso_wait(run.req)
                assert np.array_equal(run.recv.cpu().numpy().reshape(want.shape), want), (name, slabs, "restart")
        run.close()
    # ragged sizes; a schedule the mode cannot take (4-byte units) runs as if it were off
    w = wl.Workload("ragged", "alltoall", (37, 53), wl.moore(2, 2), 48, seed=7)
    run = Run(torch, w)
    want = oracle_result(w, run.send_host)
    for slabs in (1, 4, 37):
        iso.Iso_request_set_pipeline(run.req, slabs)
        assert np.array_equal(run.result(*COMB1), want), slabs
    run.close()
    w = wl.config("cfg5")
    run = Run(torch, w)
    iso.Iso_request_set_pipeline(run.req, 4)
    got = run.result(*COMB1)
    assert iso.Iso_request_get_stats(run.req)["launches"] > 1
    assert np.array_equal(got, oracle_result(w, run.send_host))
    run.close()


def test_narrow_cta_shapes(torch_cuda, monkeypatch):
    """16-byte and mixed-width launches run in CTAs of up to 1024 threads by default; the shapes of
    256 and 512 threads (ISO_VEC_THREADS) stay available and must give the same bytes."""
    for threads in ("256", "512"):
        monkeypatch.setenv("ISO_VEC_THREADS", threads)
        check(torch_cuda, wl.config("cfg2_alltoall"), [COMB1, COMB0, DIRECT])
        check(torch_cuda, wl.config("cfg4"), [COMB1])
        check(torch_cuda, wl.config("cfg5_32x32x32"), [COMB1, DIRECT])
        check(torch_cuda, wl.config("cfg2_allgather"), [COMB1])
        check(torch_cuda, wl.Workload("ragged", "alltoall", (37, 53), wl.moore(2, 2), 48, seed=7), [COMB1])


def test_cfg2_allgather(torch_cuda):
    check(torch_cuda, wl.config("cfg2_allgather"), [COMB0, COMB1, COMB2, COMBD, DIRECT])


def test_allgather_phases_in_sender_side_form(torch_cuda):
    """Allgather phases as one load and up to four stores per 16-byte unit (forced on with
    mode 2; left to the library, only large phases take this form): same bytes as the oracle
    on the configuration, the paper's neighbourhoods (blocks with up to fourteen copies, so a
    block is listed several times), tiny and aliasing tori, repeated vectors, the zero vector,
    the irregular allgather, and after switching the form off again."""
    torch = torch_cuda
    cases = [wl.config("cfg2_allgather"), wl.config("octant_d3r3_allgather"), wl.config("moore_d4r1_allgather"),
             wl.Workload("sh", "allgather", (16, 15, 17), wl.shells(3, (3, 7)), 16, seed=3),
             wl.Workload("m33", "allgather", (9, 8, 7), wl.moore(3, 3), 48, seed=4),
             wl.Workload("rag", "allgather", (37, 53), wl.moore(2, 2), 80, seed=5)]
    cases += [w for w in _tiny_cases() if w.collective == "allgather" and w.block_bytes % 16 == 0]
    for w in cases:
        run = Run(torch, w)
        want = oracle_result(w, run.send_host)
        for mode in (2, 0, 1):
            iso.Iso_request_set_sender_side(run.req, mode)
            for alg, fusion in (COMB1, COMB0):
                got = run.result(alg, fusion)
                assert np.array_equal(got, want), (w.name, w.dims, mode, alg, fusion)
                used = {p["kernel"] for p in iso.Iso_request_get_parts(run.req)}
                # (with one launch per round a block has two copies in a launch only if a vector is repeated)
                if mode == 0:
                    assert 2 not in used, (w.name, mode, fusion, used)
                elif mode == 2 and fusion == 1 and w.name != "t":
                    assert 2 in used, (w.name, mode, used)
            assert iso.Iso_request_check_guards(run.req) == 0
        run.close()
    # left to the library, the large phases of the 80-neighbour allgather take this form
    run = Run(torch, wl.config("moore_d4r1_allgather"))
    run.result(*COMB1)
    assert {p["phase"] for p in iso.Iso_request_get_parts(run.req) if p["kernel"] == 2} == {2, 3}
    run.close()


def test_allgather_visiting_orders(torch_cuda):
    """The allgather's trie may visit the dimensions in any order (Section III-B): every order
    gives the oracle's bytes, on the configuration, on a neighbourhood that is not symmetric in
    the dimensions (where the number of parts depends on the order), with intermediate storage,
    on a mesh, in both forms of the phases; the tuner may pick either order."""
    torch = torch_cuda
    lop = np.array([(0, 0, 0), (0, 0, 1), (1, 0, 0), (1, 1, 0), (1, 1, 1), (3, 2, 0), (3, 3, 2), (4, 0, 1), (4, 0, 2),
                    (4, 1, 1), (-2, 5, 1), (1, 1, 1)], np.int32)
    cases = [(wl.config("cfg2_allgather"), None), (wl.Workload("lop", "allgather", (9, 8, 7), lop, 48, seed=8), None),
             (wl.Workload("sh", "allgather", (16, 15, 17), wl.shells(3, (3, 7)), 16, seed=3), None),
             (wl.Workload("mesh", "allgather", (6, 5, 7), wl.moore(3, 1), 32, seed=9), [0, 1, 0]),
             (wl.Workload("d4", "allgather", (5, 4, 6, 3), wl.moore(4, 1), 16, seed=10), None)]
    for w, periodic in cases:
        run = Run(torch, w, periodic=periodic)
        want = oracle_result(w, run.send_host, periodic=periodic)
        d = len(w.dims)
        default = iso.Iso_request_get_dimension_order(run.req, d)
        assert sorted(default) == list(range(d))
        orders = [list(range(d)), list(range(d))[::-1], [1, 0] + list(range(2, d)), list(range(1, d)) + [0]]
        for order in orders:
            iso.Iso_request_set_dimension_order(run.req, order)
            assert iso.Iso_request_get_dimension_order(run.req, d) == order
            for mode in (0, 2):
                iso.Iso_request_set_sender_side(run.req, mode)
                got = run.result(*COMB1)
                assert np.array_equal(got, want), (w.name, order, mode)
            if periodic is None:
                st = iso.Iso_request_get_stats(run.req)
                # one part per non-zero edge of the trie, and one more per repetition of a vector
                repeats = len(w.offsets) - len({tuple(v) for v in w.offsets.tolist()})
                assert st["parts"] == counters.allgather_direct_volume(w.offsets, d, w.dims, order) + repeats
            assert iso.Iso_request_check_guards(run.req) == 0
        run.close()
    run = Run(torch, wl.config("moore_d4r1_allgather"))
    want = oracle_result(run.w, run.send_host)
    assert iso.Iso_request_get_dimension_order(run.req, 4) == [3, 2, 1, 0]
    iso.Iso_request_tune(run.req, None, schedule=True)
    assert sorted(iso.Iso_request_get_dimension_order(run.req, 4)) == [0, 1, 2, 3]
    run.recv.fill_(POISON)
    torch.cuda.synchronize()
    iso.Iso_Start(run.req, None)
    iso.Iso_wait(run.req)
    assert np.array_equal(run.recv.cpu().numpy(), want)
    run.close()
    with pytest.raises(iso.IsoError):
        r2 = Run(torch, wl.config("cfg1"))
        try:
            iso.Iso_request_set_dimension_order(r2.req, [0, 0])
        finally:
            r2.close()


@pytest.mark.parametrize("m", [4, 64, 512])
def test_cfg3(torch_cuda, m):
    check(torch_cuda, wl.config("cfg3_m%d" % m), [COMB0, COMB1, COMBD, ALT1, DIRECT, TORUS])


def test_cfg3_512_both_kernels(torch_cuda):
    # 512-byte blocks go to the bulk-copy kernel by default; here also through the vector
    # kernel (bulk kernel off) and with the threshold at 1 KB
    check(torch_cuda, wl.config("cfg3_m512"), [COMB1, DIRECT], bulk=0)
    check(torch_cuda, wl.config("cfg3_m512"), [COMB1], bulk=1024)


def test_cfg4(torch_cuda):
    check(torch_cuda, wl.config("cfg4"), [COMB0, COMB1, COMB2, ALT1, DIRECT])


def test_cfg5(torch_cuda):
    w = wl.config("cfg5")
    check(torch_cuda, w, [COMB0, COMB1, COMB2, ALT1, DIRECT])
    check(torch_cuda, w, [COMB1], bulk=0)


def test_cfg3_4096_sampled(torch_cuda):
    """Full size (3 x 6.4 GB on the device): outputs of sampled ranks, block by block."""
    torch = torch_cuda
    w = wl.config("cfg3_m4096")
    m, s, P = 4096, w.s, w.P
    stride = s * m
    send = wl.payload_torch(w.kind, w.seed, 0, P * stride, "cuda")
    recv = torch.empty(P * stride, dtype=torch.uint8, device="cuda")
    comm, req = make_request(w, send, recv)
    rng = np.random.default_rng(5)
    ranks = sorted({0, 1, 255, 256, 257, 511, P - 1, P - 256, P - 257, *rng.integers(0, P, 24).tolist()})
    host_send = None
    try:
        # the combining schedule as the library plans it (vector kernel in 128 slabs of two
        # planes, so that a slab's intermediate blocks stay in the L2), the same schedule through
        # the bulk-copy kernel (threshold asked for), and the direct schedule (bulk-copy kernel)
        for alg, fusion, bulk in (COMB1 + (None,), COMB1 + (512,), DIRECT + (None,)):
            if bulk is not None:
                iso.Iso_request_set_bulk_threshold(req, bulk)
            iso.Iso_request_set_algorithm(req, alg, fusion)
            recv.fill_(POISON)
            iso.Iso_Start(req)
            iso.Iso_wait(req)
            st = iso.Iso_request_get_stats(req)
            if alg == iso.ISO_ALG_COMBINING and bulk is None:
                assert st["bulk_bytes"] == 0 and iso.Iso_request_get_execution(req)["slabs"] == 128
            else:
                assert st["bulk_bytes"] == st["bytes_moved"]
            for r in ranks:
                got = recv[r * stride:(r + 1) * stride].cpu().numpy().reshape(s, m)
                for i in range(s):
                    q = oracle.source_rank(w.dims, r, w.offsets[i])
                    want = wl.payload_np(w.kind, w.seed, 0, q * stride + i * m, m)
                    assert np.array_equal(got[i], want), (alg, r, i)
            # whole planes of dimension 0 at both wrap-around edges, from the oracle run on
            # their rank ranges: the host send buffer is reserved in full but only the eight
            # planes those ranks read from (252..255, 0..3) are generated
            if host_send is None:
                host_send = np.empty((P, stride), dtype=np.uint8)
                plane = w.dims[1]
                for x in (252, 253, 254, 255, 0, 1, 2, 3):
                    host_send[x * plane:(x + 1) * plane] = wl.payload_np(
                        w.kind, w.seed, 0, x * plane * stride, plane * stride).reshape(plane, stride)
            for x in (0, 1, 254, 255):
                r0, r1 = x * w.dims[1], (x + 1) * w.dims[1]
                want = oracle.alltoall(w.dims, w.offsets, m, host_send, r0, r1)
                got = recv[r0 * stride:r1 * stride].cpu().numpy().reshape(r1 - r0, stride)
                assert np.array_equal(got, want), (alg, "plane", x)
            # a property that holds at any size: the result is a permutation of the send
            # blocks, so per-slot byte sums over all processes are preserved
            a = send.view(P, s, m)[:, 3].to(torch.int64).sum().item()
            b = recv.view(P, s, m)[:, 3].to(torch.int64).sum().item()
            assert a == b
    finally:
        iso.Iso_request_free(req)
        iso.Iso_comm_free(comm)
        del send, recv
        torch.cuda.empty_cache()


def _sampled_check(torch, w, algs, nranks=12):
    """Full-size run with device-generated inputs; the outputs of sampled ranks are checked
    block by block against sources named by the oracle and regenerated on the host."""
    lens, sd, rd, ss, rs = layout(w)
    m, s, P = w.block_bytes, w.s, w.P
    send = wl.payload_torch(w.kind, w.seed, 0, P * ss, "cuda")
    recv = torch.empty(P * rs, dtype=torch.uint8, device="cuda")
    comm, req = make_request(w, send, recv)
    rng = np.random.default_rng(17)
    ranks = sorted({0, 1, P - 1, w.dims[-1] - 1, w.dims[-1], *rng.integers(0, P, nranks).tolist()})
    try:
        for alg, fusion in algs:
            iso.Iso_request_set_algorithm(req, alg, fusion)
            recv.fill_(POISON)
            iso.Iso_Start(req)
            iso.Iso_wait(req)
            for r in ranks:
                got = recv[r * rs:(r + 1) * rs].cpu().numpy().reshape(s, m)
                for i in range(s):
                    q = oracle.source_rank(w.dims, r, w.offsets[i])
                    off = q * ss + (i * m if w.collective == "alltoall" else 0)
                    assert np.array_equal(got[i], wl.payload_np(w.kind, w.seed, 0, off, m)), (w.name, alg, r, i)
    finally:
        iso.Iso_request_free(req)
        iso.Iso_comm_free(comm)
        del send, recv
        torch.cuda.empty_cache()


@pytest.mark.parametrize("name", ["shells_d3_alltoall", "shells_d3_allgather", "moore_d4r1_alltoall",
                                  "octant_d3r3_allgather", "moore_d3r3_alltoall"])
def test_paper_neighbourhoods_full_size_sampled(torch_cuda, name):
    w = wl.config(name)
    _sampled_check(torch_cuda, w, [COMB1, DIRECT] if w.s < 1000 else [COMB1])


# --------------------------------------------------------------------- edge cases
def _tiny_cases():
    rng = np.random.default_rng(99)
    cases = []
    for dims in [(1,), (2,), (7,), (3, 5), (2, 2, 3), (5, 1, 4), (3, 3, 3, 2)]:
        d = len(dims)
        for s in (1, 5, 11):
            offs = rng.integers(-6, 7, size=(s, d)).astype(np.int32)
            if s >= 5:
                offs[1] = 0
                offs[4] = offs[2]
            cases.append(wl.Workload("t", "alltoall", dims, offs, int(rng.choice([1, 2, 4, 8, 12, 16, 48])), seed=len(cases)))
            cases.append(wl.Workload("t", "allgather", dims, offs, int(rng.choice([1, 4, 16, 80])), seed=len(cases)))
            lens = rng.choice([0, 1, 3, 4, 16, 52, 64, 100, 1024, 1040], size=s).astype(np.int64)
            cases.append(wl.Workload("t", "alltoallv", dims, offs, 0, lens=lens, seed=len(cases)))
    return cases


def test_tiny_tori_and_odd_sizes(torch_cuda):
    for w in _tiny_cases():
        algs = [COMB0, COMB1, COMB2, ALT1, DIRECT] + ([TORUS] if w.collective != "allgather" else [])
        check(torch_cuda, w, algs)


def test_ragged_tail_and_many_tiles(torch_cuda):
    # P is not a multiple of any tile size; several CTAs and a partial last one
    w = wl.Workload("ragged", "alltoall", (37, 53), wl.moore(2, 2), 48, seed=7)
    check(torch_cuda, w, [COMB0, COMB1, DIRECT, TORUS])
    w = wl.Workload("ragged", "alltoallv", (37, 53), wl.moore(2, 1), 0,
                    lens=np.array([1024, 4, 2064, 16, 1040, 8, 3072, 64]), seed=8)
    check(torch_cuda, w, [COMB0, COMB1, DIRECT])
    check(torch_cuda, w, [COMB1, DIRECT], bulk=256)


def test_paper_neighbourhoods(torch_cuda):
    for offs, dims in [(wl.positive_octant(3, 3), (12, 10, 9)), (wl.shells(3, (3, 7)), (16, 15, 17)),
                       (wl.moore(4, 1), (6, 5, 4, 7))]:
        for coll in ("alltoall", "allgather"):
            w = wl.Workload("nbh", coll, dims, offs, 16, seed=3)
            check(torch_cuda, w, [COMB1, DIRECT] + ([TORUS] if coll == "alltoall" and len(offs) < 200 else []))


def test_alltoallv_with_different_send_and_receive_layouts(torch_cuda):
    """Receive displacements are a permutation of the send displacements with gaps, so source
    and destination of a block are misaligned against each other."""
    torch = torch_cuda
    rng = np.random.default_rng(31)
    dims, offs = (7, 6, 5), wl.moore(3, 1)
    P, s = 210, 26
    lens = rng.choice([0, 4, 16, 20, 64, 260, 1024, 1500], size=s).astype(np.int64)
    sd = wl.packed_displacements(lens)
    rd = np.zeros(s, np.int64)
    cur = 8
    for i in rng.permutation(s):
        rd[i] = cur
        cur += lens[i] + int(rng.choice([0, 4, 12]))
    ss = (int(lens.sum()) + 15) // 16 * 16
    rs = (int((rd + lens).max()) + 15) // 16 * 16
    send_h = wl.payload_np("uint8", 9, 0, 0, P * ss).reshape(P, ss).copy()
    send = torch.from_numpy(send_h).cuda()
    recv = torch.empty((P, rs), dtype=torch.uint8, device="cuda")
    comm = iso.Iso_neighborhood_create(dims, offs)
    req = iso.Iso_neighbor_alltoallv_init(send, lens, sd, 1, recv, lens, rd, 1, comm)
    st = iso.Iso_request_get_stats(req)
    assert (st["send_stride"], st["recv_stride"]) == (ss, rs)
    want = oracle.alltoallv(dims, offs, lens, sd, rd, ss, rs, send_h, fill=POISON)
    for alg, fusion in (COMB1, COMB0, COMB2, DIRECT, TORUS):
        iso.Iso_request_set_algorithm(req, alg, fusion)
        recv.fill_(POISON)
        iso.Iso_Start(req)
        iso.Iso_wait(req)
        assert np.array_equal(recv.cpu().numpy(), want), (alg, fusion)
    iso.Iso_request_free(req)
    iso.Iso_comm_free(comm)


def test_stencil_shaped_irregular_sizes(torch_cuda):
    # corners 1 byte, edges mhat, faces mhat^2, packed: every displacement is odd, long blocks
    # are split into a narrow head, an aligned body (bulk kernel) and a narrow tail
    for mhat in (8, 32):
        full = wl.config("stencil_d3_m%d" % mhat)
        w = wl.Workload(full.name, "alltoallv", (9, 8, 10), full.offsets, 0, lens=full.lens, seed=21)
        check(torch_cuda, w, [COMB0, COMB1, COMB2, ALT1, DIRECT, TORUS])
        check(torch_cuda, w, [COMB1], bulk=0)


def test_ragged_rows_with_bulk_warps(torch_cuda):
    """Iso_request_set_hybrid: the long bodies of ragged rows moved by bulk warps of the same
    launch.  Same bytes as the oracle for every schedule, in slabs, through host buffers and
    after the tuner (which tries the launch form both ways) has made its choice."""
    torch = torch_cuda
    stencil = wl.config("stencil_d3_m32")
    cases = [wl.config("cfg5_32x32x32"), wl.Workload("st", "alltoallv", (9, 8, 10), stencil.offsets, 0, lens=stencil.lens, seed=21),
             wl.Workload("ragged", "alltoallv", (37, 53), wl.moore(2, 1), 0,
                         lens=np.array([1024, 4, 2064, 16, 1040, 8, 3072, 64]), seed=8),
             wl.Workload("odd", "alltoallv", (5, 7, 6), wl.moore(3, 1), 0,
                         lens=np.array([1 + (977 * i) % 1500 for i in range(26)]), seed=9)]
    for w in cases:
        run = Run(torch, w)
        want = oracle_result(w, run.send_host)
        iso.Iso_request_set_hybrid(run.req, True)
        for slabs in (0, 3):
            iso.Iso_request_set_slabs(run.req, slabs)
            for alg, fusion in (COMB1, COMB0, COMB2, DIRECT, TORUS):
                got = run.result(alg, fusion)
                assert np.array_equal(got, want), (w.name, slabs, alg, fusion)
        assert any(p["kernel"] == 1 and p["len"] < 4096 for p in iso.Iso_request_get_parts(run.req))
        assert iso.Iso_request_check_guards(run.req) == 0
        hs = torch.from_numpy(run.send_host).pin_memory()
        hr = torch.zeros((w.P, run.rs), dtype=torch.uint8).pin_memory()
        run.result(*COMB1)
        iso.Iso_Start_host(run.req, hs, hr)
        iso.Iso_wait(run.req)
        lens, sd, rd, ss, rs = layout(w)
        covered = np.zeros(rs, bool)
        for i in range(w.s):
            covered[rd[i]:rd[i] + lens[i]] = True
        assert np.array_equal(hr.numpy()[:, covered], want[:, covered]), w.name
        iso.Iso_request_tune(run.req, torch.cuda.current_stream(), cold=False)
        run.recv.fill_(POISON)
        iso.Iso_Start(run.req, torch.cuda.current_stream())
        iso.Iso_wait(run.req)
        assert np.array_equal(run.recv.cpu().numpy(), want), (w.name, "tuned")
        run.close()


def test_allgatherv_and_unaligned_receive_layout(torch_cuda):
    torch = torch_cuda
    dims, offs = (6, 7), wl.moore(2, 1)
    P, s, m = 42, 8, 20
    rd = np.array([3 + 29 * i for i in range(s)], dtype=np.int64)      # gaps, odd displacements
    send_host = wl.payload_np("uint8", 1, 0, 0, P * 32).reshape(P, 32).copy()   # stride = 20 rounded up to 32
    send = torch.from_numpy(send_host).cuda()
    comm = iso.Iso_neighborhood_create(dims, offs)
    recv = torch.full((P, 240), POISON, dtype=torch.uint8, device="cuda")
    req = iso.Iso_neighbor_allgatherv_init(send, m, 1, recv, [m] * s, rd, 1, comm)
    st = iso.Iso_request_get_stats(req)
    assert (st["send_stride"], st["recv_stride"]) == (32, 240)
    for alg, fusion in (COMB1, DIRECT):
        iso.Iso_request_set_algorithm(req, alg, fusion)
        recv.fill_(POISON)
        iso.Iso_Start(req)
        iso.Iso_wait(req)
        got = recv.cpu().numpy()
        blocks = oracle.allgather(dims, offs, m, np.ascontiguousarray(send_host[:, :m])).reshape(P, s, m)
        want = np.full((P, 240), POISON, np.uint8)
        for i in range(s):
            want[:, rd[i]:rd[i] + m] = blocks[:, i]
        assert np.array_equal(got, want)
    iso.Iso_request_free(req)
    iso.Iso_comm_free(comm)


def test_mesh(torch_cuda):
    """Non-periodic dimensions: blocks whose source lies outside are not delivered."""
    torch = torch_cuda
    for dims, periodic, offs, m in [((9, 11), [0, 0], wl.moore(2, 2), 16), ((6, 7, 5), [0, 1, 0], wl.moore(3, 1), 64),
                                    ((12, 9), [1, 0], wl.moore(2, 1), 1024), ((7, 6, 5), [0, 0, 1], wl.positive_octant(3, 3), 16)]:
        for coll in ("alltoall", "allgather"):
            w = wl.Workload("mesh", coll, dims, offs, m, seed=4)
            run = Run(torch, w, periodic=periodic)
            want = oracle_result(w, run.send_host, periodic=periodic)
            algs = (DIRECT, COMB1, COMB0, COMB2, ALT1) if coll == "alltoall" else (DIRECT, COMB1, COMB0, COMB2)
            for alg, fusion in algs:
                got = run.result(alg, fusion)
                assert np.array_equal(got, want), (dims, coll, alg, fusion)
            run.close()


def test_persistent_request_streams_and_host_buffers(torch_cuda):
    torch = torch_cuda
    w = wl.Workload("p", "alltoall", (16, 16, 8), wl.moore(3, 1), 64, kind="fp32", seed=12)
    side = torch.cuda.Stream()
    run = Run(torch, w, stream=side)
    want = oracle_result(w, run.send_host)
    for _ in range(3):                       # init once, start many times
        assert np.array_equal(run.result(*COMB1), want)
    # new contents in the same buffers
    send2 = wl.payload_np(w.kind, 77, 0, 0, w.P * run.ss).reshape(w.P, run.ss).copy()
    run.send.copy_(torch.from_numpy(send2))
    torch.cuda.synchronize()
    assert np.array_equal(run.result(*COMB1), oracle_result(w, send2))
    # host buffers through the library's own copies
    hs = torch.from_numpy(run.send_host).pin_memory()
    hr = torch.empty((w.P, run.rs), dtype=torch.uint8).pin_memory()
    hr.fill_(0)
    iso.Iso_Start_host(run.req, hs, hr, side)
    iso.Iso_wait(run.req)
    assert np.array_equal(hr.numpy(), want)
    run.close()


def test_host_buffer_starts_replayed_from_a_graph(torch_cuda):
    """Repeated Iso_Start_host calls with the same page-locked buffers: the first is enqueued
    call by call, the second is captured into a graph, later ones replay it.  New contents in
    the same host buffer must come through every time, on a side stream as well."""
    torch = torch_cuda
    w = wl.config("cfg2_alltoall")
    side = torch.cuda.Stream()
    run = Run(torch, w, stream=side)
    hs = torch.empty((w.P, run.ss), dtype=torch.uint8).pin_memory()
    hr = torch.empty((w.P, run.rs), dtype=torch.uint8).pin_memory()
    try:
        for k in range(5):
            contents = wl.payload_np(w.kind, 900 + k, 0, 0, w.P * run.ss).reshape(w.P, run.ss)
            hs.copy_(torch.from_numpy(contents))
            hr.fill_(0)
            run.recv.fill_(POISON)
            torch.cuda.synchronize()
            iso.Iso_Start_host(run.req, hs, hr, side)
            iso.Iso_wait(run.req)
            assert np.array_equal(hr.numpy(), oracle_result(w, contents)), k
            t = iso.Iso_request_get_host_transfer_ms(run.req)
            assert t["slabs"] == 32 and 0 < t["upload_ms"] <= t["total_ms"] and 0 < t["download_ms"] <= t["total_ms"], t
        # a plain start in between, then host buffers again
        assert np.array_equal(run.result(*COMB1), oracle_result(w, contents))
        iso.Iso_Start_host(run.req, hs, hr, side)
        iso.Iso_wait(run.req)
        assert np.array_equal(hr.numpy(), oracle_result(w, contents))
    finally:
        run.close()


@pytest.mark.parametrize("name", ["cfg2_alltoall", "cfg2_allgather", "cfg3_m64", "cfg5"])
def test_host_buffers_pipelined_over_slabs(torch_cuda, name):
    """Iso_Start_host uploads, runs and downloads slab by slab along dimension 0; the result
    must not depend on that, for every schedule, twice in a row with different contents."""
    torch = torch_cuda
    w = wl.config(name)
    if name == "cfg5":
        w = wl.Workload("v", "alltoallv", (16, 8, 8), w.offsets, 0, lens=w.lens, seed=5)
    run = Run(torch, w)
    hs = torch.from_numpy(run.send_host).pin_memory()
    hr = torch.empty((w.P, run.rs), dtype=torch.uint8).pin_memory()
    algs = [COMB1, COMB0, ALT1, DIRECT] + ([TORUS] if w.collective == "alltoall" else [])
    if w.collective == "allgather":
        algs = [COMB1, DIRECT]
    try:
        for seed_shift, (alg, fusion) in enumerate(algs):
            contents = wl.send_buffer_np(wl.Workload(w.name, w.collective, w.dims, w.offsets, w.block_bytes, lens=w.lens,
                                                     kind=w.kind, seed=w.seed + seed_shift), run.ss)
            hs.copy_(torch.from_numpy(contents))
            want = oracle_result(w, contents)
            if fusion >= 100:
                iso.Iso_request_set_layout(run.req, iso.ISO_LAYOUT_ALTERNATING)
                fusion -= 100
            else:
                iso.Iso_request_set_layout(run.req, iso.ISO_LAYOUT_PACKED)
            iso.Iso_request_set_algorithm(run.req, alg, fusion)
            run.recv.fill_(POISON)
            hr.fill_(0)
            torch.cuda.synchronize()
            iso.Iso_Start_host(run.req, hs, hr)
            iso.Iso_wait(run.req)
            got = hr.numpy()
            if w.collective == "alltoallv":
                # bytes of the stride that no block covers are whatever the device buffer held
                covered = np.zeros(run.rs, bool)
                lens, sd, rd, ss, rs = layout(w)
                for i in range(w.s):
                    covered[rd[i]:rd[i] + lens[i]] = True
                assert np.array_equal(got[:, covered], want[:, covered]), (name, alg)
            else:
                assert np.array_equal(got, want), (name, alg)
    finally:
        run.close()

