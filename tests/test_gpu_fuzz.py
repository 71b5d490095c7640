"""Randomised parity: many small random tori, neighbourhoods, block layouts, schedules and
options against the CPU oracle (seeded, so every run tests the same cases)."""
import numpy as np
import pytest

import oracle
from paper_1606_07676_b200 import binding as iso
from paper_1606_07676_b200 import workloads as wl
from schedule_sim import POISON



def _expected(kind, dims, offs, lens, sd, rd, ss, rs, send, periodic):
    """The oracle's receive buffers (its mesh form where a dimension does not wrap);
    undelivered and uncovered bytes hold the poison value."""
    P, s = int(np.prod(dims)), len(offs)
    want = np.full((P, rs), POISON, np.uint8)
    if s == 0:
        return want
    if kind != "allgather":
        return oracle.alltoallv(dims, offs, lens, sd, rd, ss, rs, send, fill=POISON, periodic=periodic)
    m = int(lens[0])
    if m:
        blocks = oracle.allgather(dims, offs, m, np.ascontiguousarray(send[:, :m]), periodic=periodic, fill=POISON)
        for i in range(s):
            want[:, rd[i]:rd[i] + m] = blocks[:, i * m:(i + 1) * m]
    return want


def random_cases(chunk, trials=40):
    """Seeded random problems: geometry, neighbourhood, block layout, mesh flags."""
    rng = np.random.default_rng(1000 + chunk)
    for trial in range(trials):
        d = int(rng.integers(1, 6))
        dims = [int(x) for x in rng.integers(1, 8, size=d)]
        while int(np.prod(dims)) > 6000:
            dims[int(np.argmax(dims))] -= 1
        P = int(np.prod(dims))
        s = int(rng.integers(0, 30))
        offs = rng.integers(-9, 10, size=(s, d)).astype(np.int32)
        if s > 3 and rng.random() < 0.5:
            offs[1] = 0
            offs[3] = offs[2]
        kind = str(rng.choice(["alltoall", "allgather", "alltoallv"]))
        mesh = rng.random() < 0.25
        periodic = [int(rng.random() < 0.5) if mesh else 1 for _ in range(d)]
        if kind == "alltoallv":
            lens = rng.choice([0, 1, 2, 4, 8, 16, 24, 64, 100, 512, 528, 1024, 2048], size=s).astype(np.int64)
            sd = wl.packed_displacements(lens)
            rd = sd.copy()
            if rng.random() < 0.5 and s:
                cur = int(rng.choice([0, 4, 16]))
                for i in rng.permutation(s):
                    rd[i] = cur
                    cur += int(lens[i]) + int(rng.choice([0, 0, 4, 16]))
            ss = (int((sd + lens).max()) + 15) // 16 * 16 if s else 0
            rs = (int((rd + lens).max()) + 15) // 16 * 16 if s else 0
        else:
            m = int(rng.choice([1, 2, 4, 8, 12, 16, 32, 64, 96, 512, 1024]))
            lens = np.full(s, m, np.int64)
            rd = np.arange(s, dtype=np.int64) * m
            sd = rd.copy() if kind == "alltoall" else np.zeros(s, np.int64)
            ss = s * m if kind == "alltoall" else m
            rs = s * m
        send_h = wl.payload_np("uint8", int(rng.integers(1 << 30)), 0, 0, max(P * ss, 1))[:P * ss].reshape(P, ss).copy()
        is_mesh = not all(periodic)
        choices = [(iso.ISO_ALG_DIRECT, 1)]
        choices += [(iso.ISO_ALG_COMBINING, g) for g in (0, 1, 2, 3)]
        if not is_mesh and kind != "allgather":
            choices += [(iso.ISO_ALG_TORUS, 1)]
        options = [(int(rng.integers(0, 2)), bool(rng.integers(0, 2)), int(rng.choice([0, 256, 512, 1024])),
                    int(rng.choice([0, 1, 2, 3, 5]))) for _ in choices]
        yield dict(trial=trial, d=d, dims=dims, P=P, s=s, offs=offs, kind=kind, periodic=periodic, is_mesh=is_mesh,
                   lens=lens, sd=sd, rd=rd, ss=ss, rs=rs, send_h=send_h, choices=choices, options=options)


def make_request(c, send, recv):
    comm = iso.Iso_neighborhood_create(c["dims"], c["offs"].reshape(c["s"], c["d"]) if c["s"] else np.zeros((0, c["d"]), np.int32))
    if c["is_mesh"]:
        iso.Iso_comm_set_periodic(comm, c["periodic"])
    lens, s = c["lens"], c["s"]
    if c["kind"] == "alltoall":
        req = iso.Iso_neighbor_alltoall_init(send, int(lens[0]) if s else 4, 1, recv, int(lens[0]) if s else 4, 1, comm)
    elif c["kind"] == "allgather":
        req = iso.Iso_neighbor_allgather_init(send, int(lens[0]) if s else 4, 1, recv, int(lens[0]) if s else 4, 1, comm)
    else:
        req = iso.Iso_neighbor_alltoallv_init(send, lens, c["sd"], 1, recv, lens, c["rd"], 1, comm)
    return comm, req


def expected(c):
    return _expected(c["kind"], c["dims"], c["offs"], c["lens"], c["sd"], c["rd"], c["ss"], c["rs"], c["send_h"], c["periodic"])


def visiting_order(c, salt):
    """A permutation of the dimensions, drawn from the case's trial number (the allgather's
    trie may visit them in any order; the other collectives ignore it)."""
    d = len(c["dims"])
    return [int(x) for x in np.random.default_rng(1000 * c["trial"] + salt).permutation(d)]


@pytest.mark.gpu
@pytest.mark.parametrize("chunk", range(12))
def test_random_cases(chunk):
    import torch
    if not torch.cuda.is_available():
        pytest.fail("needs a CUDA device")
    torch.cuda.set_device(0)
    for c in random_cases(chunk):
        P, ss, rs = c["P"], c["ss"], c["rs"]
        send = torch.from_numpy(c["send_h"]).cuda() if P * ss else torch.zeros(1, dtype=torch.uint8, device="cuda")
        recv = torch.full((P, rs), POISON, dtype=torch.uint8, device="cuda") if rs else torch.zeros(1, dtype=torch.uint8, device="cuda")
        comm, req = make_request(c, send, recv)
        want = expected(c) if rs else None
        for (alg, fusion), (lay, single, bulk, slabs) in zip(c["choices"], c["options"]):
            iso.Iso_request_set_layout(req, lay)
            iso.Iso_request_set_slabs(req, slabs)
            iso.Iso_request_set_single_launch(req, single)
            iso.Iso_request_set_bulk_threshold(req, bulk)
            # two runs in five ask for the pipelined one-launch execution (1 or 3 slabs); it
            # applies where the schedule allows and is ignored elsewhere
            pipe = (0, 0, 1, 0, 3)[(c["trial"] + 2 * alg + fusion) % 5]
            iso.Iso_request_set_pipeline(req, pipe)
            iso.Iso_request_set_sender_side(req, (2, 1, 2, 0)[(c["trial"] + fusion) % 4])
            iso.Iso_request_set_hybrid(req, (c["trial"] + alg) % 2 == 0)
            iso.Iso_request_set_dimension_order(req, visiting_order(c, alg + fusion))
            iso.Iso_request_set_algorithm(req, alg, fusion)
            if rs:
                recv.fill_(POISON)
            torch.cuda.synchronize()
            via_host = bool(rs and P * ss and (c["trial"] + alg + fusion) % 3 == 0)
            if via_host:
                # through the host-buffer entry point (pipelined over slabs where it can be)
                hs = torch.from_numpy(c["send_h"]).pin_memory()
                hr = torch.zeros((P, rs), dtype=torch.uint8).pin_memory()
                iso.Iso_Start_host(req, hs, hr)
                iso.Iso_wait(req)
                got = hr.numpy()
            else:
                iso.Iso_Start(req)
                iso.Iso_wait(req)
            if rs and not via_host:
                got = recv.cpu().numpy()
            if rs:
                assert np.array_equal(got, want), dict(chunk=chunk, trial=c["trial"], dims=c["dims"], kind=c["kind"], s=c["s"],
                                                       alg=alg, fusion=fusion, layout=lay, single=single, bulk=bulk, host=via_host, slabs=slabs, pipeline=pipe,
                                                       periodic=c["periodic"], lens=c["lens"].tolist())
        iso.Iso_request_free(req)
        iso.Iso_comm_free(comm)


@pytest.mark.parametrize("chunk", range(6))
def test_random_cases_host_simulation(chunk):
    """The same random problems without a GPU: the exported parts are executed with numpy."""
    from schedule_sim import simulate
    for c in random_cases(chunk, trials=25):
        if c["rs"] == 0:
            continue
        comm, req = make_request(c, None, None)
        want = expected(c)
        for (alg, fusion), (lay, single, bulk, slabs) in zip(c["choices"], c["options"]):
            iso.Iso_request_set_layout(req, lay)
            iso.Iso_request_set_bulk_threshold(req, bulk)
            iso.Iso_request_set_hybrid(req, (c["trial"] + alg) % 2 == 0)
            iso.Iso_request_set_sender_side(req, (2, 1, 2, 0)[(c["trial"] + fusion) % 4])
            iso.Iso_request_set_dimension_order(req, visiting_order(c, alg + fusion))
            iso.Iso_request_set_algorithm(req, alg, fusion)
            st = iso.Iso_request_get_stats(req)
            got = simulate(iso.Iso_request_get_parts(req), c["dims"], st, c["send_h"] if c["ss"] else np.zeros((c["P"], 0), np.uint8),
                           periodic=c["periodic"])
            assert np.array_equal(got, want), dict(chunk=chunk, trial=c["trial"], dims=c["dims"], kind=c["kind"], alg=alg,
                                                   fusion=fusion, layout=lay, bulk=bulk, periodic=c["periodic"])
        iso.Iso_request_free(req)
        iso.Iso_comm_free(comm)
