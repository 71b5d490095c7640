"""Host-side tests of the C-ABI library: symbols, argument checking, and the schedule
builder, whose exported parts are executed with numpy and compared with the CPU oracle.
No GPU is needed: requests are created without buffers."""
import ctypes
import itertools
import re
import os

import numpy as np
import pytest

import oracle
from oracle import counters
from paper_1606_07676_b200 import binding as iso
from paper_1606_07676_b200 import workloads as wl
from schedule_sim import POISON, layout, make_request, oracle_result, send_buffer_np, simulate

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

ALGS = [(iso.ISO_ALG_COMBINING, 0), (iso.ISO_ALG_COMBINING, 1), (iso.ISO_ALG_COMBINING, 2),
        (iso.ISO_ALG_COMBINING, 8), (iso.ISO_ALG_DIRECT, 1), (iso.ISO_ALG_TORUS, 1),
        (iso.ISO_ALG_COMBINING, 100), (iso.ISO_ALG_COMBINING, 101)]


def set_alg(req, alg, fusion):
    """fusion >= 100 selects the alternating buffer layout of Algorithm 1 with fusion - 100."""
    if fusion >= 100:
        iso.Iso_request_set_layout(req, iso.ISO_LAYOUT_ALTERNATING)
        fusion -= 100
    else:
        iso.Iso_request_set_layout(req, iso.ISO_LAYOUT_PACKED)
    iso.Iso_request_set_algorithm(req, alg, fusion)


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "iso.h")).read()
    declared = set(re.findall(r"\b(Iso_[A-Za-z_]+)\s*\(", header))
    declared -= {"Iso_comm", "Iso_request"}
    lib = iso.load_library()
    assert declared == set(iso.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name
    iso.Iso_selftest()


def test_struct_layouts_match_header():
    assert ctypes.sizeof(iso.Iso_stats) == 11 * 4 + 4 + 7 * 8
    assert ctypes.sizeof(iso.Iso_part) == 8 * 4 + 3 * 8 + 8 * 4 + 8 * 4


def _tiny_workloads():
    rng = np.random.default_rng(2016)
    out = []
    for dims in [(1,), (2,), (5,), (3, 4), (2, 2, 3), (4, 1, 3), (3, 3, 3), (2, 3, 2, 2)]:
        d = len(dims)
        for s in (1, 4, 9):
            offs = rng.integers(-4, 5, size=(s, d)).astype(np.int32)
            if s >= 4:
                offs[1] = 0              # message to oneself
                offs[3] = offs[2]        # repeated neighbour
            out.append(wl.Workload("tiny", "alltoall", dims, offs, int(rng.choice([1, 4, 8, 16, 24])), seed=int(rng.integers(1 << 30))))
            out.append(wl.Workload("tiny", "allgather", dims, offs, int(rng.choice([2, 4, 16, 40])), seed=int(rng.integers(1 << 30))))
            lens = rng.choice([0, 1, 4, 12, 16, 52, 64, 100], size=s)
            out.append(wl.Workload("tiny", "alltoallv", dims, offs, 0, lens=lens.astype(np.int64), seed=int(rng.integers(1 << 30))))
    return out


@pytest.mark.parametrize("alg,fusion", ALGS)
def test_schedules_reproduce_the_oracle_on_tiny_tori(alg, fusion):
    n = 0
    for w in _tiny_workloads():
        if alg == iso.ISO_ALG_TORUS and w.collective == "allgather":
            continue
        comm, req = make_request(w)
        try:
            set_alg(req, alg, fusion)
            st = iso.Iso_request_get_stats(req)
            lens, sd, rd, ss, rs = layout(w)
            assert (st["send_stride"], st["recv_stride"]) == (ss, rs)
            send = send_buffer_np(w, ss)
            got = simulate(iso.Iso_request_get_parts(req), w.dims, st, send)
            want = oracle_result(w, send)
            assert np.array_equal(got, want), (w.dims, w.collective, w.offsets.tolist())
            n += 1
        finally:
            iso.Iso_request_free(req)
            iso.Iso_comm_free(comm)
    assert n > 40


@pytest.mark.parametrize("name", ["cfg1", "cfg3_m4"])
@pytest.mark.parametrize("alg,fusion", ALGS)
def test_schedules_on_paper_shaped_configs(name, alg, fusion):
    w = wl.config(name)
    if name == "cfg3_m4":
        w = wl.Workload(name, "alltoall", (16, 12), w.offsets, 4, kind="uint8")
    comm, req = make_request(w)
    set_alg(req, alg, fusion)
    st = iso.Iso_request_get_stats(req)
    send = send_buffer_np(w, st["send_stride"])
    got = simulate(iso.Iso_request_get_parts(req), w.dims, st, send)
    assert np.array_equal(got, oracle_result(w, send))
    iso.Iso_request_free(req)
    iso.Iso_comm_free(comm)


@pytest.mark.parametrize("coll", ["alltoall", "allgather"])
@pytest.mark.parametrize("nbh", ["moore3", "octant3", "shells", "fig1"])
def test_paper_neighbourhoods_small_torus(coll, nbh):
    offs = {"moore3": wl.moore(3, 1), "octant3": wl.positive_octant(3, 3), "shells": wl.shells(2, (1, 3)),
            "fig1": np.array([(0, 0, 0), (0, 0, 1), (1, 0, 0), (1, 1, 0), (1, 1, 1), (3, 2, 0), (3, 3, 2),
                              (4, 0, 1), (4, 0, 2), (4, 1, 1)], np.int32)}[nbh]
    dims = (5, 4, 6) if offs.shape[1] == 3 else (9, 8)
    w = wl.Workload(nbh, coll, dims, offs, 8)
    comm, req = make_request(w)
    for alg, fusion in ALGS:
        if alg == iso.ISO_ALG_TORUS and coll == "allgather":
            continue
        set_alg(req, alg, fusion)
        st = iso.Iso_request_get_stats(req)
        send = send_buffer_np(w, st["send_stride"])
        got = simulate(iso.Iso_request_get_parts(req), w.dims, st, send)
        assert np.array_equal(got, oracle_result(w, send)), (alg, fusion)
    iso.Iso_request_free(req)
    iso.Iso_comm_free(comm)


# ------------------------------------------------------------- statistics vs the paper
@pytest.mark.parametrize("name", ["cfg1", "cfg2_alltoall", "cfg3_m64", "cfg4", "cfg5"])
def test_alltoall_statistics_follow_section_v(name):
    w = wl.config(name)
    comm, req = make_request(w)
    st = iso.Iso_request_get_stats(req)
    d = w.d
    assert st["rounds"] == counters.direct_rounds(w.offsets, d, w.dims)
    assert st["parts"] == counters.direct_volume(w.offsets, d, w.dims)
    assert st["max_rounds_per_dim"] == max(counters.direct_rounds_per_dim(w.offsets, d, w.dims))
    assert st["rounds"] <= st["max_rounds_per_dim"] * d            # the N d bound on the rounds
    assert st["phases"] <= d
    lens = layout(w)[0]
    hops = counters.direct_hops(w.offsets, d, w.dims)
    assert st["bytes_min"] == 2 * w.P * int(lens.sum())
    assert st["bytes_moved"] == 2 * w.P * int(sum(int(l) * max(h, 1) for l, h in zip(lens, hops)))
    # hop-by-hop schedule of Algorithm 1
    iso.Iso_request_set_algorithm(req, iso.ISO_ALG_TORUS, 1)
    st = iso.Iso_request_get_stats(req)
    assert st["rounds"] == counters.torus_rounds(w.offsets, d, w.dims)
    assert st["parts"] == counters.torus_volume(w.offsets, d, w.dims)
    # straightforward schedule
    iso.Iso_request_set_algorithm(req, iso.ISO_ALG_DIRECT, 1)
    st = iso.Iso_request_get_stats(req)
    assert st["rounds"] == w.s and st["bytes_moved"] == st["bytes_min"] and st["launches"] >= 1
    iso.Iso_request_free(req)
    iso.Iso_comm_free(comm)


def test_hand_worked_schedule_4x4():
    # tests/golden/moore_4x4_schedule.txt: rounds, hops and first-hop buffers worked by hand
    golden = {}
    for line in open(os.path.join(ROOT, "tests", "golden", "moore_4x4_schedule.txt")):
        if line.startswith("#") or not line.strip():
            continue
        f = [x.strip() for x in line.split(":")]
        golden[f[0]] = f[1:]
    w = wl.Workload("hand", "alltoall", (4, 4), wl.moore(2, 1), 4)
    comm, req = make_request(w)
    iso.Iso_request_set_layout(req, iso.ISO_LAYOUT_ALTERNATING)
    iso.Iso_request_set_algorithm(req, iso.ISO_ALG_COMBINING, 0)
    parts = iso.Iso_request_get_parts(req)
    rounds = {}
    for p in parts:
        rounds.setdefault(p["round"], []).append(p)
    assert sorted(rounds) == [0, 1, 2, 3]
    for k in range(4):
        dim, shift = golden[str(k)][0].split()
        want_shift = [0, 0]
        want_shift[int(dim)] = int(shift) % 4
        assert sorted(q["slot"] for q in rounds[k]) == [int(x) for x in golden[str(k)][1].split()]
        assert all(q["shift"][:2] == want_shift for q in rounds[k])
    hops = [sum(1 for p in parts if p["slot"] == i) for i in range(8)]
    assert hops == [int(x) for x in golden["hops"][0].split()]
    first = {}
    for p in parts:
        first.setdefault(p["slot"], p)
    via_inter = sorted(i for i in range(8) if first[i]["dst_buf"] == iso.ISO_BUF_INTER)
    assert via_inter == [int(x) for x in golden["first_hop_into_intermediate"][0].split()]
    assert all(first[i]["src_buf"] == iso.ISO_BUF_SEND for i in range(8))
    last = {p["slot"]: p for p in parts}
    assert all(p["dst_buf"] == iso.ISO_BUF_RECV for p in last.values())
    st = iso.Iso_request_get_stats(req)
    assert (st["rounds"], st["parts"]) == (4, 12)
    iso.Iso_request_free(req)
    iso.Iso_comm_free(comm)


def test_buffer_layouts_of_a_three_hop_block():
    # 27-point stencil: the corner blocks make three hops.  Algorithm 1 sends them
    # send -> recv -> inter -> recv (receive buffer when an odd number of hops remains);
    # the packed layout keeps both intermediate copies in the library's buffer, writes the
    # receive buffer only with final hops, and lays places out so that each phase writes one
    # contiguous region of the intermediate buffer
    w = wl.Workload("s27", "alltoall", (4, 4, 4), wl.moore(3, 1), 64)
    comm, req = make_request(w)
    corner = [i for i, v in enumerate(w.offsets) if all(v)]
    assert len(corner) == 8
    iso.Iso_request_set_layout(req, iso.ISO_LAYOUT_ALTERNATING)
    parts = iso.Iso_request_get_parts(req)
    for i in corner:
        chain = [(p["src_buf"], p["dst_buf"]) for p in parts if p["slot"] == i]
        assert chain == [(iso.ISO_BUF_SEND, iso.ISO_BUF_RECV), (iso.ISO_BUF_RECV, iso.ISO_BUF_INTER),
                         (iso.ISO_BUF_INTER, iso.ISO_BUF_RECV)]
    assert iso.Iso_request_get_stats(req)["inter_stride"] == 20 * 64        # one place per multi-hop block
    moved = iso.Iso_request_get_stats(req)["bytes_moved"]
    iso.Iso_request_set_layout(req, iso.ISO_LAYOUT_PACKED)
    parts = iso.Iso_request_get_parts(req)
    st = iso.Iso_request_get_stats(req)
    assert st["bytes_moved"] == moved and st["inter_stride"] == (12 * 1 + 8 * 2) * 64
    for i in corner:
        chain = [(p["src_buf"], p["dst_buf"]) for p in parts if p["slot"] == i]
        assert chain == [(iso.ISO_BUF_SEND, iso.ISO_BUF_INTER), (iso.ISO_BUF_INTER, iso.ISO_BUF_INTER),
                         (iso.ISO_BUF_INTER, iso.ISO_BUF_RECV)]
    for ph in range(3):
        written = sorted((p["dst_off"], p["len"]) for p in parts if p["phase"] == ph and p["dst_buf"] == iso.ISO_BUF_INTER)
        for (a, n), (b, _) in zip(written, written[1:]):
            assert a + n == b, "phase %d does not write one contiguous region" % ph
        last = [p for p in parts if p["phase"] == ph and p["dst_buf"] == iso.ISO_BUF_RECV]
        assert all(sum(1 for q in parts if q["slot"] == p["slot"] and q["phase"] > ph) == 0 for p in last)
    iso.Iso_request_free(req)
    iso.Iso_comm_free(comm)


def test_allgather_statistics_follow_the_trie():
    for offs, dims in [(wl.moore(3, 1), (32, 32, 32)), (wl.positive_octant(3, 3), (16, 16, 16)),
                       (np.array([(0, 0, 0), (0, 0, 1), (1, 0, 0), (1, 1, 0), (1, 1, 1), (3, 2, 0), (3, 3, 2),
                                  (4, 0, 1), (4, 0, 2), (4, 1, 1)], np.int32), (8, 8, 8))]:
        w = wl.Workload("ag", "allgather", dims, offs, 64)
        comm, req = make_request(w)
        # the trie may visit the dimensions in any order (Section III-B): same rounds, same result,
        # and as many parts as the trie over the permuted vectors has non-zero edges
        send0 = send_buffer_np(w, 64)
        for order in itertools.permutations(range(3)):
            iso.Iso_request_set_dimension_order(req, order)
            assert iso.Iso_request_get_dimension_order(req, 3) == list(order)
            st = iso.Iso_request_get_stats(req)
            assert st["parts"] == counters.allgather_direct_volume(offs, 3, dims, order)
            assert st["rounds"] == counters.direct_rounds(offs, 3, dims)
            if w.P <= 4096:
                assert np.array_equal(simulate(iso.Iso_request_get_parts(req), w.dims, st, send0), oracle_result(w, send0))
        # default: last dimension first for these neighbourhoods (at most 8 distinct coordinates in dimension 0)
        iso.Iso_request_free(req)
        iso.Iso_comm_free(comm)
        comm, req = make_request(w)
        order = iso.Iso_request_get_dimension_order(req, 3)
        assert order == [2, 1, 0]
        st = iso.Iso_request_get_stats(req)
        assert st["parts"] == counters.allgather_direct_volume(offs, 3, dims, order)
        assert st["rounds"] == counters.direct_rounds(offs, 3, dims)
        assert st["bytes_moved"] == 2 * w.P * 64 * (st["parts"] + st["local_copies"])
        # sender-side launches: a parent block is read once for up to four of the places it is
        # copied to, every copy is written
        iso.Iso_request_set_sender_side(req, 2)
        st = iso.Iso_request_get_stats(req)
        parts = iso.Iso_request_get_parts(req)
        assert len(parts) == st["parts"] + st["local_copies"] and all(p["kernel"] == 2 for p in parts)
        children = {}
        for p in parts:
            key = (p["phase"], p["src_buf"], p["src_off"])
            children[key] = children.get(key, 0) + 1
        reads = sum(-(-n // 4) for n in children.values())
        assert st["bytes_moved"] == w.P * 64 * (reads + len(parts))
        # the schedule is the same one: executed on the host it gives the oracle's result
        send = send_buffer_np(w, st["send_stride"])
        if w.P <= 4096:
            assert np.array_equal(simulate(parts, w.dims, st, send), oracle_result(w, send))
        # the receiver-side form (asked for through a slab count) reads a block once per copy
        iso.Iso_request_set_slabs(req, 2)
        iso.Iso_request_set_bulk_threshold(req, 512)
        st2 = iso.Iso_request_get_stats(req)
        assert st2["bytes_moved"] == 2 * w.P * 64 * (st["parts"] + st["local_copies"])
        assert all(p["kernel"] == 0 for p in iso.Iso_request_get_parts(req))
        iso.Iso_request_free(req)
        iso.Iso_comm_free(comm)
    # Moore neighbourhoods need no intermediate storage: every padded prefix is a neighbour
    w = wl.config("cfg2_allgather")
    comm, req = make_request(w)
    st = iso.Iso_request_get_stats(req)
    assert (st["parts"], st["rounds"], st["inter_stride"]) == (26, 6, 0)
    iso.Iso_request_free(req)
    iso.Iso_comm_free(comm)


def test_fused_levels_interpolate_between_combining_and_direct():
    w = wl.config("cfg4")
    comm, req = make_request(w)
    moved = []
    for g in (1, 2, 3, 5):
        iso.Iso_request_set_algorithm(req, iso.ISO_ALG_COMBINING, g)
        st = iso.Iso_request_get_stats(req)
        moved.append(st["bytes_moved"])
        assert st["phases"] == -(-5 // g)
    assert moved == sorted(moved, reverse=True)
    assert moved[-1] == st["bytes_min"]
    iso.Iso_request_free(req)
    iso.Iso_comm_free(comm)


def test_alignment_classes_and_bulk_selection():
    # 4-byte aligned packed displacements: long blocks are split into a 16-byte aligned
    # body and narrow head / tail pieces; in such a ragged phase bodies from 4 KB on go to the
    # bulk kernel, shorter ones stay with the small pieces in the launch of mixed widths
    # (or, with Iso_request_set_hybrid, bodies from 256 bytes on go to the bulk warps of that launch)
    w = wl.Workload("v", "alltoallv", (4, 4), wl.moore(2, 1), 0, lens=np.array([4, 1024, 16, 8192, 64, 4, 256, 1024]))
    comm, req = make_request(w)
    parts = iso.Iso_request_get_parts(req)
    assert any(p["kernel"] == 1 for p in parts)
    for p in parts:
        assert p["src_off"] % p["width"] == 0 or p["kernel"] == 1
        if p["kernel"] == 1:
            assert p["src_off"] % 16 == 0 and p["dst_off"] % 16 == 0 and p["len"] % 16 == 0 and p["len"] >= 4096
    st = iso.Iso_request_get_stats(req)
    send = send_buffer_np(w, st["send_stride"])
    assert np.array_equal(simulate(parts, w.dims, st, send), oracle_result(w, send))
    iso.Iso_request_set_hybrid(req, True)
    parts = iso.Iso_request_get_parts(req)
    assert all(p["len"] >= 256 and p["len"] % 16 == 0 and p["src_off"] % 16 == 0 for p in parts if p["kernel"] == 1)
    assert any(p["kernel"] == 1 and p["len"] < 4096 for p in parts)
    assert all(p["len"] < 256 or p["width"] < 16 for p in parts if p["kernel"] == 0)
    assert np.array_equal(simulate(parts, w.dims, st, send), oracle_result(w, send))
    iso.Iso_request_set_hybrid(req, False)
    iso.Iso_request_set_bulk_threshold(req, 0)
    assert all(p["kernel"] == 0 for p in iso.Iso_request_get_parts(req))
    assert iso.Iso_request_get_stats(req)["bulk_bytes"] == 0
    iso.Iso_request_free(req)
    iso.Iso_comm_free(comm)


def test_bulk_threshold_left_to_the_library():
    """Which kernel moves large blocks when nobody says: the vector kernel where the library may
    run the all-to-all in slabs of its own that fit the L2, the bulk-copy kernel from 512 bytes
    elsewhere (a slab count asked for, slabs that would be too small, the direct schedule, the
    allgather), and whatever threshold the caller sets."""
    def kernels(req):
        return {p["kernel"] for p in iso.Iso_request_get_parts(req)}
    for name, want in (("cfg3_m512", {0}), ("cfg3_m4096", {0}), ("cfg3_m8192", {1}), ("cfg3_m512_8x256", {0}),
                       ("cfg3_m4096_2x256", {1})):
        comm, req = make_request(wl.config(name))
        assert kernels(req) == want, name
        if want == {0}:
            assert iso.Iso_request_get_stats(req)["bulk_bytes"] == 0
            iso.Iso_request_set_slabs(req, 2)            # the caller's slabs: back to the crossover of single launches
            assert kernels(req) == {1}, name
            iso.Iso_request_set_slabs(req, 0)
            assert kernels(req) == {0}, name
            set_alg(req, iso.ISO_ALG_DIRECT, 1)          # nothing to reuse: bulk copies
            assert kernels(req) == {1}, name
            set_alg(req, iso.ISO_ALG_COMBINING, 1)
            iso.Iso_request_set_bulk_threshold(req, 512)
            assert kernels(req) == {1}, name
            iso.Iso_request_set_bulk_threshold(req, 0)
            assert kernels(req) == {0}, name
        iso.Iso_request_free(req)
        iso.Iso_comm_free(comm)
    w = wl.Workload("ag", "allgather", (16, 16, 16), wl.moore(3, 1), 1024)
    comm, req = make_request(w)
    assert kernels(req) == {1}
    iso.Iso_request_free(req)
    iso.Iso_comm_free(comm)


def test_ragged_phases_lower_to_one_launch_of_mixed_widths(monkeypatch):
    """Irregular sizes: a phase whose pieces need several unit widths is one launch (the unit
    descriptors carry their width); ragged ends are cut into aligned power-of-two pieces of
    at most 4 bytes around a body of whole 16-byte units; bodies of 256 bytes and more are
    bulk copies of that same launch.  The exported parts still reproduce the oracle, with
    and without that lowering."""
    for name, phases, hybrid in (("cfg5_32x32x32", 3, False), ("stencil_d3_m32", 3, False), ("cfg5_32x32x32", 3, True),
                                 ("stencil_d3_m32", 3, True)):
        w = wl.config(name)
        comm, req = make_request(w)
        iso.Iso_request_set_hybrid(req, hybrid)
        st = iso.Iso_request_get_stats(req)
        assert st["phases"] == phases and st["launches"] == phases, st
        parts = iso.Iso_request_get_parts(req)
        for ph in range(phases):
            assert len({p["width"] for p in parts if p["phase"] == ph}) >= 2
        for p in parts:
            if p["kernel"] == 1:
                # a long 16-byte-aligned body: moved by the bulk warp of the same launch, in chunks
                assert p["len"] >= 256 and p["src_off"] % 16 == 0 and p["dst_off"] % 16 == 0 and p["len"] % 16 == 0
                continue
            assert p["kernel"] == 0 and p["width"] in (1, 2, 4, 8, 16)
            assert p["src_off"] % p["width"] == 0 and p["dst_off"] % p["width"] == 0 and p["len"] % p["width"] == 0
            assert not hybrid or p["width"] < 16 or p["len"] < 256
        assert any(p["kernel"] == 1 for p in parts) == hybrid
        iso.Iso_request_free(req)
        iso.Iso_comm_free(comm)
    # a small ragged case, executed on the host, both ways
    lens = np.array([1, 1024, 7, 33, 4, 250, 16, 2])
    w = wl.Workload("v", "alltoallv", (4, 3, 5), wl.moore(3, 1)[:8], 0, lens=lens, seed=11)
    for mixed in ("1", "0"):
        monkeypatch.setenv("ISO_MIXED", mixed)
        comm, req = make_request(w)
        st = iso.Iso_request_get_stats(req)
        parts = iso.Iso_request_get_parts(req)
        send = send_buffer_np(w, st["send_stride"])
        assert np.array_equal(simulate(parts, w.dims, st, send), oracle_result(w, send)), mixed
        if mixed == "1":
            assert st["launches"] == st["phases"]
        else:
            assert st["launches"] > st["phases"]
        iso.Iso_request_free(req)
        iso.Iso_comm_free(comm)


@pytest.mark.parametrize("dims,periodic,nbh", [((4, 5), [0, 1], "moore2"), ((5, 4, 3), [0, 0, 0], "moore1"),
                                               ((3, 6, 4), [1, 0, 1], "moore1"), ((7, 2), [0, 0], "far")])
def test_mesh_schedules(dims, periodic, nbh):
    offs = {"moore2": wl.moore(2, 2), "moore1": wl.moore(len(dims), 1),
            "far": np.array([[1, 0], [-3, 1], [7, 0], [0, 0], [2, -1], [-1, -1]], np.int32)}[nbh]
    w = wl.Workload("mesh", "alltoall", dims, offs, 4)
    comm, req = make_request(w, periodic=periodic)
    assert iso.Iso_request_get_stats(req)["algorithm"] == iso.ISO_ALG_COMBINING
    for alg, fusion in [(iso.ISO_ALG_DIRECT, 1), (iso.ISO_ALG_COMBINING, 0), (iso.ISO_ALG_COMBINING, 1),
                        (iso.ISO_ALG_COMBINING, 2), (iso.ISO_ALG_COMBINING, 101)]:
        set_alg(req, alg, fusion)
        st = iso.Iso_request_get_stats(req)
        send = send_buffer_np(w, st["send_stride"])
        got = simulate(iso.Iso_request_get_parts(req), w.dims, st, send, periodic=periodic)
        assert np.array_equal(got, oracle_result(w, send, periodic=periodic)), (alg, fusion)
    with pytest.raises(iso.IsoError):
        iso.Iso_request_set_algorithm(req, iso.ISO_ALG_TORUS, 1)
    iso.Iso_request_free(req)
    iso.Iso_comm_free(comm)
    # allgather on a mesh: direct and combining (a trie node exists only where its source does)
    wg = wl.Workload("mesh", "allgather", dims, offs, 4)
    comm, req = make_request(wg, periodic=periodic)
    assert iso.Iso_request_get_stats(req)["algorithm"] == iso.ISO_ALG_COMBINING
    for alg, fusion in [(iso.ISO_ALG_COMBINING, 1), (iso.ISO_ALG_COMBINING, 0), (iso.ISO_ALG_COMBINING, 2), (iso.ISO_ALG_DIRECT, 1)]:
        set_alg(req, alg, fusion)
        st = iso.Iso_request_get_stats(req)
        send = send_buffer_np(wg, st["send_stride"])
        got = simulate(iso.Iso_request_get_parts(req), wg.dims, st, send, periodic=periodic)
        assert np.array_equal(got, oracle_result(wg, send, periodic=periodic)), (alg, fusion)
    with pytest.raises(iso.IsoError):
        iso.Iso_request_set_algorithm(req, iso.ISO_ALG_TORUS, 1)
    iso.Iso_request_free(req)
    iso.Iso_comm_free(comm)


# ------------------------------------------------------------------------- error paths
def _code(fn, *a):
    with pytest.raises(iso.IsoError) as e:
        fn(*a)
    return e.value.code


def test_argument_errors():
    assert _code(iso.Iso_neighborhood_create, [0, 4], [[1, 0]]) == iso.ISO_ERR_DIMS
    assert _code(iso.Iso_neighborhood_create, [2] * 9, [[0] * 9]) == iso.ISO_ERR_DIMS
    assert _code(iso.Iso_neighborhood_create, [1 << 16, 1 << 16], [[1, 0]]) == iso.ISO_ERR_DIMS
    comm = iso.Iso_neighborhood_create([4, 4], wl.moore(2, 1))
    assert _code(iso.Iso_neighbor_alltoall_init, None, 2, 4, None, 4, 4, comm) == iso.ISO_ERR_COUNT
    assert _code(iso.Iso_neighbor_alltoall_init, None, -1, 4, None, -1, 4, comm) == iso.ISO_ERR_ARG
    assert _code(iso.Iso_neighbor_alltoall_init, 4096, 2, 4, None, 2, 4, comm) == iso.ISO_ERR_ARG
    ok = [4] * 8
    dd = [4 * i for i in range(8)]
    assert _code(iso.Iso_neighbor_alltoallv_init, None, ok, dd, 1, None, ok, [0] * 8, 1, comm) == iso.ISO_ERR_OVERLAP
    assert _code(iso.Iso_neighbor_alltoallv_init, None, ok, dd, 1, None, [8] * 8, dd, 1, comm) == iso.ISO_ERR_COUNT
    assert _code(iso.Iso_neighbor_alltoallv_init, None, ok, [-4] + dd[1:], 1, None, ok, dd, 1, comm) == iso.ISO_ERR_ARG
    # overlapping user buffers (addresses only; nothing is dereferenced at init)
    assert _code(iso.Iso_neighbor_alltoall_init, 1 << 20, 4, 1, (1 << 20) + 64, 4, 1, comm) == iso.ISO_ERR_OVERLAP
    req = iso.Iso_neighbor_alltoall_init(None, 4, 1, None, 1, 4, comm)     # 4 x 1 byte == 1 x 4 bytes
    assert _code(iso.Iso_request_set_algorithm, req, 7, 1) == iso.ISO_ERR_ARG
    assert _code(iso.Iso_request_set_algorithm, req, 0, -1) == iso.ISO_ERR_ARG
    assert _code(iso.Iso_Start, req) == iso.ISO_ERR_STATE                   # no buffers bound
    iso.Iso_wait(req)                                                       # nothing started: fine
    iso.Iso_comm_free(comm)                                                 # the request keeps the comm alive
    assert iso.Iso_request_get_stats(req)["s"] == 8
    iso.Iso_request_free(req)
    assert "overlap" in iso.Iso_error_string(iso.ISO_ERR_OVERLAP)


def test_empty_neighbourhood_and_zero_sized_blocks():
    comm = iso.Iso_neighborhood_create([3, 3], np.zeros((0, 2), np.int32))
    req = iso.Iso_neighbor_alltoall_init(None, 4, 4, None, 4, 4, comm)
    st = iso.Iso_request_get_stats(req)
    assert (st["s"], st["parts"], st["launches"], st["bytes_moved"]) == (0, 0, 0, 0)
    iso.Iso_request_free(req)
    iso.Iso_comm_free(comm)
    comm = iso.Iso_neighborhood_create([3, 3], wl.moore(2, 1))
    req = iso.Iso_neighbor_alltoall_init(None, 0, 4, None, 0, 4, comm)
    assert iso.Iso_request_get_stats(req)["launches"] == 0
    iso.Iso_request_free(req)
    iso.Iso_comm_free(comm)
