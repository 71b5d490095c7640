"""Pins for the paper's round / volume formulas and for the input generators."""
import itertools

import numpy as np
import pytest

from oracle import counters
from paper_1606_07676_b200 import workloads as wl


@pytest.mark.parametrize("d,r,s", [(2, 1, 8), (3, 1, 26), (4, 1, 80), (5, 1, 242), (3, 3, 342), (2, 2, 24)])
def test_moore_sizes_and_rounds(d, r, s):
    # Section IV: s = (2r+1)^d - 1 neighbours, D = 2rd rounds
    offs = wl.moore(d, r)
    assert offs.shape == (s, d) and counters.moore_size(d, r) == s
    assert counters.torus_rounds(offs, d) == 2 * r * d
    # Section V: rounds per dimension = number of distinct non-zero coordinates (2r here),
    # hops per block = number of non-zero coordinates
    assert counters.direct_rounds(offs, d) == 2 * r * d
    assert counters.direct_rounds_per_dim(offs, d) == [2 * r] * d
    hops = counters.direct_hops(offs, d)
    assert hops == [int(np.count_nonzero(v)) for v in offs]
    # counted directly: a coordinate is non-zero in 2r(2r+1)^(d-1) of the vectors
    assert sum(hops) == 2 * r * d * (2 * r + 1) ** (d - 1)
    # V = sum of 1-norms; per dimension sum|c| = 2*(1+..+r)*(2r+1)^(d-1)
    assert counters.torus_volume(offs, d) == d * r * (r + 1) * (2 * r + 1) ** (d - 1)
    # allgather volume never exceeds the all-to-all volume (Section III-B)
    assert counters.allgather_torus_volume(offs, d) <= counters.torus_volume(offs, d)
    assert counters.allgather_direct_volume(offs, d) <= counters.direct_volume(offs, d)
    # every zero-padded prefix of a Moore vector is itself in the neighbourhood
    assert counters.allgather_direct_volume(offs, d) == s


def test_27_point_stencil_26_to_6():
    # Introduction: the 27-point stencil needs 6 rounds instead of 26
    offs = wl.moore(3, 1)
    assert len(offs) == 26 and counters.torus_rounds(offs, 3) == 6


def test_moore_order_is_lexicographic_last_fastest():
    offs = wl.moore(2, 1).tolist()
    assert offs == [[-1, -1], [-1, 0], [-1, 1], [0, -1], [0, 1], [1, -1], [1, 0], [1, 1]]


def test_paper_neighbourhood_sizes():
    # Section IV / VI figure captions
    assert len(wl.positive_octant(3, 3)) == 63
    assert len(wl.shells(3, (3, 7))) == 1396
    assert len(wl.positive_octant(3, 1)) == 7     # the octant example of Section II
    sh = wl.shells(3, (3, 7))
    assert counters.torus_rounds(sh, 3) == 2 * 7 * 3    # the paper puts the hop-by-hop schedule at about 2*r2*d = 42 rounds


def test_fig1_trie_shape():
    # the ten leaves drawn in Fig. 1; the figure shows 4, 7 and 10 nodes per level
    leaves = [(0, 0, 0), (0, 0, 1), (1, 0, 0), (1, 1, 0), (1, 1, 1), (3, 2, 0), (3, 3, 2), (4, 0, 1),
              (4, 0, 2), (4, 1, 1)]
    assert counters.trie_level_sizes(leaves, 3) == [4, 7, 10]
    # hop-by-hop volume: edge weights of the figure summed by hand:
    # level 0->1: 0+1+3+4 = 8; level 1->2: 0 | 0+1 | 2+3 | 0+1 = 7; leaves: 0+1 | 0 | 0+1 | 0 | 2 | 1+2 | 1 = 8
    assert counters.allgather_torus_volume(leaves, 3) == 8 + 7 + 8
    assert counters.torus_volume(leaves, 3) == sum(sum(v) for v in leaves)
    # direct variant: one transmission per non-zero edge: 3 + 4 + 6
    assert counters.allgather_direct_volume(leaves, 3) == 13


def test_trie_volume_under_another_visiting_order():
    # Section III-B leaves the order in which the trie visits the dimensions open.  Worked by
    # hand: {(1,1), (2,1)} has the non-zero edges 1, 1-1, 2, 2-1 first-to-last (4 blocks) and
    # 1, 1-1, 1-2 last-to-first (3 blocks: the two vectors then share their first edge)
    pair = [[1, 1], [2, 1]]
    assert counters.allgather_direct_volume(pair, 2) == 4
    assert counters.allgather_direct_volume(pair, 2, order=(0, 1)) == 4
    assert counters.allgather_direct_volume(pair, 2, order=(1, 0)) == 3
    # a Moore neighbourhood is symmetric in the dimensions: s blocks in any order
    for order in ((0, 1, 2), (2, 1, 0), (1, 0, 2), (2, 0, 1)):
        assert counters.allgather_direct_volume(wl.moore(3, 2), 3, order=order) == 124


def test_small_torus_aliasing():
    # coordinates that are equal modulo p_j share a round; a multiple of p_j needs no hop
    offs = [[1], [4], [-2], [3], [0]]
    assert counters.direct_rounds(offs, 1, dims=(3,)) == 1          # residues 1,1,1,0,0
    assert counters.direct_hops(offs, 1, dims=(3,)) == [1, 1, 1, 0, 0]
    assert counters.symmetric([[2], [3]], (4,)) == [(2,), (-1,)]


def test_irregular_size_rule_total():
    # Section IV: block to neighbour i has size mhat^(d - ||C^i||); mhat = 512, d = 3, r = 1
    offs = wl.moore(3, 1)
    total = sum(512 ** (3 - int(np.abs(v).sum())) for v in offs)
    assert total == 8 * 1 + 12 * 512 + 6 * 512 ** 2
    assert abs(total / 2 ** 20 - 1.5) < 0.01      # the paper gives 1.5 MB for the whole send buffer


# ----------------------------------------------------------------------- generators
def test_words_are_counter_based_and_match_torch():
    import torch
    a = wl.words_np(123, 0, 0, 1000)
    b = wl.words_np(123, 0, 400, 50)
    assert np.array_equal(a[400:450], b)
    assert not np.array_equal(a, wl.words_np(124, 0, 0, 1000))
    assert not np.array_equal(a, wl.words_np(123, 1, 0, 1000))
    t = wl.words_torch(123, 0, 0, 1000, "cpu", chunk=300).numpy().view(np.uint32)
    assert np.array_equal(a, t)
    # scalar definition
    g = 77
    base = wl._base(123, 0)
    assert int(a[g]) == wl.mix64((base + g * wl._GOLDEN) & wl._MASK64) >> 32


def test_splitmix64_first_outputs():
    # published reference outputs of splitmix64 seeded with 1234567
    st = wl.Stream(1234567)
    assert [st.next() for _ in range(3)] == [6457827717110365317, 3203168211198807973, 9817491932198370423]


@pytest.mark.parametrize("kind", wl.KINDS)
def test_payload_slices_and_ranges(kind):
    import torch
    full = wl.payload_np(kind, 5, 0, 0, 4096)
    assert np.array_equal(full[100:1000], wl.payload_np(kind, 5, 0, 100, 900))
    assert np.array_equal(full, wl.payload_torch(kind, 5, 0, 4096, "cpu").numpy())
    if kind == "fp32":
        f = full.view(np.float32)
        assert f.min() >= -1.0 and f.max() < 1.0 and len(np.unique(f)) > 1000
    else:
        assert len(np.unique(full)) > 200


def test_config5_recipe():
    w = wl.config("cfg5")
    assert w.offsets.shape == (30, 3) and w.P == 131072
    rows = [tuple(v) for v in w.offsets.tolist()]
    assert len(set(rows)) == 30 and (0, 0, 0) not in rows
    assert np.abs(w.offsets).max() <= 3
    assert set(w.lens.tolist()) <= {4, 16, 64, 256, 1024}
    w2 = wl.config("cfg5")
    assert np.array_equal(w.offsets, w2.offsets) and np.array_equal(w.lens, w2.lens)
    assert not np.array_equal(w.offsets, wl.config("cfg5", seed=1).offsets)


def test_named_configs():
    shapes = {"cfg1": (64, 8), "cfg2_alltoall": (32768, 26), "cfg2_allgather": (32768, 26),
              "cfg3_m64": (65536, 24), "cfg4": (32768, 242), "cfg5": (131072, 30)}
    for name, (P, s) in shapes.items():
        w = wl.config(name)
        assert (w.P, w.s) == (P, s)
    assert wl.packed_displacements([4, 16, 64]).tolist() == [0, 4, 20]
