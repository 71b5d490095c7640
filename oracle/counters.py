"""Round and volume counts of the paper's schedules, by their definitions.

TEST INFRASTRUCTURE ONLY (see the package docstring).  Every function takes the
neighbourhood as a list of s integer offset vectors and applies the formula the
paper states, with plain Python loops and sets; nothing is shared with the
schedule builder of the CUDA library, whose statistics the tests compare with
these numbers.

Where ``dims`` is given the coordinates are first replaced by their residue
modulo p_j (Section II notes that on a small torus several coordinates can name the same process):
the residue in [0, p_j) for the direct-communication schedules, the
representative of smallest magnitude (ties towards the positive one) for the
hop-by-hop schedules.
"""
from __future__ import annotations

import numpy as np


def _vectors(offsets, d):
    flat = np.asarray(offsets, dtype=np.int64).reshape(-1).tolist()
    if d <= 0 or len(flat) % d:
        raise ValueError("offsets must hold s*d integers")
    return [tuple(flat[i * d:(i + 1) * d]) for i in range(len(flat) // d)]


def residues(offsets, dims):
    """Offsets with every coordinate reduced to [0, p_j)."""
    d = len(dims)
    return [tuple(c % p for c, p in zip(v, dims)) for v in _vectors(offsets, d)]


def symmetric(offsets, dims):
    """Offsets with every coordinate replaced by its smallest-magnitude representative."""
    out = []
    for v in residues(offsets, dims):
        out.append(tuple(c if 2 * c <= p else c - p for c, p in zip(v, dims)))
    return out


def moore_size(d: int, r: int) -> int:
    """s = (2r+1)^d - 1 (Section IV)."""
    return (2 * r + 1) ** d - 1


# --- hop-by-hop torus schedules (Section III-A, Algorithm 1) -------------------------

def torus_rounds(offsets, d, dims=None) -> int:
    """D = sum_j ( max_i max(c^i_j, 0) + max_i max(-c^i_j, 0) ): the two loops of Algorithm 1."""
    vs = symmetric(offsets, dims) if dims is not None else _vectors(offsets, d)
    D = 0
    for j in range(d):
        D += max([max(v[j], 0) for v in vs], default=0)
        D += max([max(-v[j], 0) for v in vs], default=0)
    return D


def torus_volume(offsets, d, dims=None) -> int:
    """V = sum_i ||C^i||_1 (Section III-A)."""
    vs = symmetric(offsets, dims) if dims is not None else _vectors(offsets, d)
    return sum(sum(abs(c) for c in v) for v in vs)


def allgather_torus_volume(offsets, d, dims=None) -> int:
    """W: blocks received per process by the hop-by-hop allgather (Section III-B).

    Every edge of the prefix trie is one block routed |weight| hops, so W is the
    sum of |weight| over the distinct edges (equivalently over distinct non-empty
    prefixes of the offset vectors).
    """
    vs = symmetric(offsets, dims) if dims is not None else _vectors(offsets, d)
    prefixes = set()
    for v in vs:
        for j in range(1, d + 1):
            prefixes.add(v[:j])
    return sum(abs(p[-1]) for p in prefixes)


# --- direct communication along the dimensions (Section V) ---------------------------

def direct_hops(offsets, d, dims=None):
    """Per neighbour: the number of non-zero coordinates of C^i."""
    vs = residues(offsets, dims) if dims is not None else _vectors(offsets, d)
    return [sum(1 for c in v if c != 0) for v in vs]


def direct_rounds_per_dim(offsets, d, dims=None):
    """Per dimension: the number of different non-zero coordinates."""
    vs = residues(offsets, dims) if dims is not None else _vectors(offsets, d)
    return [len({v[j] for v in vs if v[j] != 0}) for j in range(d)]


def direct_rounds(offsets, d, dims=None) -> int:
    return sum(direct_rounds_per_dim(offsets, d, dims))


def direct_volume(offsets, d, dims=None) -> int:
    """Total number of block transmissions per process: sum of the hop counts."""
    return sum(direct_hops(offsets, d, dims))


def allgather_direct_volume(offsets, d, dims=None, order=None) -> int:
    """Blocks received per process by the direct-communication allgather: one per
    trie edge with a non-zero weight (a zero edge forwards nothing).  `order` is the
    order in which the trie visits the dimensions (Section III-B leaves it open;
    default 0..d-1): the count depends on it unless the neighbourhood is symmetric
    in the dimensions."""
    vs = residues(offsets, dims) if dims is not None else _vectors(offsets, d)
    if order is not None:
        vs = [tuple(v[k] for k in order) for v in vs]
    prefixes = set()
    for v in vs:
        for j in range(1, d + 1):
            prefixes.add(v[:j])
    return sum(1 for p in prefixes if p[-1] != 0)


def trie_level_sizes(offsets, d):
    """Number of distinct prefixes of length 1..d (the node counts of Fig. 1)."""
    vs = _vectors(offsets, d)
    return [len({v[:j] for v in vs}) for j in range(1, d + 1)]
