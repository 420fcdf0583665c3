"""Oracle-side shard-map generators (test infrastructure; numpy only, 0-based token ids).

(c, delta)-sharding, Section 6 (definition of a (c, delta)-sequence): shard i holds the tokens
i*c .. i*c+c-1, then the same window shifted by delta, 2*delta, ...; alpha = ceil(delta / c) shards cover [N].
m-split, Section 6.4: each hidden shard R_i is cut into m pieces R_{i,x}; the worked example (N=18, alpha=3,
c=2, delta=6, m=2) fixes the rule: R_{i,x} takes the elements of sorted R_i at ranks x, x+m, x+2m, ...;
query/KV shard number m*i + x.
"""
from __future__ import annotations

import math

import numpy as np


def alpha_of(c: int, delta: int) -> int:
    return math.ceil(delta / c)


def cdelta_shard_of(n: int, c: int, delta: int) -> np.ndarray:
    """shard_of[t] for (c, delta)-sharding of n tokens."""
    t = np.arange(n, dtype=np.int64)
    return ((t % delta) // c).astype(np.int32)


def m_split_shard_of(r_shard_of: np.ndarray, m: int) -> np.ndarray:
    """Refine hidden shards R_i into query/KV shards S_{m*i+x} = R_{i,x}."""
    r_shard_of = np.asarray(r_shard_of, dtype=np.int32)
    out = np.empty_like(r_shard_of)
    for i in np.unique(r_shard_of):
        members = np.flatnonzero(r_shard_of == i)  # ascending token order
        out[members] = m * i + (np.arange(members.size) % m)
    return out


def cluster_gap(c: int, delta: int) -> int:
    """Tokens between the end of one cluster of a (c, delta)-sequence and the start of the next, plus one
    (Section 6.2: delta - c + 1 = (alpha - 1) c + 1 when delta = alpha c)."""
    return delta - c + 1


def index_set_gaps(held) -> dict:
    """Clusters and gaps of an index set (Sections 6.2-6.3; collusion discussion of the appendix).

    ``held``: the token indices a node -- or a colluding set of nodes, whose members pool the union of their sets --
    has direct access to.  A cluster is a maximal run of consecutive indices; the gap between two neighbouring
    clusters is the number of indices strictly between them (the unknown tokens a vocab-matching attacker would have
    to enumerate, V ** gap candidates).  For a (c, delta)-sequence every gap is delta - c, i.e. the paper's
    "distance from one cluster to the next" delta - c + 1 minus one.  Written with Python sets, no arithmetic tricks.
    """
    held = sorted(set(int(t) for t in held))
    gaps = []
    clusters = 0
    for pos, t in enumerate(held):
        if pos == 0 or held[pos - 1] != t - 1:
            clusters += 1
            if pos > 0:
                gaps.append(len([u for u in range(held[pos - 1] + 1, t)]))
    return {"n_indices": len(held), "n_clusters": clusters, "min_gap": min(gaps) if gaps else -1,
            "max_gap": max(gaps) if gaps else -1}


def secure_hidden_state_criterion(held, rho: int) -> bool:
    """Section 6.2: the distance from a cluster to the next (gap + 1) must reach the vocab-matching threshold rho."""
    g = index_set_gaps(held)
    return g["min_gap"] < 0 or g["min_gap"] + 1 >= rho


def secure_full_criterion(held, rho: int) -> bool:
    """Theorem of Section 6.3 (and the collusion appendix: non-consecutive held indices must be more than rho
    positions apart): every gap between clusters must contain at least rho indices."""
    g = index_set_gaps(held)
    return g["min_gap"] < 0 or g["min_gap"] >= rho


def kl_gaps(r_held, s_shard_of, n_s_shards: int):
    """The (k, l)-gaps in the proof of the Section 6.3 theorem: for the node's sorted indices r_1 < r_2 < ... and KV
    shard S_k, gap (k, l) = {s in S_k : r_l < s < r_{l+1}} minus the node's own indices.  Returns, per k, the smallest
    NON-EMPTY gap size over l (-1 if all are empty): the attack needs a non-empty gap with fewer than rho members."""
    r = sorted(set(int(t) for t in r_held))
    own = set(r)
    s_shard_of = np.asarray(s_shard_of)
    out = []
    for k in range(n_s_shards):
        members = set(int(t) for t in np.flatnonzero(s_shard_of == k))
        best = -1
        for l in range(len(r) - 1):
            gap = {s for s in members if r[l] < s < r[l + 1]} - own
            if gap and (best < 0 or len(gap) < best):
                best = len(gap)
        out.append(best)
    return np.asarray(out, dtype=np.int32)
