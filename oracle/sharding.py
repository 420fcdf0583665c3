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
