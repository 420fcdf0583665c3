"""Seeded synthetic workloads shaped like the paper's attention layers.

This module only draws inputs (random tensors, token-to-shard maps, row samples).  It holds none of the
method's arithmetic and is the one module that both the CUDA tests/benchmark and the CPU oracle's tests
read, so that a random number never has to be reproduced in two places.  numpy only.

Recipe (all from ``numpy.random.Generator(PCG64(seed))``, in this order): Q, K, V ~ N(0,1) iid float32;
optional outlier tokens (a fraction of token ids per sequence, K rows of every KV head multiplied by 8);
values rounded to the I/O type (bf16 round-to-nearest-even, or kept fp32); then the token-to-shard maps.
"""
from __future__ import annotations

import dataclasses
import math

import numpy as np


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """float32 -> nearest bf16 (ties to even), returned as float32 holding the rounded value."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + bias) & np.uint32(0xFFFF0000)).view(np.float32)


def bf16_bits(x_rounded: np.ndarray) -> np.ndarray:
    """Upper 16 bits of float32 values that are already bf16-representable (uint16 view for upload)."""
    u = np.ascontiguousarray(x_rounded, dtype=np.float32).view(np.uint32)
    return (u >> np.uint32(16)).astype(np.uint16)


def shard_map(kind: str, n: int, n_shards: int, rng: np.random.Generator | None = None, block: int = 64) -> np.ndarray:
    """token -> shard id.

    round_robin : t % n_shards                      (a (c=1, delta=n_shards) sharding)
    block_rr    : (t // block) % n_shards           (a (c=block, delta=block*n_shards) sharding)
    random      : perm = rng.permutation(n); shard_of[perm[i]] = i % n_shards (equal-sized random shards)
    contiguous  : t * n_shards // n
    """
    t = np.arange(n, dtype=np.int64)
    if kind == "round_robin":
        return (t % n_shards).astype(np.int32)
    if kind == "block_rr":
        return ((t // block) % n_shards).astype(np.int32)
    if kind == "contiguous":
        return (t * n_shards // max(n, 1)).astype(np.int32)
    if kind == "random":
        assert rng is not None
        perm = rng.permutation(n)
        out = np.empty(n, np.int32)
        out[perm] = (np.arange(n) % n_shards).astype(np.int32)
        return out
    raise ValueError(kind)


@dataclasses.dataclass
class Workload:
    name: str
    B: int
    n_q: int
    n_kv: int
    H: int
    Hkv: int
    d: int
    dtype: str  # "f32" | "bf16"
    n_q_shards: int
    n_kv_shards: int
    q_pos_offset: int
    causal: bool
    scale: float
    seed: int
    q: np.ndarray  # [B, n_q, H, d]   float32, rounded to dtype
    k: np.ndarray  # [B, n_kv, Hkv, d]
    v: np.ndarray
    q_shard_of: np.ndarray  # [n_q]  int32
    kv_shard_of: np.ndarray  # [n_kv] int32

    @property
    def tol(self) -> float:
        return 2e-2 if self.dtype == "bf16" else 1e-4

    def visible_pairs(self) -> int:
        """Number of (query row, KV row) pairs that attention touches, summed over the batch."""
        if not self.causal:
            return self.B * self.n_q * self.n_kv
        pos = np.arange(self.n_q, dtype=np.int64) + self.q_pos_offset
        return int(self.B * np.clip(pos + 1, 0, self.n_kv).sum())

    def flops(self) -> float:
        """Algorithmic FLOP of QK^T and PV over visible pairs: 4 * d * H * pairs."""
        return 4.0 * self.d * self.H * self.visible_pairs()

    def kv_bytes(self) -> int:
        return 2 * self.B * self.n_kv * self.Hkv * self.d * (2 if self.dtype == "bf16" else 4)


def make_workload(name, B, n_q, n_kv, H, Hkv, d, dtype, q_map, kv_map, n_q_shards, n_kv_shards, seed,
                  outlier_frac=0.0, block=64, causal=True, q_pos_offset=None, symmetric=None) -> Workload:
    rng = np.random.Generator(np.random.PCG64(seed))
    q = rng.standard_normal((B, n_q, H, d), dtype=np.float32)
    k = rng.standard_normal((B, n_kv, Hkv, d), dtype=np.float32)
    v = rng.standard_normal((B, n_kv, Hkv, d), dtype=np.float32)
    if outlier_frac > 0.0:
        n_out = int(round(outlier_frac * n_kv))
        for b in range(B):
            toks = rng.choice(n_kv, size=n_out, replace=False)
            k[b, toks] *= np.float32(8.0)
    if dtype == "bf16":
        q, k, v = round_to_bf16(q), round_to_bf16(k), round_to_bf16(v)
    if symmetric is None:
        symmetric = (n_q == n_kv and n_q_shards == n_kv_shards and q_map == kv_map)
    kv_shard_of = shard_map(kv_map, n_kv, n_kv_shards, rng, block)
    q_shard_of = kv_shard_of.copy() if symmetric else shard_map(q_map, n_q, n_q_shards, rng, block)
    if q_pos_offset is None:
        q_pos_offset = n_kv - n_q
    return Workload(name, B, n_q, n_kv, H, Hkv, d, dtype, n_q_shards, n_kv_shards, q_pos_offset, causal,
                    1.0 / math.sqrt(d), seed, q, k, v, q_shard_of, kv_shard_of)


# The five benchmark configurations (index 0..4 = configs 1..5), with optional size overrides so tests
# can run a reduced copy of the same recipe.
_CONFIGS = {
    "c1_tiny_f32": dict(B=1, n_q=256, n_kv=256, H=8, Hkv=8, d=64, dtype="f32", q_map="round_robin",
                        kv_map="round_robin", n_q_shards=4, n_kv_shards=4, seed=0),
    "c2_prefill_8b": dict(B=1, n_q=2048, n_kv=2048, H=32, Hkv=8, d=128, dtype="bf16", q_map="random",
                          kv_map="random", n_q_shards=8, n_kv_shards=8, seed=1),
    "c3_batched": dict(B=4, n_q=8192, n_kv=8192, H=32, Hkv=8, d=128, dtype="bf16", q_map="block_rr",
                       kv_map="block_rr", n_q_shards=16, n_kv_shards=16, seed=2, outlier_frac=0.01,
                       block=64),
    "c4_long_70b": dict(B=1, n_q=32768, n_kv=32768, H=64, Hkv=8, d=128, dtype="bf16", q_map="random",
                        kv_map="random", n_q_shards=32, n_kv_shards=32, seed=3),
    "c5_decode": dict(B=64, n_q=1, n_kv=16384, H=32, Hkv=8, d=128, dtype="bf16", q_map="round_robin",
                      kv_map="random", n_q_shards=1, n_kv_shards=16, seed=4),
}
CONFIG_NAMES = list(_CONFIGS)


def config(name: str, **overrides) -> Workload:
    kw = dict(_CONFIGS[name])
    kw.update(overrides)
    return make_workload(name, **kw)


def sample_rows(w: Workload, per_shard: int, seed: int = 1234, tile_edges: bool = False) -> np.ndarray:
    """A seeded sample of query rows (token ids), stratified over query shards: the first and last token of
    every shard plus ``per_shard`` random members, ascending and unique.  With ``tile_edges`` also the members at
    the positions of a shard's list where kernels change tile or sub-tile: 31, 32, 63, 64, 127 and the first of
    every group of 128."""
    rng = np.random.Generator(np.random.PCG64(seed))
    picked = []
    for j in range(w.n_q_shards):
        members = np.flatnonzero(w.q_shard_of == j)
        if members.size == 0:
            continue
        picked += [members[0], members[-1]]
        if tile_edges:
            slots = [s for s in (31, 32, 63, 64, 127) if s < members.size] + list(range(0, members.size, 128))
            picked += list(members[slots])
        picked += list(rng.choice(members, size=min(per_shard, members.size), replace=False))
    return np.unique(np.asarray(picked, dtype=np.int32))
