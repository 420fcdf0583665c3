"""Pins for the oracle's integer side: shard plan, sharded causal mask, shard-map generators (no GPU)."""
import itertools
import os

import numpy as np
import pytest

import oracle
from oracle import sharding
from paper_2507_05228_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "sharding_example_n18.txt")


def _golden():
    out = {}
    with open(GOLDEN) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            name, vals = line.split(":")
            out[name.strip()] = [int(x) for x in vals.split()]
    return out


def test_paper_worked_example_n18():
    """Section 6.4 example: alpha=3, c=2, delta=6, N=18, m=2 (1-based ids in the paper)."""
    g = _golden()
    c, delta, n, m = 2, 6, 18, 2
    assert sharding.alpha_of(c, delta) == 3
    r_of = sharding.cdelta_shard_of(n, c, delta)
    for i in range(3):
        assert (np.flatnonzero(r_of == i) + 1).tolist() == g[f"R_{i + 1}"]
    s_of = sharding.m_split_shard_of(r_of, m)
    for i in range(3):
        for x in range(m):
            assert (np.flatnonzero(s_of == m * i + x) + 1).tolist() == g[f"R_{i + 1},{x + 1}"]
    # the plan's sorted per-shard lists reproduce R_{i,x}; the unions are the AttnNode token sets
    plan = oracle.shard_plan(s_of, s_of, 6, 6)
    listed = {k: v for k, v in g.items() if k.startswith("S_")}
    assert len(listed) == 21
    for name, toks in listed.items():
        i, x, j, y = (int(ch) for ch in name[2:])
        a, b = m * (i - 1) + (x - 1), m * (j - 1) + (y - 1)
        sa = plan.q_idx[plan.q_off[a]:plan.q_off[a + 1]]
        sb = plan.kv_idx[plan.kv_off[b]:plan.kv_off[b + 1]]
        assert sorted(set((sa + 1).tolist()) | set((sb + 1).tolist())) == toks
    # the product-side workload generator for block-interleaved maps is the same family
    assert np.array_equal(wl.shard_map("block_rr", n, 3, block=c), r_of)


@pytest.mark.parametrize("c,delta", [(1, 4), (2, 6), (64, 1024), (3, 7), (8, 64)])
def test_cdelta_closed_forms(c, delta):
    alpha = sharding.alpha_of(c, delta)
    assert alpha == -(-delta // c)
    n = 5 * delta
    r_of = sharding.cdelta_shard_of(n, c, delta)
    assert r_of.max() == alpha - 1
    if delta % c == 0:
        assert sharding.cluster_gap(c, delta) == (alpha - 1) * c + 1
    # gap between consecutive clusters of shard 0, measured on the map itself
    members = np.flatnonzero(r_of == 0)
    jumps = np.diff(members)
    assert jumps.max() == sharding.cluster_gap(c, delta)


def _plan_by_sets(q_of, kv_of, nq_s, nkv_s, off, causal):
    """Independent restatement with Python sets / sorted lists."""
    S = [sorted(t for t in range(len(q_of)) if q_of[t] == j) for j in range(nq_s)]
    T = [sorted(t for t in range(len(kv_of)) if kv_of[t] == k) for k in range(nkv_s)]
    q_idx = [t for s in S for t in s]
    vis = [[sum(1 for y in T[k] if (not causal) or y <= x + off) for k in range(nkv_s)] for x in q_idx]
    return S, T, q_idx, vis


def test_plan_brute_force_all_maps_of_8_tokens_into_3_shards():
    for m in itertools.product(range(3), repeat=8):
        m = np.array(m, np.int32)
        plan = oracle.shard_plan(m, m, 3, 3)
        S, T, q_idx, vis = _plan_by_sets(m, m, 3, 3, 0, True)
        assert plan.q_idx.tolist() == q_idx and plan.kv_idx.tolist() == q_idx
        assert plan.q_off.tolist() == np.cumsum([0] + [len(s) for s in S]).tolist()
        assert plan.vis.tolist() == vis
        assert (plan.q_idx[plan.q_inv] == np.arange(8)).all()
        for j in range(3):
            for k in range(3):
                dm = oracle.dense_mask(plan, j, k)
                # structural invariant: every mask row is a prefix of ones (sorted shards, causal mask)
                rows = plan.vis[plan.q_off[j]:plan.q_off[j + 1], k]
                want = (np.arange(len(T[k]))[None, :] < rows[:, None]).astype(np.uint8)
                assert np.array_equal(dm, want)
                if len(S[j]) == 0 or len(T[k]) == 0 or dm.sum() == 0:
                    cls = oracle.EMPTY
                elif dm.all():
                    cls = oracle.FULL
                else:
                    cls = oracle.PARTIAL
                assert plan.pair_class[j, k] == cls


def test_plan_asymmetric_offsets_empty_shards_noncausal():
    rng = np.random.Generator(np.random.PCG64(5))
    for trial in range(50):
        n_q, n_kv = int(rng.integers(1, 40)), int(rng.integers(1, 60))
        nq_s, nkv_s = int(rng.integers(1, 6)), int(rng.integers(1, 9))
        q_of = rng.integers(0, nq_s, n_q).astype(np.int32)
        kv_of = rng.integers(0, nkv_s, n_kv).astype(np.int32)
        off = int(rng.integers(-3, n_kv))
        causal = bool(trial % 3)
        plan = oracle.shard_plan(q_of, kv_of, nq_s, nkv_s, q_pos_offset=off, causal=causal)
        S, T, q_idx, vis = _plan_by_sets(q_of, kv_of, nq_s, nkv_s, off, causal)
        assert plan.q_idx.tolist() == q_idx and plan.vis.tolist() == vis
        assert plan.kv_idx.tolist() == [t for s in T for t in s]
        assert (plan.kv_idx[plan.kv_inv] == np.arange(n_kv)).all()
        # vis is non-decreasing down the rows of a query shard (rows ascend in position)
        for j in range(nq_s):
            blk = plan.vis[plan.q_off[j]:plan.q_off[j + 1]]
            assert (np.diff(blk, axis=0) >= 0).all()
    with pytest.raises(ValueError):
        oracle.shard_plan(np.array([0, 3], np.int32), np.array([0, 1], np.int32), 2, 2)


def test_visible_pair_count_matches_closed_form():
    w = wl.config("c2_prefill_8b", n_q=256, n_kv=256, H=4, Hkv=2)
    plan = oracle.shard_plan(w.q_shard_of, w.kv_shard_of, w.n_q_shards, w.n_kv_shards)
    assert int(plan.vis.sum()) == 256 * 257 // 2 == w.visible_pairs()
    assert w.flops() == 4 * 128 * 4 * (256 * 257 // 2)
