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


def test_gaps_of_the_paper_example_and_closed_forms():
    """Section 6.2: in a (c, delta)-sequence the distance from one cluster to the next is delta - c + 1, i.e. delta - c
    indices lie between them; Section 6.3: (c, delta)-sharding meets the theorem iff delta - c + 1 >= rho + 1."""
    g = _golden()
    # R_1 = {1,2,7,8,13,14}: three clusters, four unknown tokens between neighbours (delta - c = 4)
    assert sharding.index_set_gaps(g["R_1"]) == {"n_indices": 6, "n_clusters": 3, "min_gap": 4, "max_gap": 4}
    # AttnNode set S_1121 = {1,3,7,9,13,15}: six singletons, gaps 1,3,1,3,1
    assert sharding.index_set_gaps(g["S_1121"]) == {"n_indices": 6, "n_clusters": 6, "min_gap": 1, "max_gap": 3}
    # S_1112 = R_1 (both halves of one hidden shard) and a single cluster has no gap
    assert sharding.index_set_gaps(g["S_1112"]) == sharding.index_set_gaps(g["R_1"])
    assert sharding.index_set_gaps([4, 5, 6])["min_gap"] == -1 and sharding.index_set_gaps([])["n_clusters"] == 0
    # colluding CompNodes 1 and 2 pool {1,2,3,4,7,8,9,10,...}: clusters of 4, gaps of 2
    union = g["R_1"] + g["R_2"]
    assert sharding.index_set_gaps(union) == {"n_indices": 12, "n_clusters": 3, "min_gap": 2, "max_gap": 2}
    for c, delta, n in [(2, 6, 18), (8, 64, 512), (3, 10, 100), (1, 5, 23), (8, 96, 1000)]:
        r_of = sharding.cdelta_shard_of(n, c, delta)
        for i in range(sharding.alpha_of(c, delta)):
            held = np.flatnonzero(r_of == i)
            gp = sharding.index_set_gaps(held)
            if i >= delta // c:  # c does not divide delta: the last shard's clusters are cut to delta mod c tokens
                assert gp["n_clusters"] < 2 or gp["min_gap"] == gp["max_gap"] == delta - delta % c
                continue
            if gp["n_clusters"] > 1:
                assert gp["min_gap"] == gp["max_gap"] == delta - c == sharding.cluster_gap(c, delta) - 1
            for rho in range(1, delta + 2):
                if gp["n_clusters"] > 1:
                    assert sharding.secure_hidden_state_criterion(held, rho) == (delta - c + 1 >= rho)
                    assert sharding.secure_full_criterion(held, rho) == (delta - c + 1 >= rho + 1)


def test_kl_gaps_follow_the_proof_of_the_theorem():
    g = _golden()
    r_of = sharding.cdelta_shard_of(18, 2, 6)
    s_of = sharding.m_split_shard_of(r_of, 2)
    R1 = [t - 1 for t in g["R_1"]]  # 0-based
    # without m-split (S = R): between 2 and 7 (1-based) lie {3,4} of R_2 and {5,6} of R_3; R_1's own shard adds nothing
    assert sharding.kl_gaps(R1, r_of, 3).tolist() == [-1, 2, 2]
    # with the m = 2 split every foreign KV shard contributes one token per gap; R_1's own pieces none
    assert sharding.kl_gaps(R1, s_of, 6).tolist() == [-1, -1, 1, 1, 1, 1]
    # brute force over all index pairs on random sets
    rng = np.random.default_rng(0)
    for _ in range(50):
        n = int(rng.integers(2, 30))
        s_map = rng.integers(0, 3, n)
        held = np.flatnonzero(rng.random(n) < 0.4)
        got = sharding.kl_gaps(held, s_map, 3)
        for k in range(3):
            sizes = []
            hs = sorted(held.tolist())
            for a, b in zip(hs[:-1], hs[1:]):
                cnt = sum(1 for t in range(a + 1, b) if s_map[t] == k)  # nothing between neighbours is held
                if cnt:
                    sizes.append(cnt)
            assert got[k] == (min(sizes) if sizes else -1)
