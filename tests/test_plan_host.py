"""cascade_shard_plan's arrays against the oracle's, bit for bit (host-only plan: no GPU needed).
The library builds them with a counting sort and binary searches; the oracle scans the mask definition."""
import numpy as np
import pytest

import oracle
from oracle import sharding
from paper_2507_05228_b200 import workloads as wl


@pytest.fixture(scope="module")
def binding():
    from paper_2507_05228_b200 import build
    build.build_library()
    from paper_2507_05228_b200 import binding as b
    return b


def _compare(binding, q_of, kv_of, nq_s, nkv_s, off, causal):
    ref = oracle.shard_plan(q_of, kv_of, nq_s, nkv_s, q_pos_offset=off, causal=causal)
    plan = binding.cascade_shard_plan_host(q_of, kv_of, nq_s, nkv_s, q_pos_offset=off, causal=causal)
    for f in ("q_off", "q_idx", "q_inv", "kv_off", "kv_idx", "kv_inv", "vis", "pair_class"):
        got = plan.get(f)[0]
        want = getattr(ref, f)
        assert got.dtype == want.dtype and np.array_equal(got, want), f
    return ref, plan


@pytest.mark.parametrize("name", ["c1_tiny_f32", "c2_prefill_8b", "c3_batched", "c5_decode"])
def test_plan_of_benchmark_maps_full_size(binding, name):
    # only the maps matter here: shrink heads/batch so that no large tensor is drawn
    w = wl.config(name, H=1, Hkv=1, B=1, d=8) if name != "c3_batched" else wl.config(name, H=1, Hkv=1, B=1, d=8,
                                                                                        outlier_frac=0.0)
    ref, plan = _compare(binding, w.q_shard_of, w.kv_shard_of, w.n_q_shards, w.n_kv_shards, w.q_pos_offset, True)
    assert int(ref.vis.sum()) * 1 == w.visible_pairs()
    j, k = w.n_q_shards - 1, 0
    assert np.array_equal(plan.dense_mask(j, k), oracle.dense_mask(ref, j, k))
    plan.destroy()


def test_plan_of_long_context_map_full_size(binding):
    w = wl.config("c4_long_70b", H=1, Hkv=1, d=8)
    ref, plan = _compare(binding, w.q_shard_of, w.kv_shard_of, 32, 32, 0, True)
    assert int(ref.vis.sum()) == 536887296
    plan.destroy()


def test_plan_random_maps_edge_cases(binding):
    rng = np.random.Generator(np.random.PCG64(12))
    for trial in range(60):
        n_q, n_kv = int(rng.integers(1, 300)), int(rng.integers(1, 300))
        nq_s, nkv_s = int(rng.integers(1, 9)), int(rng.integers(1, 12))
        q_of = rng.integers(0, nq_s, n_q).astype(np.int32)
        kv_of = rng.integers(0, nkv_s, n_kv).astype(np.int32)
        if trial % 5 == 0:  # leave some shards empty, make one a single token
            q_of[:] = 0
            kv_of[:] = nkv_s - 1
            kv_of[0] = 0
        off = int(rng.integers(-5, n_kv + 5))
        ref, plan = _compare(binding, q_of, kv_of, nq_s, nkv_s, off, causal=bool(trial % 4))
        for j in range(nq_s):
            for k in range(nkv_s):
                assert np.array_equal(plan.dense_mask(j, k), oracle.dense_mask(ref, j, k))
        plan.destroy()


def test_plan_per_sequence_maps_and_paper_example(binding):
    r_of = sharding.cdelta_shard_of(18, 2, 6)
    s_of = sharding.m_split_shard_of(r_of, 2)
    maps = np.stack([s_of, s_of[::-1].copy(), (np.arange(18) % 6).astype(np.int32)])
    plan = binding.cascade_shard_plan_host(maps, maps, 6, 6)
    for i in range(3):
        ref = oracle.shard_plan(maps[i], maps[i], 6, 6)
        assert np.array_equal(plan.get("q_idx")[i], ref.q_idx)
        assert np.array_equal(plan.get("vis")[i], ref.vis)
        assert np.array_equal(plan.get("pair_class")[i], ref.pair_class)
    # Section 6.4 example: shard 0 = R_{1,1} = {1,7,13} (1-based)
    assert (plan.get("q_idx")[0][:3] + 1).tolist() == [1, 7, 13]
    plan.destroy()


def test_partial_buffer_sizes_match_stage_b_cost_model():
    """Appendix D: the partial outputs and statistics sent back are beta * (d + 2) * H * N values."""
    w = wl.config("c2_prefill_8b", B=1, H=1, Hkv=1, d=8)
    beta, d, H, N = 8, 128, 32, 2048
    o_elems = beta * N * H * d
    stat_elems = 2 * beta * N * H
    assert o_elems + stat_elems == beta * (d + 2) * H * N
    assert w.n_kv_shards == beta and w.n_q == N


def test_plan_advance_matches_a_plan_built_at_that_position(binding):
    """Token-sharded KV caching: one plan over the cache capacity, advanced token by token, equals the oracle's plan
    built for each position (prefix lengths and pair classes bit-exact); the index lists never change."""
    n_cap, P = 96, 5
    kv_of = sharding.cdelta_shard_of(n_cap, 4, 20)          # every future slot already has its shard
    q_of = np.zeros(1, np.int32)
    plan = binding.cascade_shard_plan_host(q_of, kv_of, 1, P, q_pos_offset=0)
    kv_idx0 = plan.get("kv_idx").copy()
    for pos in [0, 1, 3, 4, 19, 20, 57, 95, 96, 200, -1, 7]:
        plan.advance(pos)
        ref = oracle.shard_plan(q_of, kv_of, 1, P, q_pos_offset=pos)
        assert np.array_equal(plan.get("vis")[0], ref.vis), pos
        assert np.array_equal(plan.get("pair_class")[0], ref.pair_class), pos
        assert np.array_equal(plan.get("kv_idx"), kv_idx0)
        assert int(plan.get("vis")[0].sum()) == min(max(pos + 1, 0), n_cap)  # exactly the rows written so far
    plan.destroy()
    # a sliding prefill chunk (n_q > 1) and a bidirectional plan (nothing to cut)
    q_chunk = (np.arange(12) % 3).astype(np.int32)
    plan = binding.cascade_shard_plan_host(q_chunk, kv_of, 3, P, q_pos_offset=0)
    for off in (0, 12, 50, 84):
        plan.advance(off)
        ref = oracle.shard_plan(q_chunk, kv_of, 3, P, q_pos_offset=off)
        assert np.array_equal(plan.get("vis")[0], ref.vis) and np.array_equal(plan.get("pair_class")[0], ref.pair_class)
    plan.destroy()
    plan = binding.cascade_shard_plan_host(q_chunk, kv_of, 3, P, causal=False)
    before = plan.get("vis").copy()
    plan.advance(40)
    assert np.array_equal(plan.get("vis"), before)
    plan.destroy()


def test_resident_plans_are_the_columns_of_the_full_plan(binding):
    """A party that keeps only the K/V rows of its own shards (every world-th shard): the plan over those rows, with
    their original positions, must be the full plan restricted to those shards - lists re-indexed to the resident
    rows, prefix lengths and pair classes copied.  Checked against the oracle's plan of the whole sequence, also
    after moving the query block (cascade_plan_advance) and for a bidirectional mask."""
    from paper_2507_05228_b200 import exchange as ex
    rng = np.random.Generator(np.random.PCG64(77))
    for trial in range(24):
        n_q, n_kv = int(rng.integers(1, 200)), int(rng.integers(8, 260))
        J, P = int(rng.integers(1, 6)), int(rng.integers(2, 9))
        world = int(rng.integers(1, P + 1))
        q_of = rng.integers(0, J, n_q).astype(np.int32)
        kv_of = rng.integers(0, P, n_kv).astype(np.int32)
        causal = bool(trial % 5)
        off = int(rng.integers(-3, n_kv))
        ref = oracle.shard_plan(q_of, kv_of, J, P, q_pos_offset=off, causal=causal)
        for rank in range(world):
            tokens, local_of, n_local = ex.resident_kv(kv_of, P, rank, world)
            mine = ex.owned_shards(P, rank, world)
            assert n_local == mine.size
            if tokens.size == 0:
                continue  # a plan needs at least one K/V row
            plan = binding.cascade_shard_plan_resident(q_of, local_of, tokens, J, n_local, q_pos_offset=off,
                                                       causal=causal, host_only=True)
            assert np.array_equal(plan.get("q_idx")[0], ref.q_idx) and np.array_equal(plan.get("q_off")[0], ref.q_off)
            assert np.array_equal(plan.get("vis")[0], ref.vis[:, mine])
            assert np.array_equal(plan.get("pair_class")[0], ref.pair_class[:, mine])
            # the lists hold resident-row indices; through `tokens` they are the full plan's lists of those shards
            kv_off, kv_idx = plan.get("kv_off")[0], plan.get("kv_idx")[0]
            for i, k in enumerate(mine):
                assert np.array_equal(tokens[kv_idx[kv_off[i]:kv_off[i + 1]]], ref.kv_idx[ref.kv_off[k]:ref.kv_off[k + 1]])
            new_off = off + 7
            plan.advance(new_off)
            ref2 = oracle.shard_plan(q_of, kv_of, J, P, q_pos_offset=new_off, causal=causal)
            assert np.array_equal(plan.get("vis")[0], ref2.vis[:, mine])
            assert np.array_equal(plan.get("pair_class")[0], ref2.pair_class[:, mine])
            plan.destroy()


def test_resident_plan_rejects_unordered_positions(binding):
    q_of = np.zeros(4, np.int32)
    kv_of = np.zeros(3, np.int32)
    for bad in ([0, 2, 2], [3, 1, 5], [-1, 0, 1]):
        with pytest.raises(binding.CascadeError) as ei:
            binding.cascade_shard_plan_resident(q_of, kv_of, np.array(bad, np.int32), 1, 1, host_only=True)
        assert ei.value.status == 2
