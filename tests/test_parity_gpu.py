"""GPU parity: the CUDA library through its C ABI against the fp64 oracle, element by element.

Tolerances (max-abs on unit-variance Gaussian inputs with 1/sqrt(d) scaling): 2e-2 for bf16, 1e-4 for fp32,
on partial outputs, merged outputs and fused outputs; same absolute bound on m and on m + ln l, relative bound
|dl| <= tol * max(1, l) on l.  Plan arrays are compared bit-exactly.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2507_05228_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def gu():
    import gpu_util
    return gpu_util


def test_c1_tiny_fp32_full(gu):
    gu.full_parity(wl.config("c1_tiny_f32"))


def test_c2_prefill_8b_full(gu):
    gu.full_parity(wl.config("c2_prefill_8b"))


def test_c3_batched_reduced_and_outliers(gu):
    gu.full_parity(wl.config("c3_batched", B=2, n_q=1024, n_kv=1024))


def test_c3_batched_full_size_sampled(gu):
    """Full size, in the launch configuration the benchmark times; at least 1024 query rows (every batch entry, all
    heads) go through the oracle."""
    gu.sampled_parity(wl.config("c3_batched"), per_shard=56, min_rows=1024)


def test_c4_long_reduced(gu):
    gu.full_parity(wl.config("c4_long_70b", n_q=2048, n_kv=2048, H=16, Hkv=2))


def test_c4_long_full_size_sampled(gu):
    gu.sampled_parity(wl.config("c4_long_70b"), per_shard=19, min_rows=1024)


def test_all_rows_in_the_grid_order_of_large_problems(gu):
    """More CTAs than eight per SM switch the tensor-core kernel to its other block-index decoding (head group
    slowest); every row of such a launch goes through the oracle."""
    w = wl.config("c2_prefill_8b", B=3, n_q=4096, n_kv=4096)
    assert (4096 // 64) * (w.H // 4) * w.B > 8 * 148
    gu.full_parity(w)


def test_c5_decode_full(gu):
    gu.full_parity(wl.config("c5_decode"))


@pytest.mark.parametrize("dtype,d", [("f32", 64), ("f32", 128), ("bf16", 64), ("bf16", 128)])
@pytest.mark.parametrize("H,Hkv", [(4, 4), (8, 2), (8, 1)])
def test_ragged_shards_all_dtypes(gu, dtype, d, H, Hkv):
    """Shard sizes from 1 to ~130 rows, N not a multiple of any tile, asymmetric query/KV maps, rows that see
    nothing of some shard, an empty shard."""
    rng = np.random.Generator(np.random.PCG64(d + H))
    n = 517
    sizes = [1, 2, 31, 33, 127, 129, 130, 64]  # sums to 517; shard 8 stays empty
    assert sum(sizes) == n
    kv_of = np.repeat(np.arange(8), sizes).astype(np.int32)
    rng.shuffle(kv_of)
    q_of = rng.integers(0, 5, n).astype(np.int32)
    w = wl.make_workload("ragged", 2, n, n, H, Hkv, d, dtype, "random", "random", 5, 9, seed=77)
    w.q_shard_of, w.kv_shard_of = q_of, kv_of
    gu.full_parity(w)


def test_contiguous_shards_have_empty_and_full_pairs(gu):
    w = wl.make_workload("contig", 1, 640, 640, 8, 2, 128, "bf16", "contiguous", "contiguous", 5, 5, seed=5)
    p = oracle.shard_plan(w.q_shard_of, w.kv_shard_of, 5, 5)
    assert (p.pair_class == oracle.EMPTY).any() and (p.pair_class == oracle.FULL).any()
    gu.full_parity(w)


def test_non_causal_and_single_shard(gu):
    gu.full_parity(wl.make_workload("bert_like", 2, 128, 128, 12, 12, 64, "f32", "round_robin", "round_robin",
                                    4, 4, seed=3, causal=False))
    gu.full_parity(wl.make_workload("one_shard", 1, 300, 300, 4, 2, 128, "bf16", "random", "random", 1, 1, seed=4))


def test_non_causal_on_the_tensor_core_route(gu):
    """Bidirectional mask (the BERT case) in bf16 with head_dim 128: every key of every shard is visible."""
    gu.full_parity(wl.make_workload("bidir_tc", 2, 384, 384, 8, 2, 128, "bf16", "random", "random", 3, 3, seed=15,
                                    causal=False))
    gu.full_parity(wl.make_workload("bidir_tc_cross", 1, 100, 700, 4, 4, 128, "bf16", "round_robin", "block_rr", 2, 5,
                                    seed=16, causal=False, block=16))


def test_chunked_prefill_offsets(gu):
    """n_q < n_kv with the query block at the end of the cache, and a block in the middle."""
    gu.full_parity(wl.make_workload("chunk_end", 2, 96, 400, 8, 2, 128, "bf16", "random", "random", 3, 7, seed=8))
    gu.full_parity(wl.make_workload("chunk_mid", 1, 50, 333, 4, 4, 64, "f32", "round_robin", "random", 2, 5,
                                    seed=9, q_pos_offset=100))


@pytest.mark.parametrize("H,Hkv", [(8, 8), (8, 4), (32, 8), (16, 2)])
def test_decode_group_sizes_and_ragged_cache(gu, H, Hkv):
    w = wl.make_workload("decode_small", 3, 1, 1000, H, Hkv, 128, "bf16", "round_robin", "random", 1, 7, seed=H)
    gu.full_parity(w)
    # cache not fully visible (query position in the middle) and a shard with nothing visible
    w2 = wl.make_workload("decode_partial", 2, 1, 500, H, Hkv, 128, "bf16", "round_robin", "contiguous", 1, 5,
                          seed=H + 1, q_pos_offset=250)
    gu.full_parity(w2)


def test_per_sequence_maps_and_strided_inputs(gu):
    from paper_2507_05228_b200 import binding as cb
    B, n, H, Hkv, d = 3, 200, 8, 2, 128
    w = wl.make_workload("perseq", B, n, n, H, Hkv, d, "bf16", "random", "random", 4, 4, seed=21)
    rng = np.random.Generator(np.random.PCG64(5))
    maps = np.stack([wl.shard_map("random", n, 4, rng) for _ in range(B)])
    q, k, v = gu.to_device(w)
    # pack q, k, v into one [B, n, H + 2 Hkv, d] tensor: strided views, as a fused QKV projection would give
    packed = torch.cat([q, k, v], dim=2).contiguous()
    qv, kv, vv = packed[:, :, :H], packed[:, :, H:H + Hkv], packed[:, :, H + Hkv:]
    plan = cb.cascade_shard_plan(maps, maps, 4, 4)
    o_part, m_part, l_part = cb.cascade_attn_partials(plan, qv, kv, vv, w.scale)
    o_m, _ = cb.cascade_merge(o_part, m_part, l_part, plan.dev_ptr("q_idx"), row_scatter_batch_stride=n)
    o_f, lse_f = cb.cascade_attn_sharded(plan, qv, kv, vv, w.scale)
    o_ref, lse_ref = oracle.attention_unsharded(w.q, w.k, w.v, w.scale)
    gu.check_output(o_m, None, o_ref, lse_ref, w.tol, "per-sequence maps merge", stored_partials=True)
    gu.check_output(o_f, lse_f, o_ref, lse_ref, w.tol, "per-sequence maps fused")
    for b in range(B):
        op = oracle.shard_plan(maps[b], maps[b], 4, 4)
        u, m, e = oracle.attn_pass(w.q[b:b + 1], w.k[b:b + 1], w.v[b:b + 1], w.scale, op)
        gu.check_partials((o_part[b:b + 1].double().cpu().numpy(), m_part[b:b + 1].double().cpu().numpy(),
                           l_part[b:b + 1].double().cpu().numpy()), (u, m, e), w.tol, f"per-sequence maps b={b}")
    assert plan.device_status() == 0
    plan.destroy()


def test_merge_alone_matches_oracle_post_pass(gu):
    """cascade_merge on synthetic partials (no attention involved), including empty parts and huge maxima."""
    from paper_2507_05228_b200 import binding as cb
    rng = np.random.Generator(np.random.PCG64(31))
    for dtype, d, tol in ((torch.float32, 64, 1e-4), (torch.bfloat16, 128, 2e-2), (torch.float32, 128, 1e-4),
                          (torch.bfloat16, 64, 2e-2)):
        B, P, R, H = 2, 7, 37, 5
        u = rng.standard_normal((B, P, R, H, d)).astype(np.float32)
        if dtype == torch.bfloat16:
            u = wl.round_to_bf16(u)
        m = (rng.standard_normal((B, P, R, H)) * 30).astype(np.float32)
        l = rng.uniform(1, 40, (B, P, R, H)).astype(np.float32)
        dead = rng.random((B, P, R, H)) < 0.2
        dead[0, :, 3, 1] = True  # a row whose parts are all empty
        m[dead], l[dead] = -np.inf, 0.0
        u[dead] = 0.0
        scatter = rng.permutation(R).astype(np.int32)
        o_ref, lse_ref = oracle.post_pass(u.astype(np.float64), m.astype(np.float64), l.astype(np.float64),
                                          row_scatter=scatter)
        sc = torch.from_numpy(scatter).cuda()
        o, lse = cb.cascade_merge(torch.from_numpy(u).cuda().to(dtype), torch.from_numpy(m).cuda(),
                                  torch.from_numpy(l).cuda(), sc.data_ptr())
        gu.check_output(o, lse, o_ref, lse_ref, tol, f"merge {dtype} d={d}")
        assert (o[0, scatter[3], 1] == 0).all() and torch.isneginf(lse[0, scatter[3], 1])


def test_workspace_contract_for_decode(gu):
    from paper_2507_05228_b200 import binding as cb
    w = wl.make_workload("decode_ws", 2, 1, 256, 8, 2, 128, "bf16", "round_robin", "random", 1, 4, seed=2)
    q, k, v = gu.to_device(w)
    plan = gu.make_plan(w)
    need = cb.cascade_workspace_bytes(plan, cb.CALL_SHARDED, cb.BF16, 2, 8, 2, 128)
    assert need >= 2 * 4 * 8 * (128 * 2 + 8)
    small = torch.empty(need - 256, dtype=torch.uint8, device="cuda")
    with pytest.raises(cb.CascadeError) as ei:
        cb.cascade_attn_sharded(plan, q, k, v, w.scale, workspace=small)
    assert ei.value.status == 4
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    o, _ = cb.cascade_attn_sharded(plan, q, k, v, w.scale, workspace=ws)
    o_ref, lse_ref = oracle.attention_unsharded(w.q, w.k, w.v, w.scale, q_pos_offset=w.q_pos_offset)
    gu.check_output(o, None, o_ref, lse_ref, w.tol, "decode with caller workspace")
    plan.destroy()


def test_many_small_shards_tiles_span_several_shards(gu):
    """64 shards of 16 keys: every 32-key chunk of the KV stream is half empty and an MMA tile takes its four chunks
    from four different shards; 300 shards exceed the tensor-core kernel's shard table and take the ALU kernel."""
    gu.full_parity(wl.make_workload("shards64", 1, 1024, 1024, 8, 2, 128, "bf16", "random", "random", 64, 64, seed=11))
    gu.full_parity(wl.make_workload("shards300", 1, 600, 600, 4, 2, 128, "bf16", "random", "random", 300, 300,
                                    seed=12))


def test_tensor_core_route_workspace_contract_and_unaligned_output(gu):
    from paper_2507_05228_b200 import binding as cb
    w = wl.make_workload("ws_tc", 2, 300, 300, 8, 2, 128, "bf16", "random", "random", 3, 3, seed=13)
    q, k, v = gu.to_device(w)
    plan = gu.make_plan(w)
    need = cb.cascade_workspace_bytes(plan, cb.CALL_SHARDED, cb.BF16, 2, 8, 2, 128)
    assert need == cb.cascade_workspace_bytes(plan, cb.CALL_PARTIALS, cb.BF16, 2, 8, 2, 128)
    assert need >= 2 * 2 * 2 * 300 * 256  # shard-major K and V copies
    small = torch.empty(need - 256, dtype=torch.uint8, device="cuda")
    for call in (cb.cascade_attn_sharded, cb.cascade_attn_partials):
        with pytest.raises(cb.CascadeError) as ei:
            call(plan, q, k, v, w.scale, workspace=small)
        assert ei.value.status == 4
    # an output whose rows are 16- but not 32-byte aligned (the interface asks for 16; the row copies need no more)
    flat = torch.zeros(q.numel() + 8, dtype=torch.bfloat16, device="cuda")
    o_view = flat[8:].view(q.shape)
    assert o_view.data_ptr() % 32 == 16
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    o, lse = cb.cascade_attn_sharded(plan, q, k, v, w.scale, out=o_view, workspace=ws)
    o_ref, lse_ref = oracle.attention_unsharded(w.q, w.k, w.v, w.scale)
    gu.check_output(o, lse, o_ref, lse_ref, w.tol, "unaligned output")
    assert (flat[:8] == 0).all()
    assert plan.device_status() == 0
    plan.destroy()


def test_kernel_timing_counts_attention_launches(gu):
    from paper_2507_05228_b200 import binding as cb
    w = wl.make_workload("timing", 1, 256, 256, 8, 2, 128, "bf16", "random", "random", 2, 2, seed=14)
    q, k, v = gu.to_device(w)
    plan = gu.make_plan(w)
    cb.cascade_attn_sharded(plan, q, k, v, w.scale)  # not timed
    cb.cascade_kernel_timing_begin()
    for _ in range(3):
        cb.cascade_attn_sharded(plan, q, k, v, w.scale)
    ms, n = cb.cascade_kernel_timing_end()
    assert n == 3 and 0.0 < ms < 100.0
    cb.cascade_attn_sharded(plan, q, k, v, w.scale)  # recording is off again
    ms2, n2 = cb.cascade_kernel_timing_end()
    assert n2 == 0 and ms2 == 0.0
    plan.destroy()


def test_plan_advance_on_the_device_matches_a_plan_built_at_that_position(gu):
    """cascade_plan_advance on a device plan rewrites vis and pair_class with kernels: the device arrays (read through
    the pointers cascade_plan_get returns), and the host copies refreshed on demand, equal the oracle's plan built for
    each position, bit for bit; positions before 0 and past the capacity, several maps, a sliding chunk, a
    bidirectional plan."""
    from paper_2507_05228_b200 import binding as cb
    from oracle import sharding
    n_cap, P = 1000, 7
    kv_of = np.stack([sharding.cdelta_shard_of(n_cap, 4, 28),
                      np.random.default_rng(5).integers(0, P, n_cap).astype(np.int32)])
    q_of = np.zeros((2, 1), np.int32)
    plan = cb.cascade_shard_plan(q_of, kv_of, 1, P, q_pos_offset=0)
    for pos in [0, 1, 27, 28, 511, 999, 1000, 5000, -3, 77]:
        plan.advance(pos)
        for mp in range(2):
            ref = oracle.shard_plan(q_of[mp], kv_of[mp], 1, P, q_pos_offset=pos)
            assert np.array_equal(gu.read_plan_device_array(plan, "vis")[mp], ref.vis), (pos, mp)
            assert np.array_equal(gu.read_plan_device_array(plan, "pair_class")[mp], ref.pair_class), (pos, mp)
            assert np.array_equal(plan.get("vis")[mp], ref.vis) and np.array_equal(plan.get("pair_class")[mp], ref.pair_class)
    plan.destroy()
    # more than 256 (row, shard) entries: the kernels; two maps with different query and KV shardings
    q_chunk = np.stack([(np.arange(96) % 3), np.random.default_rng(6).integers(0, 3, 96)]).astype(np.int32)
    for causal in (True, False):
        plan = cb.cascade_shard_plan(q_chunk, kv_of, 3, P, q_pos_offset=0, causal=causal)
        for off in (0, 96, 500, 904, 950, -40):
            plan.advance(off)
            for mp in range(2):
                ref = oracle.shard_plan(q_chunk[mp], kv_of[mp], 3, P, q_pos_offset=off, causal=causal)
                assert np.array_equal(gu.read_plan_device_array(plan, "vis")[mp], ref.vis), (causal, off, mp)
                assert np.array_equal(gu.read_plan_device_array(plan, "pair_class")[mp], ref.pair_class), (causal, off)
                # the host copies are refreshed by whichever call reads them first
                assert np.array_equal(plan.dense_mask(1, 2, map=mp), oracle.dense_mask(ref, 1, 2))
                assert np.array_equal(plan.get("vis")[mp], ref.vis)
        plan.destroy()


def test_decode_loop_over_a_preallocated_cache_with_plan_advance(gu):
    """Token-sharded KV caching (Appendix F): one plan over the cache capacity, advanced per generated token.  Rows of
    the cache beyond the current position hold arbitrary finite values and must not influence the result."""
    from paper_2507_05228_b200 import binding as cb
    cap, B, H, Hkv, d, P = 640, 2, 8, 2, 128, 5
    w = wl.make_workload("cache", B, 1, cap, H, Hkv, d, "bf16", "round_robin", "block_rr", 1, P, seed=41, block=8,
                         q_pos_offset=0)
    q, k, v = gu.to_device(w)
    plan = gu.make_plan(w)
    steps = [0, 1, 7, 8, 63, 300, 639]
    for pos in steps:
        plan.advance(pos)
        # poison everything the new token must not see
        k_p, v_p = k.clone(), v.clone()
        if pos + 1 < cap:
            k_p[:, pos + 1:] = 3.0e4
            v_p[:, pos + 1:] = -3.0e4
        o, lse = cb.cascade_attn_sharded(plan, q, k_p, v_p, w.scale)
        o_ref, lse_ref = oracle.attention_unsharded(w.q, w.k, w.v, w.scale, causal=True, q_pos_offset=pos)
        gu.check_output(o, lse, o_ref, lse_ref, w.tol, f"decode at position {pos}")
        assert int(plan.get("vis")[0].sum()) == pos + 1
    # a sliding prefill chunk on the tensor-core route
    w2 = wl.make_workload("chunk_slide", 1, 64, 512, 8, 2, 128, "bf16", "round_robin", "block_rr", 2, 4, seed=42,
                          block=16, q_pos_offset=0)
    q, k, v = gu.to_device(w2)
    plan2 = gu.make_plan(w2)
    for off in (0, 64, 200, 448):
        plan2.advance(off)
        o, lse = cb.cascade_attn_sharded(plan2, q, k, v, w2.scale)
        o_ref, lse_ref = oracle.attention_unsharded(w2.q, w2.k, w2.v, w2.scale, causal=True, q_pos_offset=off)
        gu.check_output(o, lse, o_ref, lse_ref, w2.tol, f"prefill chunk at offset {off}")
    assert plan.device_status() == 0 and plan2.device_status() == 0
    plan.destroy()
    plan2.destroy()


@pytest.mark.parametrize("dtype,d,n_q", [("bf16", 128, 64), ("bf16", 128, 1), ("f32", 64, 48)])
def test_unwritten_cache_tail_may_hold_nan(gu, dtype, d, n_q):
    """A preallocated cache whose rows beyond the last query position were never written (NaN bit patterns here) must not
    leak into the result on any route: tensor cores (whole 32-key chunks are loaded, rows past a prefix get weight 0,
    and 0 x NaN would poison the output), decode and the ALU kernel."""
    from paper_2507_05228_b200 import binding as cb
    cap, B, H, Hkv, P = 512, 2, 8, 2, 4
    w = wl.make_workload("nan_tail", B, n_q, cap, H, Hkv, d, dtype, "round_robin", "block_rr", 2 if n_q > 1 else 1, P,
                         seed=51, block=8, q_pos_offset=0)
    q, k, v = gu.to_device(w)
    plan = gu.make_plan(w)
    for off in (0, 100, cap - n_q):
        plan.advance(off)
        last = off + n_q - 1
        k_p, v_p = k.clone(), v.clone()
        if last + 1 < cap:
            k_p[:, last + 1:] = float("nan")
            v_p[:, last + 1:] = float("nan")
        o_ref, lse_ref = oracle.attention_unsharded(w.q, w.k, w.v, w.scale, causal=True, q_pos_offset=off)
        o, lse = cb.cascade_attn_sharded(plan, q, k_p, v_p, w.scale)
        gu.check_output(o, lse, o_ref, lse_ref, w.tol, f"fused, NaN tail after position {last}")
        o_part, m_part, l_part = cb.cascade_attn_partials(plan, q, k_p, v_p, w.scale)
        assert torch.isfinite(o_part.float()).all() and not torch.isnan(m_part).any() and torch.isfinite(l_part).all()
        o_m, lse_m = cb.cascade_merge(o_part, m_part, l_part, plan.dev_ptr("q_idx"))
        gu.check_output(o_m, lse_m, o_ref, lse_ref, w.tol, f"merge, NaN tail after position {last}",
                        stored_partials=True)
    assert plan.device_status() == 0
    plan.destroy()


def test_scale_must_be_positive_and_finite(gu):
    from paper_2507_05228_b200 import binding as cb
    w = wl.make_workload("scale", 1, 64, 64, 4, 2, 128, "bf16", "random", "random", 2, 2, seed=52)
    q, k, v = gu.to_device(w)
    plan = gu.make_plan(w)
    for bad in (0.0, -0.5, float("inf"), float("nan")):
        for call in (cb.cascade_attn_sharded, cb.cascade_attn_partials):
            with pytest.raises(cb.CascadeError) as ei:
                call(plan, q, k, v, bad)
            assert ei.value.status == 1
    plan.destroy()


@pytest.mark.parametrize("shape", ["tc", "tc_walk_ragged", "decode", "alu"])
def test_outputs_stay_inside_their_buffers(gu, shape):
    """Every output buffer is carved out of a larger allocation whose surroundings hold a pattern; after partials,
    merge and the fused call the pattern must be intact on both sides (the stand-in for a memory checker)."""
    from paper_2507_05228_b200 import binding as cb
    w = {"tc": wl.make_workload("canary_tc", 2, 200, 200, 8, 2, 128, "bf16", "random", "random", 3, 3, seed=81),
         "tc_walk_ragged": wl.make_workload("canary_walk", 1, 333, 333, 4, 1, 128, "bf16", "random", "contiguous", 2, 7,
                                            seed=82),
         "decode": wl.make_workload("canary_dec", 3, 1, 500, 8, 2, 128, "bf16", "round_robin", "random", 1, 6, seed=83),
         "alu": wl.make_workload("canary_alu", 2, 70, 90, 4, 2, 64, "f32", "random", "random", 2, 3, seed=84)}[shape]
    q, k, v = gu.to_device(w)
    plan = gu.make_plan(w)
    pad = 1024  # elements of padding on each side

    def guarded(shape_, dtype, fill):
        n = int(np.prod(shape_))
        raw = torch.full((n + 2 * pad,), fill, dtype=dtype, device="cuda")
        return raw, raw[pad:pad + n].view(shape_)

    B, n_q, H, d, P = w.B, w.n_q, w.H, w.d, w.n_kv_shards
    bufs = {"o_part": guarded((B, P, n_q, H, d), q.dtype, 7.0), "m_part": guarded((B, P, n_q, H), torch.float32, 7.0),
            "l_part": guarded((B, P, n_q, H), torch.float32, 7.0), "o": guarded((B, n_q, H, d), q.dtype, 7.0)}
    code = cb.BF16 if w.dtype == "bf16" else cb.F32
    ws_bytes = max(cb.cascade_workspace_bytes(plan, cb.CALL_SHARDED, code, B, H, w.Hkv, d),
                   cb.cascade_workspace_bytes(plan, cb.CALL_PARTIALS, code, B, H, w.Hkv, d), 256)
    ws_raw = torch.full((ws_bytes + 2 * 4096,), 0x5A, dtype=torch.uint8, device="cuda")
    off = ((ws_raw.data_ptr() + 2048 + 255) // 256) * 256 - ws_raw.data_ptr()
    ws = ws_raw[off:off + ws_bytes]
    parts = (bufs["o_part"][1], bufs["m_part"][1], bufs["l_part"][1])
    cb.cascade_attn_partials(plan, q, k, v, w.scale, out=parts, workspace=ws)
    cb.cascade_merge(*parts, plan.dev_ptr("q_idx"), out=bufs["o"][1], want_lse=False)
    cb.cascade_attn_sharded(plan, q, k, v, w.scale, out=bufs["o"][1], want_lse=False, workspace=ws)
    torch.cuda.synchronize()
    for name, (raw, view) in bufs.items():
        n = view.numel()
        assert (raw[:pad] == 7.0).all() and (raw[pad + n:] == 7.0).all(), f"{name}: written outside the buffer"
        assert torch.isfinite(view.float()).all() or name == "m_part"
    assert (ws_raw[:off] == 0x5A).all() and (ws_raw[off + ws_bytes:] == 0x5A).all(), "workspace overrun"
    o_ref, _ = oracle.attention_unsharded(w.q, w.k, w.v, w.scale, causal=w.causal, q_pos_offset=w.q_pos_offset)
    gu.check_output(bufs["o"][1], None, o_ref, None, w.tol, "fused into a guarded buffer")
    assert plan.device_status() == 0
    plan.destroy()


def test_merge_peers_matches_oracle_post_pass_on_split_sources(gu):
    """cascade_merge_peers on synthetic partials split over three sources with different part counts (one of them
    empty-handed), gathering a subset of rows in a scrambled order; reference: the oracle's post-pass over all parts."""
    from paper_2507_05228_b200 import binding as cb
    rng = np.random.Generator(np.random.PCG64(33))
    for dtype, d, tol in ((torch.bfloat16, 128, 2e-2), (torch.float32, 64, 1e-4)):
        B, P, R, H = 2, 7, 41, 3
        u = rng.standard_normal((B, P, R, H, d)).astype(np.float32)
        if dtype == torch.bfloat16:
            u = wl.round_to_bf16(u)
        m = (rng.standard_normal((B, P, R, H)) * 20).astype(np.float32)
        l = rng.uniform(1, 30, (B, P, R, H)).astype(np.float32)
        dead = rng.random((B, P, R, H)) < 0.25
        dead[1, :, 5, 2] = True  # a row whose parts are all empty
        m[dead], l[dead] = -np.inf, 0.0
        u[dead] = 0.0
        split = [[0, 3, 4], [1, 6], [2, 5]]  # which parts each source holds, in its own order
        rows = rng.permutation(R)[:17].astype(np.int32)
        order = [k for s in split for k in s]
        o_ref, lse_ref = oracle.post_pass(u[:, order][:, :, rows].astype(np.float64), m[:, order][:, :, rows].astype(np.float64),
                                          l[:, order][:, :, rows].astype(np.float64))
        sources = [(torch.from_numpy(u[:, s]).cuda().to(dtype).contiguous(), torch.from_numpy(m[:, s]).cuda().contiguous(),
                    torch.from_numpy(l[:, s]).cuda().contiguous()) for s in split]
        o, lse = cb.cascade_merge_peers(sources, torch.from_numpy(rows).cuda(), rows.size)
        gu.check_output(o, lse, o_ref, lse_ref, tol, f"merge_peers {dtype}")
        where = int(np.flatnonzero(rows == 5)[0]) if (rows == 5).any() else None
        if where is not None:
            assert (o[1, where, 2] == 0).all() and torch.isneginf(lse[1, where, 2])
        # identity gather over all rows == cascade_merge on the concatenated parts
        o_all, lse_all = cb.cascade_merge_peers(sources, None, R)
        o_m, lse_m = cb.cascade_merge(torch.from_numpy(u[:, order]).cuda().to(dtype).contiguous(),
                                      torch.from_numpy(m[:, order]).cuda().contiguous(),
                                      torch.from_numpy(l[:, order]).cuda().contiguous())
        # (the two kernels add the parts in different orders: equal up to fp32 summation order, then one rounding)
        step = 2.0 ** -7 if dtype == torch.bfloat16 else 1e-5
        assert ((o_all.float() - o_m.float()).abs() <= step * o_m.float().abs().clamp(min=1.0)).all()
        assert torch.allclose(torch.nan_to_num(lse_all, neginf=-1e30), torch.nan_to_num(lse_m, neginf=-1e30), atol=1e-5)
    with pytest.raises(cb.CascadeError):
        cb.cascade_merge_peers(sources * 6, None, R)  # 18 sources: more than the kernel's table holds


@pytest.mark.parametrize("seed", [101, 102, 103])
def test_random_shapes_on_every_route(gu, seed):
    """Seeded random problems: sizes that are no multiple of any tile, shard counts from 1 to 9 with every map kind,
    query blocks anywhere in the cache, both masks, several head groupings - every element of plan, partials, merge and
    fused output against the oracle.  Twelve problems per seed; which route runs follows from the shape."""
    rng = np.random.Generator(np.random.PCG64(seed))
    kinds = ["random", "contiguous", "round_robin", "block_rr"]
    heads = [(4, 4), (8, 2), (8, 1), (16, 2), (2, 1), (6, 2)]
    for trial in range(12):
        dtype, d = [("bf16", 128), ("bf16", 128), ("bf16", 128), ("f32", 64), ("bf16", 64), ("f32", 128)][trial % 6]
        H, Hkv = heads[int(rng.integers(len(heads)))]
        B = int(rng.integers(1, 3))
        n_q = 1 if trial % 6 == 2 and rng.random() < 0.5 else int(rng.integers(2, 420))
        n_kv = int(rng.integers(n_q, 640))
        J = 1 if n_q == 1 else int(rng.integers(1, 7))
        P = int(rng.integers(1, 10))
        causal = bool(rng.random() < 0.8)
        off = n_kv - n_q if rng.random() < 0.6 else int(rng.integers(0, n_kv - n_q + 1))
        w = wl.make_workload(f"fuzz{seed}_{trial}", B, n_q, n_kv, H, Hkv, d, dtype, kinds[int(rng.integers(4))],
                             kinds[int(rng.integers(4))], J, P, seed=1000 * seed + trial,
                             block=int(rng.choice([4, 16, 64])), causal=causal, q_pos_offset=off, symmetric=False)
        gu.full_parity(w)
