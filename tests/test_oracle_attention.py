"""Pins for the CPU oracle's floating-point functions (no GPU).

Each test checks the oracle against something other than itself: a library routine on a special case,
a closed form, an identity the paper states, or brute force on tiny inputs.
"""
import itertools
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2507_05228_b200 import workloads as wl


def _rand(B, n_q, n_kv, H, Hkv, d, seed, std=1.0):
    rng = np.random.Generator(np.random.PCG64(seed))
    q = (rng.standard_normal((B, n_q, H, d)) * std).astype(np.float32)
    k = (rng.standard_normal((B, n_kv, Hkv, d)) * std).astype(np.float32)
    v = rng.standard_normal((B, n_kv, Hkv, d)).astype(np.float32)
    return q, k, v


def _sdpa_fp64(q, k, v, scale, causal):
    """torch's scaled_dot_product_attention in fp64 on CPU: a library routine for the unsharded case."""
    H, Hkv = q.shape[2], k.shape[2]
    tq = torch.from_numpy(q).double().permute(0, 2, 1, 3)
    tk = torch.from_numpy(k).double().permute(0, 2, 1, 3).repeat_interleave(H // Hkv, dim=1)
    tv = torch.from_numpy(v).double().permute(0, 2, 1, 3).repeat_interleave(H // Hkv, dim=1)
    o = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=causal, scale=scale)
    return o.permute(0, 2, 1, 3).numpy()


@pytest.mark.parametrize("causal", [True, False])
@pytest.mark.parametrize("H,Hkv,d", [(4, 4, 16), (8, 2, 32), (6, 1, 8)])
def test_unsharded_matches_library_sdpa(causal, H, Hkv, d):
    q, k, v = _rand(2, 37, 37, H, Hkv, d, seed=5)
    scale = 1.0 / math.sqrt(d)
    o, lse = oracle.attention_unsharded(q, k, v, scale, causal=causal)
    ref = _sdpa_fp64(q, k, v, scale, causal)
    assert np.abs(o - ref).max() < 1e-12
    # lse against torch.logsumexp of explicitly built logits
    G = H // Hkv
    a = np.einsum("bihc,bjhc->bhij", q.astype(np.float64), np.repeat(k, G, axis=2).astype(np.float64)) * scale
    if causal:
        a = np.where(np.tril(np.ones((37, 37), bool))[None, None], a, -np.inf)
    ref_lse = torch.logsumexp(torch.from_numpy(a), dim=-1).numpy().transpose(0, 2, 1)
    # The library routine itself wanders: about one process in twenty returns values 1e-9 away from its usual ones (and
    # from the max-subtracted sum written out below, which the oracle matches to 1e-15 every time), depending on how
    # the buffer happens to be aligned.  Any mistake in the oracle's statistic would show at 1e-3 or more.
    assert np.abs(lse - ref_lse).max() < 1e-8
    m = a.max(-1, keepdims=True)
    direct = (m[..., 0] + np.log(np.exp(a - m).sum(-1))).transpose(0, 2, 1)
    assert np.abs(lse - direct).max() < 1e-12


def _brute_force(q, k, v, scale, causal, q_pos_offset=0):
    """Direct definition in pure Python: exp without max subtraction (inputs are small)."""
    B, n_q, H, d = q.shape
    n_kv, Hkv = k.shape[1], k.shape[2]
    G = H // Hkv
    o = np.zeros((B, n_q, H, d))
    for b in range(B):
        for i in range(n_q):
            for h in range(H):
                num = [0.0] * d
                den = 0.0
                for y in range(n_kv):
                    if causal and y > i + q_pos_offset:
                        continue
                    a = sum(float(q[b, i, h, c]) * float(k[b, y, h // G, c]) for c in range(d)) * scale
                    w = math.exp(a)
                    den += w
                    for c in range(d):
                        num[c] += w * float(v[b, y, h // G, c])
                o[b, i, h] = [x / den for x in num] if den > 0 else 0.0
    return o


def test_brute_force_8_tokens_all_two_shard_maps_and_sampled_three_shard_maps():
    q, k, v = _rand(1, 8, 8, 2, 1, 4, seed=11, std=0.7)
    scale = 0.5
    ref = _brute_force(q, k, v, scale, True)
    o, _ = oracle.attention_unsharded(q, k, v, scale)
    assert np.abs(o - ref).max() < 1e-13
    maps = [np.array(m, np.int32) for m in itertools.product(range(2), repeat=8)]
    rng = np.random.Generator(np.random.PCG64(3))
    all3 = list(itertools.product(range(3), repeat=8))
    maps += [np.array(all3[i], np.int32) for i in rng.choice(len(all3), 200, replace=False)]
    for m in maps:
        ns = 3
        plan = oracle.shard_plan(m, m, ns, ns)
        u, mm, e = oracle.attn_pass(q, k, v, scale, plan)
        merged, _ = oracle.post_pass(u, mm, e, row_scatter=plan.q_idx)
        assert np.abs(merged - ref).max() < 1e-13, m


def test_softmax_rows_sum_to_one_and_respect_mask():
    q, k, v = _rand(1, 19, 19, 1, 1, 8, seed=2)
    for pos in range(19):
        w = oracle.softmax_row(q[0, pos, 0], k[0, :, 0], 0.3, pos, causal=True)
        assert abs(w.sum() - 1.0) < 1e-14
        assert (w[pos + 1:] == 0).all() and (w[:pos + 1] > 0).all()
    o, _ = oracle.attention_unsharded(q, k, v, 0.3)
    w = np.stack([oracle.softmax_row(q[0, i, 0], k[0, :, 0], 0.3, i) for i in range(19)])
    assert np.abs(w @ v[0, :, 0].astype(np.float64) - o[0, :, 0]).max() < 1e-13


@pytest.mark.parametrize("kind,ns", [("round_robin", 4), ("random", 5), ("block_rr", 3), ("contiguous", 7),
                                     ("random", 1), ("random", 16)])
def test_merged_partials_equal_unsharded_for_any_partition(kind, ns):
    """Section 5.2.3: the post-pass sum reproduces softmax(a) v exactly, for any disjoint cover."""
    n = 96
    q, k, v = _rand(2, n, n, 4, 2, 16, seed=7)
    scale = 0.25
    rng = np.random.Generator(np.random.PCG64(99))
    m = wl.shard_map(kind, n, ns, rng, block=8)
    plan = oracle.shard_plan(m, m, ns, ns)
    u, mm, e = oracle.attn_pass(q, k, v, scale, plan)
    merged, lse = oracle.post_pass(u, mm, e, row_scatter=plan.q_idx)
    ref, ref_lse = oracle.attention_unsharded(q, k, v, scale)
    assert np.abs(merged - ref).max() < 1e-12
    assert np.abs(lse - ref_lse).max() < 1e-12


def test_result_invariant_to_shard_count_and_token_permutation_and_asymmetric_maps():
    n = 64
    q, k, v = _rand(1, n, n, 2, 2, 8, seed=21)
    outs = []
    for seed, (nq_s, nkv_s) in enumerate([(1, 1), (2, 8), (8, 2), (5, 5), (64, 64), (3, 70)]):
        rng = np.random.Generator(np.random.PCG64(seed))
        qm = wl.shard_map("random", n, nq_s, rng)
        km = wl.shard_map("random", n, nkv_s, rng)
        plan = oracle.shard_plan(qm, km, nq_s, nkv_s)
        u, mm, e = oracle.attn_pass(q, k, v, 0.35, plan)
        outs.append(oracle.post_pass(u, mm, e, row_scatter=plan.q_idx)[0])
    for o in outs[1:]:
        assert np.abs(o - outs[0]).max() < 1e-12


def test_partials_satisfy_unnormalised_identities():
    """u * e * exp(m) = exp(a) v and e * exp(m) = expsum(a) on each shard (Appendix E), with the
    right-hand sides built here from plain numpy products, no max subtraction."""
    n, H, d = 40, 2, 8
    q, k, v = _rand(1, n, n, H, H, d, seed=4, std=0.5)
    scale = 0.4
    rng = np.random.Generator(np.random.PCG64(8))
    m = wl.shard_map("random", n, 4, rng)
    plan = oracle.shard_plan(m, m, 4, 4)
    u, mm, e = oracle.attn_pass(q, k, v, scale, plan)
    for kk in range(4):
        cols = plan.kv_idx[plan.kv_off[kk]:plan.kv_off[kk + 1]]
        for h in range(H):
            a = q[0, plan.q_idx, h].astype(np.float64) @ k[0, cols, h].astype(np.float64).T * scale
            vis = cols[None, :] <= plan.q_idx[:, None]
            ea = np.where(vis, np.exp(a), 0.0)
            rhs_sum = ea.sum(1)
            rhs_vec = ea @ v[0, cols, h].astype(np.float64)
            nonempty = rhs_sum > 0
            em = np.where(nonempty, np.exp(mm[0, kk, :, h]), 0.0)
            assert np.abs(e[0, kk, :, h] * em - rhs_sum).max() < 1e-12
            assert np.abs(u[0, kk, :, h] * (e[0, kk, :, h] * em)[:, None] - rhs_vec).max() < 1e-12
            # empty rows follow the convention m = -inf, e = 0, u = 0
            assert np.isneginf(mm[0, kk, ~nonempty, h]).all() and (e[0, kk, ~nonempty, h] == 0).all()
            assert (u[0, kk, ~nonempty, h] == 0).all()
            # the row max is attained by a visible logit and 1 <= e <= visible count
            amax = np.where(vis, a, -np.inf).max(1)
            assert np.array_equal(mm[0, kk, :, h], amax)
            cnt = vis.sum(1)
            assert (e[0, kk, nonempty, h] >= 1 - 1e-15).all() and (e[0, kk, :, h] <= cnt + 1e-12).all()


def test_single_shard_is_textbook_attention_and_merge_is_identity():
    n = 33
    q, k, v = _rand(1, n, n, 4, 1, 16, seed=6)
    z = np.zeros(n, np.int32)
    plan = oracle.shard_plan(z, z, 1, 1)
    u, mm, e = oracle.attn_pass(q, k, v, 0.25, plan)
    ref = _sdpa_fp64(q, k, v, 0.25, True)
    assert np.abs(u[:, 0] - ref).max() < 1e-12
    merged, lse = oracle.post_pass(u, mm, e)
    assert np.abs(merged - u[:, 0]).max() < 1e-15
    assert np.abs(lse - (mm[:, 0] + np.log(e[:, 0]))).max() < 1e-13


def test_merge_is_stable_and_matches_direct_weighted_average():
    """Every m_k - n <= 0 (Section 5.2.3); large maxima do not overflow; the result equals the weighted
    average with weights exp(m_k) e_k computed in log space with torch.logsumexp."""
    rng = np.random.Generator(np.random.PCG64(17))
    B, P, R, H, d = 1, 6, 9, 3, 5
    u = rng.standard_normal((B, P, R, H, d))
    m = rng.standard_normal((B, P, R, H)) * 300.0  # exp(m) alone would overflow fp64
    e = rng.uniform(1.0, 50.0, (B, P, R, H))
    m[0, 2, 4, 1] = -np.inf
    e[0, 2, 4, 1] = 0.0
    u[0, 2, 4, 1] = 0.0
    o, lse = oracle.post_pass(u, m, e)
    logw = torch.from_numpy(m + np.log(np.where(e > 0, e, 1.0)))
    logw[0, 2, 4, 1] = -np.inf
    ref_lse = torch.logsumexp(logw, dim=1).numpy()
    wts = torch.softmax(logw, dim=1).numpy()
    ref = (wts[..., None] * u).sum(1)
    assert np.isfinite(o).all()
    # torch.logsumexp is held to 1e-8 (it is not repeatable below 1e-9, see test_unsharded_matches_library_sdpa);
    # the same log-space sum written out with numpy is held to 1e-10
    assert np.abs(o - ref).max() < 1e-12 and np.abs(lse - ref_lse).max() < 1e-8
    lw = logw.numpy()
    top = lw.max(1, keepdims=True)
    assert np.abs(lse - (top[:, 0] + np.log(np.exp(lw - top).sum(1)))).max() < 1e-10
    scatter = np.array([3, 0, 8, 1, 2, 7, 6, 5, 4], np.int32)
    o2, lse2 = oracle.post_pass(u, m, e, row_scatter=scatter)
    assert np.array_equal(o2[:, scatter], o) and np.array_equal(lse2[:, scatter], lse)


def test_decode_shape_and_noncausal_and_row_selection():
    # one new query row at the last position of a 50-token cache: everything visible
    q, k, v = _rand(3, 1, 50, 8, 2, 16, seed=9)
    rng = np.random.Generator(np.random.PCG64(1))
    km = wl.shard_map("random", 50, 4, rng)
    plan = oracle.shard_plan(np.zeros(1, np.int32), km, 1, 4, q_pos_offset=49)
    assert (plan.vis[0] == np.bincount(km, minlength=4)).all()
    u, mm, e = oracle.attn_pass(q, k, v, 0.25, plan)
    merged, _ = oracle.post_pass(u, mm, e)
    ref, _ = oracle.attention_unsharded(q, k, v, 0.25, causal=True, q_pos_offset=49)
    full = _sdpa_fp64(q, k, v, 0.25, False)
    assert np.abs(merged - ref).max() < 1e-12 and np.abs(ref - full).max() < 1e-12
    # non-causal plan
    q, k, v = _rand(1, 20, 20, 2, 2, 8, seed=10)
    sm = wl.shard_map("round_robin", 20, 3)
    plan = oracle.shard_plan(sm, sm, 3, 3, causal=False)
    u, mm, e = oracle.attn_pass(q, k, v, 0.3, plan)
    merged, _ = oracle.post_pass(u, mm, e, row_scatter=plan.q_idx)
    assert np.abs(merged - _sdpa_fp64(q, k, v, 0.3, False)).max() < 1e-12
    # row selection returns the same rows as the full evaluation
    rows = np.array([0, 7, 19], np.int32)
    o_all, l_all = oracle.attention_unsharded(q, k, v, 0.3)
    o_sel, l_sel = oracle.attention_unsharded(q, k, v, 0.3, rows=rows)
    assert np.array_equal(o_sel, o_all[:, rows]) and np.array_equal(l_sel, l_all[:, rows])


def test_workload_recipe_is_deterministic_and_bf16_exact():
    a = wl.config("c2_prefill_8b", n_q=128, n_kv=128)
    b = wl.config("c2_prefill_8b", n_q=128, n_kv=128)
    assert np.array_equal(a.q, b.q) and np.array_equal(a.kv_shard_of, b.kv_shard_of)
    assert np.array_equal(a.q_shard_of, a.kv_shard_of)
    # rounded values survive a bf16 round trip through torch bit-exactly
    t = torch.from_numpy(a.k).to(torch.bfloat16).float().numpy()
    assert np.array_equal(t, a.k)
    raw = np.random.Generator(np.random.PCG64(0)).standard_normal(4096, dtype=np.float32)
    assert np.array_equal(wl.round_to_bf16(raw), torch.from_numpy(raw).to(torch.bfloat16).float().numpy())
    bits = wl.bf16_bits(a.k)
    back = torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).float().numpy()
    assert np.array_equal(back, a.k)
    c3 = wl.config("c3_batched", B=2, n_q=512, n_kv=512)
    norms = np.abs(c3.k).mean(axis=(2, 3))
    assert ((norms > 3.0).sum(axis=1) == round(0.01 * 512)).all()  # outlier tokens: K rows x8
    assert wl.config("c1_tiny_f32").visible_pairs() == 32896
    assert wl.config("c5_decode", B=2, n_kv=64).q_pos_offset == 63
