"""GPU parity of the fused rotary step (the rotary steps of the Pre-Pass algorithm inside the staging of Q and K rows) against the
fp64 oracle: the positional table, the rotated key rows left in the workspace, and the attention output.

Tolerances: the table is fp32 of an fp64 evaluation (|err| <= 2^-24 + angle error); rotated key rows are computed in
fp32 from that table and rounded to bf16, so they equal the oracle's fp64-then-bf16 values except where the fp32
result falls on the other side of a rounding boundary (at most one bf16 step, on a small fraction of elements);
attention outputs keep the library's bf16 bound of 2e-2 max-abs.
"""
import numpy as np
import pytest
import torch

import oracle
from oracle import rope
from paper_2507_05228_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def gu():
    import gpu_util
    return gpu_util


@pytest.fixture(scope="module")
def cb():
    from paper_2507_05228_b200 import binding
    return binding


def _rotated_reference(w, base):
    """q, k after the oracle's pre-pass tail, as float32 arrays holding bf16 values."""
    q_pos = np.arange(w.n_q) + w.q_pos_offset
    qr = rope.rotary_pos_emb(w.q, q_pos, base, "bf16").astype(np.float32)
    kr = rope.rotary_pos_emb(w.k, np.arange(w.n_kv), base, "bf16").astype(np.float32)
    return qr, kr


@pytest.mark.parametrize("n,d,base", [(8192, 128, 500000.0), (4096, 128, 10000.0), (300, 64, 10000.0), (1, 2, 2.0)])
def test_positional_table_matches_oracle(cb, n, d, base):
    t = cb.cascade_rope_table(n, d, base).cpu().numpy().astype(np.float64)
    cos, sin = rope.positional_table(n, d, base)
    assert t.shape == (n, d // 2, 2)
    assert np.abs(t[..., 0] - cos).max() <= 1e-7 and np.abs(t[..., 1] - sin).max() <= 1e-7
    assert (t[0, :, 0] == 1).all() and (t[0, :, 1] == 0).all()


def _run(cb, gu, w, base, n_positions=None):
    q, k, v = gu.to_device(w)
    plan = gu.make_plan(w)
    n_pos = n_positions or max(w.q_pos_offset + w.n_q, w.n_kv)
    table = cb.cascade_rope_table(n_pos, w.d, base)
    need = cb.cascade_workspace_bytes(plan, cb.CALL_SHARDED, cb.BF16, w.B, w.H, w.Hkv, w.d)
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    o, lse = cb.cascade_attn_sharded_rope(plan, q, k, v, w.scale, table, workspace=ws)
    torch.cuda.synchronize()
    assert plan.device_status() == 0
    return plan, ws, o, lse


def _check_rotated_keys(w, plan, ws, kr):
    """The first half of the workspace holds the rotated key rows in shard-major order [B][Hkv][slot][d]."""
    kv_idx = plan.get("kv_idx")
    n_el = w.B * w.Hkv * w.n_kv * w.d
    got = ws[: 2 * n_el].view(torch.bfloat16).view(w.B, w.Hkv, w.n_kv, w.d).float().cpu().numpy()
    worst, flips = 0.0, 0
    for b in range(w.B):
        idx = kv_idx[0 if kv_idx.shape[0] == 1 else b]
        want = kr[b][idx].transpose(1, 0, 2)  # [Hkv][slot][d]
        diff = np.abs(got[b].astype(np.float64) - want)
        step = np.maximum(np.abs(want), 2.0 ** -126) * 2.0 ** -7  # one bf16 step is at most 2^-7 relative
        assert (diff <= step).all(), "rotated key off by more than one bf16 step"
        flips += int((diff > 0).sum())
        worst = max(worst, diff.max())
    assert flips <= 2e-3 * n_el, f"{flips} of {n_el} rotated key elements differ from the oracle's rounding"
    # the value rows are copied untouched
    v_got = ws[2 * n_el: 4 * n_el].view(torch.bfloat16).view(w.B, w.Hkv, w.n_kv, w.d).float().cpu().numpy()
    for b in range(w.B):
        idx = kv_idx[0 if kv_idx.shape[0] == 1 else b]
        assert np.array_equal(v_got[b], w.v[b][idx].transpose(1, 0, 2))


@pytest.mark.parametrize("case", [
    dict(B=2, n_q=600, n_kv=600, H=8, Hkv=2, q_map="random", kv_map="random", n_q_shards=5, n_kv_shards=5),
    dict(B=1, n_q=1000, n_kv=1000, H=4, Hkv=4, q_map="block_rr", kv_map="block_rr", n_q_shards=4, n_kv_shards=4,
         block=8),
    dict(B=1, n_q=515, n_kv=515, H=16, Hkv=2, q_map="round_robin", kv_map="round_robin", n_q_shards=3,
         n_kv_shards=3),
    dict(B=1, n_q=200, n_kv=777, H=6, Hkv=2, q_map="random", kv_map="random", n_q_shards=2, n_kv_shards=7),
])
def test_fused_rotary_attention_matches_oracle(cb, gu, case):
    base = 500000.0
    w = wl.make_workload("rope", d=128, dtype="bf16", seed=21, **case)
    plan, ws, o, lse = _run(cb, gu, w, base)
    qr, kr = _rotated_reference(w, base)
    _check_rotated_keys(w, plan, ws, kr)
    o_ref, lse_ref = oracle.attention_unsharded(qr, kr, w.v, w.scale, causal=True, q_pos_offset=w.q_pos_offset)
    gu.check_output(o, lse, o_ref, lse_ref, w.tol, "fused rotary attention")
    # the check has power: leaving either rotation out moves the result far beyond the tolerance
    o_noq, _ = oracle.attention_unsharded(w.q, kr, w.v, w.scale, causal=True, q_pos_offset=w.q_pos_offset)
    o_nok, _ = oracle.attention_unsharded(qr, w.k, w.v, w.scale, causal=True, q_pos_offset=w.q_pos_offset)
    assert np.abs(o_noq - o_ref).max() > 10 * w.tol and np.abs(o_nok - o_ref).max() > 10 * w.tol
    plan.destroy()


def test_rotation_at_position_zero_table_is_plain_attention(cb, gu):
    """With a table of identity rotations (every row = row 0) the rope entry point is bit-identical to the plain one."""
    w = wl.make_workload("rope_id", 1, 400, 400, 8, 2, 128, "bf16", "random", "random", 3, 3, seed=22)
    q, k, v = gu.to_device(w)
    plan = gu.make_plan(w)
    table = cb.cascade_rope_table(1, 128, 10000.0).expand(400, 64, 2).contiguous()
    o_r, lse_r = cb.cascade_attn_sharded_rope(plan, q, k, v, w.scale, table)
    o_p, lse_p = cb.cascade_attn_sharded(plan, q, k, v, w.scale)
    assert torch.equal(o_r, o_p) and torch.equal(lse_r, lse_p)
    plan.destroy()


def test_headline_size_sampled_rows(cb, gu):
    """The headline prefill shape (2048 tokens, 32/8 heads, 8 random shards) with the rotary step fused; the oracle
    evaluates a stratified sample of rows."""
    base = 500000.0
    w = wl.config("c2_prefill_8b")
    plan, ws, o, lse = _run(cb, gu, w, base)
    qr, kr = _rotated_reference(w, base)
    _check_rotated_keys(w, plan, ws, kr)
    rows = wl.sample_rows(w, 3)
    o_ref, lse_ref = oracle.attention_unsharded(qr, kr, w.v, w.scale, causal=True, rows=rows)
    rt = torch.from_numpy(rows.astype(np.int64)).cuda()
    gu.check_output(o[:, rt], lse[:, rt], o_ref, lse_ref, w.tol, "headline shape, fused rotary (sampled rows)")
    assert torch.isfinite(o.float()).all() and torch.isfinite(lse).all()
    plan.destroy()


def test_argument_checks(cb, gu):
    w = wl.make_workload("rope_err", 1, 64, 64, 4, 2, 128, "bf16", "random", "random", 2, 2, seed=23)
    q, k, v = gu.to_device(w)
    plan = gu.make_plan(w)
    short = cb.cascade_rope_table(63, 128, 10000.0)
    with pytest.raises(cb.CascadeError) as ei:
        cb.cascade_attn_sharded_rope(plan, q, k, v, w.scale, short)
    assert ei.value.status == 1 and "63 rows" in str(ei.value)
    plan.destroy()
    # shapes outside the tensor-core route are refused, not silently left unrotated
    w32 = wl.make_workload("rope_f32", 1, 64, 64, 4, 2, 64, "f32", "random", "random", 2, 2, seed=24)
    q, k, v = gu.to_device(w32)
    plan = gu.make_plan(w32)
    with pytest.raises(cb.CascadeError) as ei:
        cb.cascade_attn_sharded_rope(plan, q, k, v, w32.scale, cb.cascade_rope_table(64, 64, 10000.0))
    assert ei.value.status == 3
    plan.destroy()
    wd = wl.config("c5_decode", B=2, n_kv=256)
    q, k, v = gu.to_device(wd)
    plan = gu.make_plan(wd)
    with pytest.raises(cb.CascadeError) as ei:
        cb.cascade_attn_sharded_rope(plan, q, k, v, wd.scale, cb.cascade_rope_table(256, 128, 10000.0))
    assert ei.value.status == 3
    plan.destroy()
    for bad in [(0, 128, 10000.0), (8, 127, 10000.0), (8, 128, 1.0)]:
        with pytest.raises(cb.CascadeError):
            cb.cascade_rope_table(*bad)


@pytest.mark.parametrize("dtype,d,H", [("bf16", 128, 8), ("bf16", 64, 4), ("f32", 64, 3), ("f32", 128, 2)])
def test_standalone_rotary_pass_matches_oracle(cb, gu, dtype, d, H):
    """cascade_rope_apply on a block of rows that starts in the middle of the sequence, out of place and in place, on
    a strided view."""
    base, first, n = 10000.0, 37, 45
    w = wl.make_workload("rope_rows", 2, n, n, H, H, d, dtype, "round_robin", "round_robin", 1, 1, seed=91)
    (x,) = gu.to_device(w, which=("q",))
    table = cb.cascade_rope_table(first + n, d, base)
    want = rope.rotary_pos_emb(w.q, np.arange(first, first + n), base, dtype)
    y = cb.cascade_rope_apply(x, first, table)
    packed = torch.cat([x, x], dim=2).contiguous()  # a strided view: heads H..2H-1 of a wider tensor
    view = packed[:, :, H:]
    cb.cascade_rope_apply(view, first, table, out=view)
    torch.cuda.synchronize()
    for got in (y, view):
        g = got.double().cpu().numpy()
        if dtype == "bf16":
            step = np.maximum(np.abs(want), 2.0 ** -126) * 2.0 ** -7  # one bf16 step at that magnitude
            assert (np.abs(g - want) <= step).all()
            assert (g != want).mean() < 5e-3
        else:
            assert np.abs(g - want).max() <= 2e-6
    assert torch.equal(packed[:, :, :H], x)  # the neighbouring heads of the packed tensor are untouched


def test_decode_steps_with_rotary_append_over_a_sharded_cache(cb, gu):
    """A decode loop: every step hands the new token's unrotated q, k, v rows to cascade_decode_step_rope, which appends
    to a cache whose unwritten rows hold NaN.  Reference: the oracle's rotary step on the whole sequence, then
    unsharded attention at that position."""
    base, cap, B, H, Hkv, d, P = 500000.0, 300, 2, 8, 2, 128, 5
    w = wl.make_workload("decode_rope", B, cap, cap, H, Hkv, d, "bf16", "block_rr", "block_rr", P, P, seed=92, block=4)
    q_all, k_all, v_all = gu.to_device(w)
    qr = rope.rotary_pos_emb(w.q, np.arange(cap), base, "bf16").astype(np.float32)
    kr = rope.rotary_pos_emb(w.k, np.arange(cap), base, "bf16").astype(np.float32)
    table = cb.cascade_rope_table(cap, d, base)
    plan = cb.cascade_shard_plan(np.zeros(1, np.int32), w.kv_shard_of, 1, P, 0, True)
    k_cache = torch.full_like(k_all, float("nan"))
    v_cache = torch.full_like(v_all, float("nan"))
    for pos in range(0, 40):
        o, lse = cb.cascade_decode_step_rope(plan, q_all[:, pos:pos + 1], k_all[:, pos:pos + 1], v_all[:, pos:pos + 1],
                                             k_cache, v_cache, pos, w.scale, table)
        o_ref, lse_ref = oracle.attention_unsharded(qr[:, pos:pos + 1], kr, w.v, w.scale, causal=True, q_pos_offset=pos)
        gu.check_output(o, lse, o_ref, lse_ref, w.tol, f"decode step at position {pos}")
    # the cache now holds the rotated keys and the values of the tokens seen so far, and nothing else
    got_k = k_cache[:, :40].double().cpu().numpy()
    step = np.maximum(np.abs(kr[:, :40]), 2.0 ** -126) * 2.0 ** -7
    assert (np.abs(got_k - kr[:, :40]) <= step).all()
    assert torch.equal(v_cache[:, :40], v_all[:, :40]) and torch.isnan(k_cache[:, 40:].float()).all()
    # jump ahead: fill rows 40..199 in one go with the standalone pass, then continue decoding at position 200
    cb.cascade_rope_apply(k_all[:, 40:200], 40, table, out=k_cache[:, 40:200])
    v_cache[:, 40:200] = v_all[:, 40:200]
    for pos in (200, 201, 299):
        if pos == 299:
            cb.cascade_rope_apply(k_all[:, 202:299], 202, table, out=k_cache[:, 202:299])
            v_cache[:, 202:299] = v_all[:, 202:299]
        o, lse = cb.cascade_decode_step_rope(plan, q_all[:, pos:pos + 1], k_all[:, pos:pos + 1], v_all[:, pos:pos + 1],
                                             k_cache, v_cache, pos, w.scale, table)
        o_ref, lse_ref = oracle.attention_unsharded(qr[:, pos:pos + 1], kr, w.v, w.scale, causal=True, q_pos_offset=pos)
        gu.check_output(o, lse, o_ref, lse_ref, w.tol, f"decode step at position {pos}")
    assert plan.device_status() == 0
    with pytest.raises(cb.CascadeError):
        cb.cascade_decode_step_rope(plan, q_all[:, :1], k_all[:, :1], v_all[:, :1], k_cache, v_cache, cap, w.scale, table)
    plan.destroy()
