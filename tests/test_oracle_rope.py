"""Pins for the rotary step of the oracle (the rotary steps of the Pre-Pass algorithm), against what the mathematics fixes:
textbook values, the rotation group law, the relative-position property and an independent complex-number route."""
import numpy as np

import oracle
from oracle import rope
from paper_2507_05228_b200 import workloads


def _x(B, n, H, d, seed):
    return np.random.default_rng(seed).standard_normal((B, n, H, d))


def test_textbook_values_fix_pairing_frequency_and_direction():
    # d = 2: one pair, theta_0 = 1 whatever the base; position 1 turns (1, 0) to (cos 1, sin 1)
    y = rope.rotary_pos_emb(np.array([1.0, 0.0]).reshape(1, 1, 1, 2), np.array([1]), base=10000.0)
    np.testing.assert_allclose(y.ravel(), [0.5403023058681398, 0.8414709848078965], rtol=0, atol=1e-15)
    # d = 4, base 10000: theta_1 = 10000 ** (-2/4) = 0.01, so position 100 turns the pair (x[1], x[3]) by one radian
    # and the pair (x[0], x[2]) by 100 radians
    e1 = np.zeros((1, 1, 1, 4))
    e1[..., 1] = 1.0
    y = rope.rotary_pos_emb(e1, np.array([100]), base=10000.0).ravel()
    np.testing.assert_allclose(y, [0.0, 0.5403023058681398, 0.0, 0.8414709848078965], rtol=0, atol=1e-13)
    e0 = np.zeros((1, 1, 1, 4))
    e0[..., 0] = 1.0
    y = rope.rotary_pos_emb(e0, np.array([100]), base=10000.0).ravel()
    np.testing.assert_allclose(y, [0.8623188722876839, 0.0, -0.5063656411097588, 0.0], rtol=0, atol=1e-13)
    # row 0 of the positional table is the identity rotation, whatever the base
    cos, sin = rope.positional_table(4, 2, 7.0)
    assert cos.shape == (4, 1) and cos[0, 0] == 1 and sin[0, 0] == 0


def test_position_zero_is_identity_and_norms_are_kept():
    x = _x(2, 9, 3, 16, 0)
    y0 = rope.rotary_pos_emb(x, np.zeros(9, np.int64), 500000.0)
    assert np.array_equal(y0, x)
    pos = np.array([0, 1, 2, 50, 1000, 8191, 7, 7, 3])
    y = rope.rotary_pos_emb(x, pos, 500000.0)
    d = 16
    for i in range(d // 2):  # every pair keeps its length
        np.testing.assert_allclose(np.hypot(y[..., i], y[..., i + d // 2]), np.hypot(x[..., i], x[..., i + d // 2]),
                                   rtol=1e-13)


def test_group_law_and_relative_position_property():
    d, base = 32, 10000.0
    x = _x(1, 5, 2, d, 1)
    p1 = np.array([3, 0, 17, 1000, 4095])
    p2 = np.array([5, 9, 100, 24, 1])
    twice = rope.rotary_pos_emb(rope.rotary_pos_emb(x, p1, base), p2, base)
    np.testing.assert_allclose(twice, rope.rotary_pos_emb(x, p1 + p2, base), atol=1e-11)
    # <rot(q, p), rot(k, s)> depends on p - s only, and equals <rot(q, p - s), k>
    q, k = _x(1, 1, 1, d, 2), _x(1, 1, 1, d, 3)
    for p, s in [(10, 3), (1007, 1000), (8000, 7993)]:
        a = (rope.rotary_pos_emb(q, np.array([p]), base) * rope.rotary_pos_emb(k, np.array([s]), base)).sum()
        b = (rope.rotary_pos_emb(q, np.array([p - s]), base) * k).sum()
        np.testing.assert_allclose(a, b, atol=1e-10)
    # and it does depend on the offset (a dropped rotation would pass the lines above)
    a7 = (rope.rotary_pos_emb(q, np.array([7]), base) * k).sum()
    assert abs(a7 - (q * k).sum()) > 1e-3


def test_complex_multiplication_route():
    # the pair (x[i], x[i + d/2]) as the complex number x[i] + j x[i + d/2], times exp(j t theta_i)
    d, base = 128, 500000.0
    x = _x(2, 6, 2, d, 4)
    pos = np.array([0, 1, 63, 64, 4097, 8191])
    z = x[..., : d // 2] + 1j * x[..., d // 2:]
    theta = np.array([base ** (-(2 * i) / d) for i in range(d // 2)])
    w = np.exp(1j * pos[:, None] * theta[None, :])[None, :, None, :]
    zz = z * w
    want = np.concatenate([zz.real, zz.imag], axis=-1)
    np.testing.assert_allclose(rope.rotary_pos_emb(x, pos, base), want, atol=1e-11)


def test_rounding_to_bf16_straight_from_fp64():
    # ties go to even; a value just above a tie goes up even where rounding through fp32 first would not
    assert rope.round_fp64_to_bf16(np.array([1.0 + 2.0 ** -8]))[0] == 1.0          # tie -> even (1.0)
    assert rope.round_fp64_to_bf16(np.array([1.0 + 3 * 2.0 ** -8]))[0] == 1.0 + 2.0 ** -6  # tie -> even (up)
    assert rope.round_fp64_to_bf16(np.array([1.0 + 2.0 ** -8 + 2.0 ** -40]))[0] == 1.0 + 2.0 ** -7
    x = np.random.default_rng(5).standard_normal(4096) * 3
    got = rope.round_fp64_to_bf16(x)
    f32 = x.astype(np.float32)
    exact_in_f32 = f32.astype(np.float64) == x
    via = workloads.round_to_bf16(f32).astype(np.float64)
    # the input generator's fp32 -> bf16 rounding agrees wherever fp32 holds the value exactly, and everywhere the
    # result is within half a bf16 step of the input
    assert np.array_equal(got[exact_in_f32], via[exact_in_f32])
    assert np.all(np.abs(got - x) <= np.abs(x) * 2.0 ** -8)
    assert np.array_equal(rope.round_fp64_to_bf16(got), got)
    assert np.array_equal(rope.round_fp64_to_bf16(-x), -got)


def test_rotation_commutes_with_sharding():
    # rows rotated shard by shard with p^{R_i} equal the rows of the whole sequence rotated with p (the Pre-Pass algorithm
    # takes the positions of the node's own index set), and sharded attention on them equals unsharded attention
    B, n, H, Hkv, d, base = 1, 24, 2, 1, 8, 10000.0
    rng = np.random.default_rng(6)
    q = rng.standard_normal((B, n, H, d))
    k = rng.standard_normal((B, n, Hkv, d))
    v = rng.standard_normal((B, n, Hkv, d))
    shard_of = (np.arange(n) % 6 // 2).astype(np.int32)  # (c, delta) = (2, 6)
    whole = rope.rotary_pos_emb(q, np.arange(n), base)
    for i in range(3):
        R = np.flatnonzero(shard_of == i)
        assert np.array_equal(rope.rotary_pos_emb(q[:, R], R, base), whole[:, R])
    qr = rope.rotary_pos_emb(q, np.arange(n), base).astype(np.float32)
    kr = rope.rotary_pos_emb(k, np.arange(n), base).astype(np.float32)
    v32 = v.astype(np.float32)
    plan = oracle.shard_plan(shard_of, shard_of, 3, 3)
    u, m, e = oracle.attn_pass(qr, kr, v32, 0.35, plan)
    o, _ = oracle.post_pass(u, m, e)
    o_tok = np.empty_like(o)
    o_tok[:, plan.q_idx] = o
    ref, _ = oracle.attention_unsharded(qr, kr, v32, 0.35)
    np.testing.assert_allclose(o_tok, ref, atol=1e-12)
