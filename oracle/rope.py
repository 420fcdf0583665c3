"""Oracle for the rotary step of the pre-pass -- TEST INFRASTRUCTURE ONLY (numpy, fp64).

the Pre-Pass algorithm (CompNode single-layer pre-pass) ends with q <- rotary_pos_emb(q, p^{R_i}) and the same for k,
where p^{R_i} are the rows of the positional table p (Section 5.1, Sharding and Notation) at the node's ORIGINAL token
indices R_i.  The paper does not print the rotary formula; the reading taken here is the common
"rotate-half" form with exact real-valued angles:

    theta_i  = base ** (-2 i / d),                     i = 0 .. d/2 - 1
    p[t, i]  = (cos(t * theta_i), sin(t * theta_i))    row t of the positional table
    y[i]       = x[i] * cos - x[i + d/2] * sin
    y[i + d/2] = x[i + d/2] * cos + x[i] * sin

i.e. the pair (x[i], x[i + d/2]) is turned counter-clockwise by t * theta_i.  Because the position of a row
is its original token index, rotating the rows of a shard by p^{R_i} and rotating the whole sequence by p
give the same rows: the step commutes with sharding.  The rotated q, k are returned in the tensor's I/O type
(the pre-pass hands q, k on in the model's dtype), so the result is rounded once, straight from fp64.
"""
from __future__ import annotations

import numpy as np


def positional_table(n_positions: int, d: int, base: float):
    """(cos, sin), each float64 [n_positions, d/2]: row t is p[t] (Section 5.1: p is initialised before inference)."""
    if d % 2:
        raise ValueError("head_dim must be even")
    i = np.arange(d // 2, dtype=np.float64)
    theta = np.power(np.float64(base), -2.0 * i / d)
    ang = np.arange(n_positions, dtype=np.float64)[:, None] * theta[None, :]
    return np.cos(ang), np.sin(ang)


def round_fp64_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even from fp64 to the bf16 grid (8 significant bits), returned as float64.
    Normal range only: the rotated values are O(1)."""
    x = np.asarray(x, dtype=np.float64)
    mant, exp = np.frexp(x)  # x = mant * 2**exp, 0.5 <= |mant| < 1
    return np.ldexp(np.rint(np.ldexp(mant, 8)), exp - 8)


def round_to_io(x: np.ndarray, dtype: str) -> np.ndarray:
    if dtype == "bf16":
        return round_fp64_to_bf16(x)
    if dtype == "f32":
        return np.asarray(x, dtype=np.float64).astype(np.float32).astype(np.float64)
    if dtype == "f64":
        return np.asarray(x, dtype=np.float64)
    raise ValueError(dtype)


def rotary_pos_emb(x: np.ndarray, positions: np.ndarray, base: float, io_dtype: str = "f64") -> np.ndarray:
    """the rotary steps of the Pre-Pass algorithm.  x: [B, n, heads, d]; positions: [n] original token indices of the rows.
    Returns float64 holding values rounded to ``io_dtype``."""
    x = np.asarray(x, dtype=np.float64)
    B, n, H, d = x.shape
    positions = np.asarray(positions, dtype=np.int64)
    assert positions.shape == (n,)
    cos, sin = positional_table(int(positions.max()) + 1 if n else 0, d, base)
    c = cos[positions][None, :, None, :]
    s = sin[positions][None, :, None, :]
    lo, hi = x[..., : d // 2], x[..., d // 2:]
    y = np.concatenate([lo * c - hi * s, hi * c + lo * s], axis=-1)
    return round_to_io(y, io_dtype)
