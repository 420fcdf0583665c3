"""CPU oracle for Cascade's sequence-sharded attention -- TEST INFRASTRUCTURE ONLY.

Thin ctypes wrapper around ``cascade_oracle.c`` (plain C, fp64, OpenMP).  It shares nothing with the CUDA
library and must never be imported by it: only tests, the smoke check and the benchmark's CPU-baseline /
reference legs load this package.  Arrays are numpy; q, k, v are float32 holding values already rounded
to the I/O type, laid out ``[B, n, heads, d]``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "cascade_oracle.c")
_LIB = os.path.join(_HERE, "libcascade_oracle.so")

EMPTY, PARTIAL, FULL = 0, 1, 2

_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP).  Returns the path of the shared object."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_num_threads.restype = ctypes.c_int
        _lib.oracle_shard_plan.restype = ctypes.c_int
    return _lib


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def _f32(a):
    a = np.ascontiguousarray(a, dtype=np.float32)
    return a, a.ctypes.data_as(ctypes.c_void_p)


def _i32(a):
    a = np.ascontiguousarray(a, dtype=np.int32)
    return a, a.ctypes.data_as(ctypes.c_void_p)


def _ptr(a):
    return a.ctypes.data_as(ctypes.c_void_p)


def attention_unsharded(q, k, v, scale, causal=True, q_pos_offset=0, rows=None):
    """Plain softmax attention (the definition).  Returns (o [B,n_sel,H,d], lse [B,n_sel,H]) in fp64.

    ``rows``: optional int32 list of query rows to evaluate (all rows if None).
    """
    lib = _load()
    q, qp = _f32(q)
    k, kp = _f32(k)
    v, vp = _f32(v)
    B, n_q, H, d = q.shape
    _, n_kv, Hkv, _ = k.shape
    assert k.shape == v.shape and k.shape[0] == B and k.shape[3] == d and H % Hkv == 0
    if rows is None:
        n_sel, rp = n_q, None
    else:
        rows, rp = _i32(rows)
        n_sel = rows.shape[0]
    o = np.empty((B, n_sel, H, d), dtype=np.float64)
    lse = np.empty((B, n_sel, H), dtype=np.float64)
    lib.oracle_attention_unsharded(
        ctypes.c_int(B), ctypes.c_int(n_q), ctypes.c_int(n_kv), ctypes.c_int(H), ctypes.c_int(Hkv),
        ctypes.c_int(d), ctypes.c_double(scale), ctypes.c_int(q_pos_offset), ctypes.c_int(int(causal)),
        qp, kp, vp, rp, ctypes.c_int(n_sel), _ptr(o), _ptr(lse))
    return o, lse


class Plan:
    """Arrays of the shard plan (all int32 except pair_class uint8)."""

    def __init__(self, **kw):
        self.__dict__.update(kw)


def shard_plan(q_shard_of, kv_shard_of, n_q_shards, n_kv_shards, q_pos_offset=0, causal=True) -> Plan:
    lib = _load()
    qs, qsp = _i32(q_shard_of)
    ks, ksp = _i32(kv_shard_of)
    n_q, n_kv = qs.shape[0], ks.shape[0]
    q_off = np.zeros(n_q_shards + 1, np.int32)
    kv_off = np.zeros(n_kv_shards + 1, np.int32)
    q_idx = np.zeros(n_q, np.int32)
    q_inv = np.zeros(n_q, np.int32)
    kv_idx = np.zeros(n_kv, np.int32)
    kv_inv = np.zeros(n_kv, np.int32)
    vis = np.zeros((n_q, n_kv_shards), np.int32)
    pair_class = np.zeros((n_q_shards, n_kv_shards), np.uint8)
    rc = lib.oracle_shard_plan(
        ctypes.c_int(n_q), ctypes.c_int(n_kv), qsp, ksp, ctypes.c_int(n_q_shards),
        ctypes.c_int(n_kv_shards), ctypes.c_int(q_pos_offset), ctypes.c_int(int(causal)),
        _ptr(q_off), _ptr(q_idx), _ptr(q_inv), _ptr(kv_off), _ptr(kv_idx), _ptr(kv_inv), _ptr(vis),
        _ptr(pair_class))
    if rc != 0:
        raise ValueError("shard id out of range")
    return Plan(n_q=n_q, n_kv=n_kv, n_q_shards=n_q_shards, n_kv_shards=n_kv_shards,
                q_pos_offset=q_pos_offset, causal=bool(causal), q_off=q_off, q_idx=q_idx, q_inv=q_inv,
                kv_off=kv_off, kv_idx=kv_idx, kv_inv=kv_inv, vis=vis, pair_class=pair_class)


def dense_mask(plan: Plan, j: int, k: int) -> np.ndarray:
    """Visible (1) / masked (0) matrix of pair (S_j, T_k), straight from token positions."""
    rows = plan.q_idx[plan.q_off[j]:plan.q_off[j + 1]].astype(np.int64) + plan.q_pos_offset
    cols = plan.kv_idx[plan.kv_off[k]:plan.kv_off[k + 1]].astype(np.int64)
    if not plan.causal:
        return np.ones((rows.size, cols.size), np.uint8)
    return (cols[None, :] <= rows[:, None]).astype(np.uint8)


def attn_pass(q, k, v, scale, plan: Plan, row_tokens=None):
    """Per-(query shard, KV shard) partials, the Attention-Pass algorithm.  Returns (u, m, e) in fp64 with
    u [B, n_kv_shards, n_rows, H, d] and m, e [B, n_kv_shards, n_rows, H]; rows are the query tokens listed in
    ``row_tokens`` (default: every slot in shard-major order, plan.q_idx)."""
    lib = _load()
    q, qp = _f32(q)
    k, kp = _f32(k)
    v, vp = _f32(v)
    B, n_q, H, d = q.shape
    _, n_kv, Hkv, _ = k.shape
    assert n_q == plan.n_q and n_kv == plan.n_kv
    P = plan.n_kv_shards
    rows, rows_p = _i32(plan.q_idx if row_tokens is None else row_tokens)
    n_rows = rows.shape[0]
    u = np.empty((B, P, n_rows, H, d), np.float64)
    m = np.empty((B, P, n_rows, H), np.float64)
    e = np.empty((B, P, n_rows, H), np.float64)
    lib.oracle_attn_pass(
        ctypes.c_int(B), ctypes.c_int(n_q), ctypes.c_int(n_kv), ctypes.c_int(H), ctypes.c_int(Hkv),
        ctypes.c_int(d), ctypes.c_double(scale), ctypes.c_int(plan.q_pos_offset),
        ctypes.c_int(int(plan.causal)), qp, kp, vp, rows_p, ctypes.c_int(n_rows), ctypes.c_int(P),
        _ptr(plan.kv_off),
        _ptr(plan.kv_idx), _ptr(u), _ptr(m), _ptr(e))
    return u, m, e


def post_pass(u, m, e, row_scatter=None):
    """Log-sum-exp combine over parts, the Post-Pass algorithm.  Returns (o [B,n_rows,H,d], lse)."""
    lib = _load()
    u = np.ascontiguousarray(u, np.float64)
    m = np.ascontiguousarray(m, np.float64)
    e = np.ascontiguousarray(e, np.float64)
    B, P, n_rows, H, d = u.shape
    assert m.shape == (B, P, n_rows, H) and e.shape == m.shape
    rp = None
    if row_scatter is not None:
        row_scatter, rp = _i32(row_scatter)
    o = np.zeros((B, n_rows, H, d), np.float64)
    lse = np.zeros((B, n_rows, H), np.float64)
    lib.oracle_post_pass(ctypes.c_int(B), ctypes.c_int(P), ctypes.c_int(n_rows), ctypes.c_int(H),
                         ctypes.c_int(d), _ptr(u), _ptr(m), _ptr(e), rp, _ptr(o), _ptr(lse))
    return o, lse


def softmax_row(q_row, k_rows, scale, pos, causal=True):
    lib = _load()
    q_row, qp = _f32(q_row)
    k_rows, kp = _f32(k_rows)
    n_kv, d = k_rows.shape
    w = np.zeros(n_kv, np.float64)
    lib.oracle_softmax_row(ctypes.c_int(n_kv), ctypes.c_int(d), ctypes.c_double(scale), ctypes.c_int(pos),
                           ctypes.c_int(int(causal)), qp, kp, _ptr(w))
    return w
