"""ctypes binding of libcascade_b200.so: argument marshalling only -- every step runs in the CUDA library.

Function names match the C ABI (include/cascade.h).  torch supplies device memory and the current stream.
The library must have been built (``python -m paper_2507_05228_b200.build``); loading fails loudly otherwise:
there is no fallback path.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# CASCADE_B200_LIB selects another build of the same library (the index-checking debug build)
LIB_PATH = os.environ.get("CASCADE_B200_LIB") or os.path.join(_HERE, "libcascade_b200.so")

F32, BF16 = 0, 1
CALL_PARTIALS, CALL_SHARDED = 0, 1
CALL_DECODE_STEP_ROPE = 3
PLAN_FIELDS = {"q_off": 0, "q_idx": 1, "q_inv": 2, "kv_off": 3, "kv_idx": 4, "kv_inv": 5, "vis": 6,
               "pair_class": 7}
STATUS_NAMES = {0: "OK", 1: "INVALID_ARG", 2: "BAD_MAP", 3: "UNSUPPORTED", 4: "WORKSPACE", 5: "ALLOC", 6: "CUDA",
                7: "TIMEOUT"}

EXPORTS = [
    "cascade_version", "cascade_last_error", "cascade_launch_count", "cascade_shard_plan", "cascade_shard_plan_host",
    "cascade_plan_destroy",
    "cascade_plan_get", "cascade_plan_dense_mask", "cascade_plan_device_status", "cascade_attn_partials",
    "cascade_merge", "cascade_attn_sharded", "cascade_workspace_bytes", "cascade_attn_decode_static",
    "cascade_kernel_timing_begin", "cascade_kernel_timing_end", "cascade_rope_table", "cascade_attn_sharded_rope",
    "cascade_cdelta_shard_map", "cascade_msplit_shard_map", "cascade_index_set_gaps", "cascade_kl_gaps",
    "cascade_attn_sharded_host", "cascade_plan_advance", "cascade_shard_plan_resident",
    "cascade_shard_plan_resident_host", "cascade_rope_apply", "cascade_decode_step_rope", "cascade_merge_peers",
]


class CascadeError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"cascade status {status} ({STATUS_NAMES.get(status, '?')}): {message}")
        self.status = status


class Strides(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int64), ("token", ctypes.c_int64), ("head", ctypes.c_int64)]


_lib = None


def lib() -> ctypes.CDLL:
    """The loaded shared library.  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2507_05228_b200.build` "
                "(there is no CPU or PyTorch fallback)")
        L = ctypes.CDLL(LIB_PATH)
        vp, i32, i64, f32 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_float
        L.cascade_version.restype = i32
        L.cascade_last_error.restype = ctypes.c_char_p
        L.cascade_launch_count.restype = i64
        L.cascade_shard_plan.argtypes = [i32, i32, i32, vp, vp, i32, i32, i32, i32, vp, ctypes.POINTER(vp)]
        L.cascade_shard_plan_host.argtypes = [i32, i32, i32, vp, vp, i32, i32, i32, i32, ctypes.POINTER(vp)]
        L.cascade_shard_plan_resident.argtypes = [i32, i32, i32, vp, vp, vp, i32, i32, i32, i32, vp, ctypes.POINTER(vp)]
        L.cascade_shard_plan_resident_host.argtypes = [i32, i32, i32, vp, vp, vp, i32, i32, i32, i32, ctypes.POINTER(vp)]
        L.cascade_rope_apply.argtypes = [i32, i32, i32, i32, i32, vp, Strides, i32, vp, i32, vp, Strides, vp]
        L.cascade_decode_step_rope.argtypes = [vp, i32, i32, i32, f32, vp, Strides, vp, Strides, vp, Strides, vp, Strides,
                                               vp, Strides, i32, vp, i32, vp, Strides, vp, vp, ctypes.c_size_t, vp]
        L.cascade_merge_peers.argtypes = [i32, i32, i32, vp, vp, vp, vp, i32, vp, i32, i32, i32, vp, Strides, vp, vp]
        L.cascade_plan_destroy.argtypes = [vp]
        L.cascade_plan_get.argtypes = [vp, i32, ctypes.POINTER(vp), ctypes.POINTER(vp), ctypes.POINTER(i64)]
        L.cascade_plan_dense_mask.argtypes = [vp, i32, i32, i32, vp, i64]
        L.cascade_plan_device_status.argtypes = [vp, ctypes.POINTER(i32)]
        L.cascade_attn_partials.argtypes = [vp, i32, i32, i32, i32, i32, f32, vp, Strides, vp, Strides, vp, Strides,
                                            vp, vp, vp, vp, ctypes.c_size_t, vp]
        L.cascade_merge.argtypes = [i32, i32, i32, i32, i32, i32, vp, vp, vp, vp, i64, vp, Strides, vp, vp]
        L.cascade_attn_sharded.argtypes = [vp, i32, i32, i32, i32, i32, f32, vp, Strides, vp, Strides, vp, Strides,
                                           vp, Strides, vp, vp, ctypes.c_size_t, vp]
        L.cascade_attn_decode_static.argtypes = [vp, i32, i32, i32, f32, vp, Strides, vp, Strides, vp, Strides, vp,
                                                 Strides, vp, vp]
        L.cascade_workspace_bytes.argtypes = [vp, i32, i32, i32, i32, i32, i32, ctypes.POINTER(ctypes.c_size_t)]
        L.cascade_rope_table.argtypes = [i32, i32, ctypes.c_double, vp, vp]
        L.cascade_attn_sharded_rope.argtypes = [vp, i32, i32, i32, i32, i32, f32, vp, Strides, vp, Strides, vp, Strides,
                                                vp, i32, vp, Strides, vp, vp, ctypes.c_size_t, vp]
        pi32 = ctypes.POINTER(i32)
        L.cascade_cdelta_shard_map.argtypes = [i32, i32, i32, vp, pi32]
        L.cascade_msplit_shard_map.argtypes = [i32, vp, i32, i32, vp]
        L.cascade_index_set_gaps.argtypes = [i32, vp, pi32, pi32, pi32, pi32]
        L.cascade_kl_gaps.argtypes = [i32, vp, vp, i32, vp]
        L.cascade_attn_sharded_host.argtypes = [vp, i32, i32, i32, i32, i32, f32, vp, vp, vp, vp, vp, ctypes.c_size_t, vp]
        L.cascade_plan_advance.argtypes = [vp, i32, vp]
        L.cascade_kernel_timing_begin.argtypes = []
        L.cascade_kernel_timing_end.argtypes = [ctypes.POINTER(ctypes.c_double), ctypes.POINTER(i64)]
        for name in EXPORTS:
            if name not in ("cascade_version", "cascade_last_error", "cascade_launch_count"):
                getattr(L, name).restype = i32
        _lib = L
    return _lib


def _check(status: int):
    if status != 0:
        raise CascadeError(status, lib().cascade_last_error().decode())


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise CascadeError(3, f"dtype {t.dtype} unsupported")


def _strides(t: torch.Tensor) -> Strides:
    assert t.dim() == 4 and t.stride(3) == 1, "expected [batch, tokens, heads, head_dim] with contiguous head_dim"
    return Strides(t.stride(0), t.stride(1), t.stride(2))


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream if torch.cuda.is_available() else 0


def cascade_version() -> int:
    return int(lib().cascade_version())


def cascade_launch_count() -> int:
    return int(lib().cascade_launch_count())


def cascade_kernel_timing_begin() -> None:
    _check(lib().cascade_kernel_timing_begin())


def cascade_kernel_timing_end():
    """(summed milliseconds, launches) of the attention / decode kernels launched since ..._begin()."""
    ms, n = ctypes.c_double(), ctypes.c_int64()
    _check(lib().cascade_kernel_timing_end(ctypes.byref(ms), ctypes.byref(n)))
    return ms.value, n.value


class Plan:
    """Owner of a cascade_plan_t*."""

    def __init__(self, handle: int, n_maps: int, n_q: int, n_kv: int, n_q_shards: int, n_kv_shards: int):
        self.handle = handle
        self.n_maps, self.n_q, self.n_kv = n_maps, n_q, n_kv
        self.n_q_shards, self.n_kv_shards = n_q_shards, n_kv_shards

    def get(self, field: str) -> np.ndarray:
        """Host copy of a plan array (cascade_plan_get)."""
        hp, n = ctypes.c_void_p(), ctypes.c_int64()
        _check(lib().cascade_plan_get(self.handle, PLAN_FIELDS[field], ctypes.byref(hp), None, ctypes.byref(n)))
        ctype = ctypes.c_uint8 if field == "pair_class" else ctypes.c_int32
        arr = np.ctypeslib.as_array(ctypes.cast(hp, ctypes.POINTER(ctype)), shape=(n.value,)).copy()
        return arr.reshape(self._shape(field))

    def dev_ptr(self, field: str) -> int:
        dp = ctypes.c_void_p()
        _check(lib().cascade_plan_get(self.handle, PLAN_FIELDS[field], None, ctypes.byref(dp), None))
        return dp.value

    def _shape(self, field):
        m = self.n_maps
        return {"q_off": (m, self.n_q_shards + 1), "kv_off": (m, self.n_kv_shards + 1), "q_idx": (m, self.n_q),
                "q_inv": (m, self.n_q), "kv_idx": (m, self.n_kv), "kv_inv": (m, self.n_kv),
                "vis": (m, self.n_q, self.n_kv_shards),
                "pair_class": (m, self.n_q_shards, self.n_kv_shards)}[field]

    def dense_mask(self, j: int, k: int, map: int = 0) -> np.ndarray:
        qo, ko = self.get("q_off")[map], self.get("kv_off")[map]
        rows, cols = int(qo[j + 1] - qo[j]), int(ko[k + 1] - ko[k])
        out = np.zeros((rows, cols), np.uint8)
        _check(lib().cascade_plan_dense_mask(self.handle, map, j, k, out.ctypes.data_as(ctypes.c_void_p),
                                             out.size))
        return out

    def device_status(self) -> int:
        code = ctypes.c_int32()
        _check(lib().cascade_plan_device_status(self.handle, ctypes.byref(code)))
        return code.value

    def advance(self, q_pos_offset: int):
        """Move the query block to position ``q_pos_offset`` (token-sharded KV caching): the causal prefixes are
        recomputed, on the device in the order of the current stream.  A host-only plan needs no stream."""
        _check(lib().cascade_plan_advance(self.handle, int(q_pos_offset), _stream() if torch.cuda.is_available() else None))

    def destroy(self):
        if self.handle:
            lib().cascade_plan_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


def _maps(q_shard_of, kv_shard_of):
    qs = np.ascontiguousarray(q_shard_of, dtype=np.int32)
    ks = np.ascontiguousarray(kv_shard_of, dtype=np.int32)
    if qs.ndim == 1:
        qs, ks = qs[None], ks[None]
    assert ks.shape[0] == qs.shape[0]
    return qs, ks


def cascade_shard_plan(q_shard_of, kv_shard_of, n_q_shards: int, n_kv_shards: int, q_pos_offset: int = 0,
                       causal: bool = True) -> Plan:
    """q_shard_of / kv_shard_of: int32 host arrays [n] (one map for the batch) or [n_maps, n]."""
    qs, ks = _maps(q_shard_of, kv_shard_of)
    n_maps, n_q = qs.shape
    n_kv = ks.shape[1]
    out = ctypes.c_void_p()
    _check(lib().cascade_shard_plan(n_maps, n_q, n_kv, qs.ctypes.data_as(ctypes.c_void_p),
                                    ks.ctypes.data_as(ctypes.c_void_p), n_q_shards, n_kv_shards, q_pos_offset,
                                    int(bool(causal)), _stream(), ctypes.byref(out)))
    return Plan(out.value, n_maps, n_q, n_kv, n_q_shards, n_kv_shards)


def cascade_shard_plan_host(q_shard_of, kv_shard_of, n_q_shards: int, n_kv_shards: int, q_pos_offset: int = 0,
                            causal: bool = True) -> Plan:
    """Host-only plan (no GPU needed): readable, not usable by the attention calls."""
    qs, ks = _maps(q_shard_of, kv_shard_of)
    n_maps, n_q = qs.shape
    n_kv = ks.shape[1]
    out = ctypes.c_void_p()
    _check(lib().cascade_shard_plan_host(n_maps, n_q, n_kv, qs.ctypes.data_as(ctypes.c_void_p),
                                         ks.ctypes.data_as(ctypes.c_void_p), n_q_shards, n_kv_shards, q_pos_offset,
                                         int(bool(causal)), ctypes.byref(out)))
    return Plan(out.value, n_maps, n_q, n_kv, n_q_shards, n_kv_shards)


def cascade_shard_plan_resident(q_shard_of, kv_shard_of, kv_pos, n_q_shards: int, n_kv_shards: int,
                                q_pos_offset: int = 0, causal: bool = True, host_only: bool = False) -> Plan:
    """Plan for a party that holds only some K/V rows: row y of its k/v tensors is the token at original position
    kv_pos[y] (int32, strictly ascending; shaped like kv_shard_of)."""
    qs, ks = _maps(q_shard_of, kv_shard_of)
    kp = np.ascontiguousarray(np.asarray(kv_pos, dtype=np.int32).reshape(ks.shape))
    n_maps, n_q = qs.shape
    n_kv = ks.shape[1]
    out = ctypes.c_void_p()
    args = (n_maps, n_q, n_kv, qs.ctypes.data_as(ctypes.c_void_p), ks.ctypes.data_as(ctypes.c_void_p),
            kp.ctypes.data_as(ctypes.c_void_p), n_q_shards, n_kv_shards, q_pos_offset, int(bool(causal)))
    if host_only:
        _check(lib().cascade_shard_plan_resident_host(*args, ctypes.byref(out)))
    else:
        _check(lib().cascade_shard_plan_resident(*args, _stream(), ctypes.byref(out)))
    return Plan(out.value, n_maps, n_q, n_kv, n_q_shards, n_kv_shards)


def cascade_workspace_bytes(plan: Plan, which_call: int, dtype_code: int, batch: int, n_heads: int, n_kv_heads: int,
                            head_dim: int) -> int:
    out = ctypes.c_size_t()
    _check(lib().cascade_workspace_bytes(plan.handle, which_call, dtype_code, batch, n_heads, n_kv_heads, head_dim,
                                         ctypes.byref(out)))
    return out.value


def _ws(nbytes: int, device, workspace: Optional[torch.Tensor]):
    if nbytes == 0:
        return None, 0, 0
    if workspace is None:
        workspace = torch.empty(nbytes, dtype=torch.uint8, device=device)
    return workspace, workspace.data_ptr(), workspace.numel() * workspace.element_size()


def cascade_attn_partials(plan: Plan, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, scale: float, out=None,
                          workspace=None):
    """Returns (o_part [B, n_kv_shards, n_q, H, d] in q.dtype, m_part, l_part [B, n_kv_shards, n_q, H] fp32);
    rows in shard-major order."""
    B, n_q, H, d = q.shape
    Hkv = k.shape[2]
    code = _dtype_code(q)
    if out is None:
        P = plan.n_kv_shards
        out = (torch.empty((B, P, n_q, H, d), dtype=q.dtype, device=q.device),
               torch.empty((B, P, n_q, H), dtype=torch.float32, device=q.device),
               torch.empty((B, P, n_q, H), dtype=torch.float32, device=q.device))
    o_part, m_part, l_part = out
    nbytes = cascade_workspace_bytes(plan, CALL_PARTIALS, code, B, H, Hkv, d)
    ws, ws_ptr, ws_bytes = _ws(nbytes, q.device, workspace)
    _check(lib().cascade_attn_partials(plan.handle, code, B, H, Hkv, d, scale, q.data_ptr(), _strides(q),
                                       k.data_ptr(), _strides(k), v.data_ptr(), _strides(v), o_part.data_ptr(),
                                       m_part.data_ptr(), l_part.data_ptr(), ws_ptr, ws_bytes, _stream()))
    return o_part, m_part, l_part


def cascade_merge(o_part: torch.Tensor, m_part: torch.Tensor, l_part: torch.Tensor, row_scatter_ptr: int = 0,
                  row_scatter_batch_stride: int = 0, out=None, want_lse: bool = True):
    """o_part [B, P, n_rows, H, d]; row_scatter_ptr: device pointer of an int32 [n_rows] map (a plan's q_idx) or 0.
    Returns (o [B, n_rows, H, d], lse [B, n_rows, H] or None)."""
    B, P, n_rows, H, d = o_part.shape
    code = _dtype_code(o_part)
    o = out if out is not None else torch.empty((B, n_rows, H, d), dtype=o_part.dtype, device=o_part.device)
    lse = torch.empty((B, n_rows, H), dtype=torch.float32, device=o_part.device) if want_lse else None
    _check(lib().cascade_merge(code, B, P, n_rows, H, d, o_part.data_ptr(), m_part.data_ptr(), l_part.data_ptr(),
                               row_scatter_ptr or None, row_scatter_batch_stride, o.data_ptr(), _strides(o),
                               lse.data_ptr() if lse is not None else None, _stream()))
    return o, lse


def cascade_merge_peers(sources, row_gather: Optional[torch.Tensor], n_rows: int, out=None, want_lse: bool = True):
    """Post-pass over parts left where they were computed.  sources: list of (o_part [B, P_s, n_src_rows, H, d],
    m_part, l_part [B, P_s, n_src_rows, H]) device tensors, one triple per party (P_s may differ); row_gather: device
    int32 [n_rows] rows of the source buffers to combine, or None.  Returns (o [B, n_rows, H, d], lse or None)."""
    o0 = sources[0][0]
    B, _, n_src_rows, H, d = o0.shape
    n = len(sources)
    VP = ctypes.c_void_p * n
    ptr = lambda t: t.data_ptr() if t.numel() else None
    o_ptrs = VP(*[ptr(s[0]) for s in sources])
    m_ptrs = VP(*[ptr(s[1]) for s in sources])
    l_ptrs = VP(*[ptr(s[2]) for s in sources])
    parts = (ctypes.c_int32 * n)(*[s[0].shape[1] for s in sources])
    o = out if out is not None else torch.empty((B, n_rows, H, d), dtype=o0.dtype, device=o0.device)
    lse = torch.empty((B, n_rows, H), dtype=torch.float32, device=o0.device) if want_lse else None
    _check(lib().cascade_merge_peers(_dtype_code(o0), B, n, o_ptrs, m_ptrs, l_ptrs, parts, n_src_rows,
                                     row_gather.data_ptr() if row_gather is not None else None, n_rows, H, d,
                                     o.data_ptr(), _strides(o), lse.data_ptr() if lse is not None else None, _stream()))
    return o, lse


def cascade_attn_sharded(plan: Plan, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, scale: float, out=None,
                         want_lse: bool = True, workspace=None):
    """Fused attention-pass + post-pass.  Returns (o [B, n_q, H, d] in token order, lse or None)."""
    B, n_q, H, d = q.shape
    Hkv = k.shape[2]
    code = _dtype_code(q)
    o = out if out is not None else torch.empty((B, n_q, H, d), dtype=q.dtype, device=q.device)
    lse = torch.empty((B, n_q, H), dtype=torch.float32, device=q.device) if want_lse else None
    nbytes = cascade_workspace_bytes(plan, CALL_SHARDED, code, B, H, Hkv, d)
    ws, ws_ptr, ws_bytes = _ws(nbytes, q.device, workspace)
    _check(lib().cascade_attn_sharded(plan.handle, code, B, H, Hkv, d, scale, q.data_ptr(), _strides(q),
                                      k.data_ptr(), _strides(k), v.data_ptr(), _strides(v), o.data_ptr(),
                                      _strides(o), lse.data_ptr() if lse is not None else None, ws_ptr, ws_bytes,
                                      _stream()))
    return o, lse


def cascade_rope_table(n_positions: int, head_dim: int, base: float, device="cuda") -> torch.Tensor:
    """Positional table of the rotary embedding on the device: fp32 [n_positions, head_dim/2, 2] = (cos, sin)."""
    table = torch.empty((n_positions, head_dim // 2, 2), dtype=torch.float32, device=device)
    _check(lib().cascade_rope_table(n_positions, head_dim, float(base), table.data_ptr(), _stream()))
    return table


def cascade_attn_sharded_rope(plan: Plan, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, scale: float,
                              rope_table: torch.Tensor, out=None, want_lse: bool = True, workspace=None):
    """cascade_attn_sharded on unrotated q, k with the rotary step fused into the staging of their rows."""
    B, n_q, H, d = q.shape
    Hkv = k.shape[2]
    code = _dtype_code(q)
    assert rope_table.dtype == torch.float32 and rope_table.is_contiguous() and rope_table.shape[1:] == (d // 2, 2)
    o = out if out is not None else torch.empty((B, n_q, H, d), dtype=q.dtype, device=q.device)
    lse = torch.empty((B, n_q, H), dtype=torch.float32, device=q.device) if want_lse else None
    nbytes = cascade_workspace_bytes(plan, CALL_SHARDED, code, B, H, Hkv, d)
    ws, ws_ptr, ws_bytes = _ws(nbytes, q.device, workspace)
    _check(lib().cascade_attn_sharded_rope(plan.handle, code, B, H, Hkv, d, scale, q.data_ptr(), _strides(q),
                                           k.data_ptr(), _strides(k), v.data_ptr(), _strides(v),
                                           rope_table.data_ptr(), rope_table.shape[0], o.data_ptr(), _strides(o),
                                           lse.data_ptr() if lse is not None else None, ws_ptr, ws_bytes, _stream()))
    return o, lse


CALL_SHARDED_HOST = 2


def cascade_rope_apply(x: torch.Tensor, first_position: int, rope_table: torch.Tensor, out=None) -> torch.Tensor:
    """The rotary steps of the pre-pass on x [B, n_rows, heads, d] (row r at position first_position + r); out may be x."""
    B, n_rows, H, d = x.shape
    y = out if out is not None else torch.empty_like(x)
    _check(lib().cascade_rope_apply(_dtype_code(x), B, n_rows, H, d, x.data_ptr(), _strides(x), int(first_position),
                                    rope_table.data_ptr(), rope_table.shape[0], y.data_ptr(), _strides(y), _stream()))
    return y


def cascade_decode_step_rope(plan: Plan, q_new: torch.Tensor, k_new: torch.Tensor, v_new: torch.Tensor,
                             k_cache: torch.Tensor, v_cache: torch.Tensor, position: int, scale: float,
                             rope_table: torch.Tensor, out=None, want_lse: bool = True, workspace=None):
    """One decode step over a token-sharded cache: advances the plan to `position`, appends the new token's rotated k
    row and its v row to the caches, rotates q and runs decode + merge.  Returns (o [B, 1, H, 128], lse or None)."""
    B, _, H, d = q_new.shape
    Hkv = k_new.shape[2]
    o = out if out is not None else torch.empty_like(q_new)
    lse = torch.empty((B, 1, H), dtype=torch.float32, device=q_new.device) if want_lse else None
    nbytes = cascade_workspace_bytes(plan, CALL_DECODE_STEP_ROPE, BF16, B, H, Hkv, d)
    ws, ws_ptr, ws_bytes = _ws(nbytes, q_new.device, workspace)
    _check(lib().cascade_decode_step_rope(plan.handle, B, H, Hkv, scale, q_new.data_ptr(), _strides(q_new),
                                          k_new.data_ptr(), _strides(k_new), v_new.data_ptr(), _strides(v_new),
                                          k_cache.data_ptr(), _strides(k_cache), v_cache.data_ptr(), _strides(v_cache),
                                          int(position), rope_table.data_ptr(), rope_table.shape[0], o.data_ptr(),
                                          _strides(o), lse.data_ptr() if lse is not None else None, ws_ptr, ws_bytes,
                                          _stream()))
    return o, lse


def cascade_attn_sharded_host(plan: Plan, q_host: torch.Tensor, k_host: torch.Tensor, v_host: torch.Tensor,
                              scale: float, out_host: torch.Tensor, workspace: torch.Tensor):
    """Fused attention on dense HOST tensors (pinned for asynchronous copies): uploads, computes and downloads one KV
    head group after another with the three overlapped.  `workspace` is a device uint8 tensor of
    cascade_workspace_bytes(plan, CALL_SHARDED_HOST, ...) bytes.  Returns out_host; synchronise the current stream
    before reading it."""
    B, n_q, H, d = q_host.shape
    Hkv = k_host.shape[2]
    code = _dtype_code(q_host)
    for t in (q_host, k_host, v_host, out_host):
        assert not t.is_cuda and t.is_contiguous(), "dense host tensors expected"
    assert workspace.is_cuda and workspace.dtype == torch.uint8
    _check(lib().cascade_attn_sharded_host(plan.handle, code, B, H, Hkv, d, scale, q_host.data_ptr(),
                                           k_host.data_ptr(), v_host.data_ptr(), out_host.data_ptr(),
                                           workspace.data_ptr(), workspace.numel(), _stream()))
    return out_host


def cascade_attn_decode_static(plan: Plan, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, scale: float, out=None,
                               want_lse: bool = True):
    """Decode step (one query row per sequence) that uses the library's built-in 16 MiB scratch array instead of
    a workspace: for callers that can neither pass nor allocate scratch memory.  Only the output tensors are
    created here; the C call itself allocates nothing.  Returns (o [B, 1, H, 128], lse or None)."""
    B, n_q, H, d = q.shape
    assert n_q == 1 and d == 128 and q.dtype == torch.bfloat16
    o = out if out is not None else torch.empty((B, n_q, H, d), dtype=q.dtype, device=q.device)
    lse = torch.empty((B, n_q, H), dtype=torch.float32, device=q.device) if want_lse else None
    _check(lib().cascade_attn_decode_static(plan.handle, B, H, k.shape[2], scale, q.data_ptr(), _strides(q),
                                            k.data_ptr(), _strides(k), v.data_ptr(), _strides(v), o.data_ptr(),
                                            _strides(o), lse.data_ptr() if lse is not None else None, _stream()))
    return o, lse


def _np_ptr(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def cascade_cdelta_shard_map(n_tokens: int, c: int, delta: int):
    """(c, delta)-sharding: returns (shard_of int32 [n_tokens], alpha)."""
    out = np.empty(n_tokens, np.int32)
    alpha = ctypes.c_int32()
    _check(lib().cascade_cdelta_shard_map(n_tokens, c, delta, _np_ptr(out), ctypes.byref(alpha)))
    return out, alpha.value


def cascade_msplit_shard_map(r_shard_of, n_r_shards: int, m: int) -> np.ndarray:
    """m-split of hidden shards into query/KV shards S_{m i + x} = R_{i,x}."""
    r = np.ascontiguousarray(r_shard_of, np.int32)
    out = np.empty_like(r)
    _check(lib().cascade_msplit_shard_map(r.shape[0], _np_ptr(r), n_r_shards, m, _np_ptr(out)))
    return out


def cascade_index_set_gaps(held) -> dict:
    """Clusters and gaps of an index set given as membership flags over the tokens."""
    h = np.ascontiguousarray(np.asarray(held) != 0, np.uint8)
    vals = [ctypes.c_int32() for _ in range(4)]
    _check(lib().cascade_index_set_gaps(h.shape[0], _np_ptr(h), *[ctypes.byref(v) for v in vals]))
    return dict(zip(("n_indices", "n_clusters", "min_gap", "max_gap"), (v.value for v in vals)))


def cascade_kl_gaps(r_held, s_shard_of, n_s_shards: int) -> np.ndarray:
    """Smallest non-empty (k, l)-gap per KV shard for the node whose indices are flagged in r_held."""
    h = np.ascontiguousarray(np.asarray(r_held) != 0, np.uint8)
    s = np.ascontiguousarray(s_shard_of, np.int32)
    assert h.shape == s.shape
    out = np.empty(n_s_shards, np.int32)
    _check(lib().cascade_kl_gaps(h.shape[0], _np_ptr(h), _np_ptr(s), n_s_shards, _np_ptr(out)))
    return out
