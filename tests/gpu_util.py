"""Helpers for the GPU parity tests: upload a workload, run the library, compare with the oracle."""
import numpy as np
import torch

import oracle
from paper_2507_05228_b200 import binding as cb
from paper_2507_05228_b200 import workloads as wl


def to_device(w, which=("q", "k", "v")):
    out = []
    for name in which:
        a = getattr(w, name)
        if w.dtype == "bf16":
            t = torch.from_numpy(wl.bf16_bits(a).view(np.int16)).cuda().view(torch.bfloat16)
        else:
            t = torch.from_numpy(a).cuda()
        out.append(t)
    return out


def make_plan(w):
    return cb.cascade_shard_plan(w.q_shard_of, w.kv_shard_of, w.n_q_shards, w.n_kv_shards,
                                 q_pos_offset=w.q_pos_offset, causal=w.causal)


def oracle_plan(w):
    return oracle.shard_plan(w.q_shard_of, w.kv_shard_of, w.n_q_shards, w.n_kv_shards,
                             q_pos_offset=w.q_pos_offset, causal=w.causal)


def check_partials(got, ref, tol, what=""):
    """got = (o, m, l) numpy float64 from the GPU; ref = (u, m, e) from the oracle; same shapes."""
    go, gm, gl = got
    u, m, e = ref
    empty = e == 0
    assert np.array_equal(np.isneginf(gm), empty), f"{what}: pattern of empty rows differs"
    assert (gl[empty] == 0).all() and (go[empty] == 0).all(), f"{what}: empty rows must be l=0, o=0"
    ne = ~empty
    err_o = np.abs(go - u).max() if go.size else 0.0
    err_m = np.abs(gm[ne] - m[ne]).max() if ne.any() else 0.0
    err_l = (np.abs(gl[ne] - e[ne]) / np.maximum(1.0, e[ne])).max() if ne.any() else 0.0
    err_lse = np.abs((gm[ne] + np.log(gl[ne])) - (m[ne] + np.log(e[ne]))).max() if ne.any() else 0.0
    assert np.isfinite(go).all(), f"{what}: non-finite partial output"
    assert err_o <= tol, f"{what}: partial o max-abs {err_o:.3e} > {tol}"
    assert err_m <= tol, f"{what}: m max-abs {err_m:.3e} > {tol}"
    assert err_l <= tol, f"{what}: l rel {err_l:.3e} > {tol}"
    assert err_lse <= tol, f"{what}: m + ln l {err_lse:.3e} > {tol}"
    return err_o, err_m, err_l


BF16_HALF_ULP_AT_4 = 2.0 ** -6  # spacing of bf16 in [4, 8) is 2^-5


def check_output(o_gpu, lse_gpu, o_ref, lse_ref, tol, what="", stored_partials=False):
    """stored_partials: the output was combined from partials that were themselves stored in bf16 (the unfused route:
    the paper's stage-B payload has F bytes per element).  Such an output carries two bf16 roundings.  While every
    value involved stays below 4 they sum to at most 2 * 2^-7 < tol; a partial in [4, 8) is stored with up to
    2^-6 = 0.0156 of error, which alone takes most of the 0.02.  Where the exact output reaches 3.5 (a partial of
    magnitude 4 or more then carries nearly all the weight) the bound is therefore tol plus that half-ulp.  Outputs
    computed in one go (fused route) stay at tol everywhere."""
    o = o_gpu.double().cpu().numpy() if torch.is_tensor(o_gpu) else o_gpu
    assert np.isfinite(o).all(), f"{what}: non-finite output"
    allowed = np.full(o_ref.shape, tol)
    if stored_partials and tol > 1e-3:
        allowed = allowed + BF16_HALF_ULP_AT_4 * (np.abs(o_ref) >= 3.5)
    excess = (np.abs(o - o_ref) - allowed).max() if o.size else -1.0
    err = np.abs(o - o_ref).max() if o.size else 0.0
    assert excess <= 0, f"{what}: o max-abs {err:.3e}, {excess:.3e} over the bound ({tol})"
    if lse_gpu is not None:
        lse = lse_gpu.double().cpu().numpy() if torch.is_tensor(lse_gpu) else lse_gpu
        fin = np.isfinite(lse_ref)
        assert np.array_equal(np.isfinite(lse), fin), f"{what}: lse finiteness differs"
        err_l = np.abs(lse[fin] - lse_ref[fin]).max() if fin.any() else 0.0
        assert err_l <= tol, f"{what}: lse max-abs {err_l:.3e} > {tol}"
    return err


def _check_routes_agree(o_f, o_m, w):
    """Fused output against merge(partials) on every element: tol each, plus the stored partial's half-ulp from 4 on."""
    diff = (o_f.float() - o_m.float()).abs()
    allowed = 2 * w.tol + (BF16_HALF_ULP_AT_4 if w.dtype == "bf16" else 0.0) * (o_f.float().abs() >= 3.4).float()
    excess = (diff - allowed).max().item()
    assert excess <= 0, f"{w.name}: fused vs merge(partials): {diff.max().item():.3e}, {excess:.3e} over the bound"


def full_parity(w, check_lse=True):
    """Every element of partials, merge and the fused call against the oracle.  Returns the error triple."""
    q, k, v = to_device(w)
    plan = make_plan(w)
    oplan = oracle_plan(w)
    for f in ("q_idx", "kv_idx", "vis", "pair_class", "q_off", "kv_off"):
        assert np.array_equal(plan.get(f)[0], getattr(oplan, f)), f
    u, m, e = oracle.attn_pass(w.q, w.k, w.v, w.scale, oplan)
    o_ref, lse_ref = oracle.attention_unsharded(w.q, w.k, w.v, w.scale, causal=w.causal,
                                                q_pos_offset=w.q_pos_offset)
    o_part, m_part, l_part = cb.cascade_attn_partials(plan, q, k, v, w.scale)
    torch.cuda.synchronize()
    errs = check_partials((o_part.double().cpu().numpy(), m_part.double().cpu().numpy(),
                           l_part.double().cpu().numpy()), (u, m, e), w.tol, w.name + " partials")
    o_m, lse_m = cb.cascade_merge(o_part, m_part, l_part, plan.dev_ptr("q_idx"))
    e_merge = check_output(o_m, lse_m if check_lse else None, o_ref, lse_ref, w.tol, w.name + " merge",
                           stored_partials=True)
    o_f, lse_f = cb.cascade_attn_sharded(plan, q, k, v, w.scale)
    e_fused = check_output(o_f, lse_f if check_lse else None, o_ref, lse_ref, w.tol, w.name + " fused")
    # both routes are within their bound of the exact result, hence within the sum of the bounds of each other
    _check_routes_agree(o_f, o_m, w)
    assert plan.device_status() == 0
    plan.destroy()
    return errs, e_merge, e_fused


def sampled_parity(w, per_shard=2, min_rows=0):
    """Full-size run on the GPU; the oracle evaluates a stratified sample of query rows (all heads), which includes the
    rows at tile and sub-tile boundaries of every shard."""
    q, k, v = to_device(w)
    plan = make_plan(w)
    oplan = oracle_plan(w)
    assert np.array_equal(plan.get("vis")[0], oplan.vis)
    rows = wl.sample_rows(w, per_shard, tile_edges=True)
    assert rows.size >= min_rows, (rows.size, min_rows)
    slots = oplan.q_inv[rows]
    o_ref, lse_ref = oracle.attention_unsharded(w.q, w.k, w.v, w.scale, causal=w.causal,
                                                q_pos_offset=w.q_pos_offset, rows=rows)
    u, m, e = oracle.attn_pass(w.q, w.k, w.v, w.scale, oplan, row_tokens=rows)
    o_part, m_part, l_part = cb.cascade_attn_partials(plan, q, k, v, w.scale)
    torch.cuda.synchronize()
    st = torch.from_numpy(slots.astype(np.int64)).cuda()
    got = (o_part[:, :, st].double().cpu().numpy(), m_part[:, :, st].double().cpu().numpy(),
           l_part[:, :, st].double().cpu().numpy())
    errs = check_partials(got, (u, m, e), w.tol, w.name + " partials (sampled rows)")
    rt = torch.from_numpy(rows.astype(np.int64)).cuda()
    o_m, lse_m = cb.cascade_merge(o_part, m_part, l_part, plan.dev_ptr("q_idx"))
    e_merge = check_output(o_m[:, rt], lse_m[:, rt], o_ref, lse_ref, w.tol, w.name + " merge (sampled rows)",
                           stored_partials=True)
    del o_part, m_part, l_part
    o_f, lse_f = cb.cascade_attn_sharded(plan, q, k, v, w.scale)
    e_fused = check_output(o_f[:, rt], lse_f[:, rt], o_ref, lse_ref, w.tol, w.name + " fused (sampled rows)")
    # properties that hold at any size: finite everywhere, fused == merge(partials) on every row
    assert torch.isfinite(o_f.float()).all() and torch.isfinite(lse_f).all()
    _check_routes_agree(o_f, o_m, w)
    assert plan.device_status() == 0
    plan.destroy()
    return errs, e_merge, e_fused


class _DevicePointer:
    """A raw device pointer presented through the CUDA array interface, so that torch can copy it to the host."""

    def __init__(self, ptr, n, typestr):
        self.__cuda_array_interface__ = {"shape": (n,), "typestr": typestr, "data": (int(ptr), False), "version": 2}


def read_plan_device_array(plan, field):
    """Device copy of a plan array, fetched with the pointer cascade_plan_get returns (not the library's host copy)."""
    shape = plan._shape(field)
    n = int(np.prod(shape))
    torch.cuda.synchronize()
    t = torch.as_tensor(_DevicePointer(plan.dev_ptr(field), n, "|u1" if field == "pair_class" else "<i4"), device="cuda")
    return t.cpu().numpy().reshape(shape)
