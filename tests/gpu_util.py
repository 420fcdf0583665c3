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


def check_output(o_gpu, lse_gpu, o_ref, lse_ref, tol, what=""):
    o = o_gpu.double().cpu().numpy() if torch.is_tensor(o_gpu) else o_gpu
    assert np.isfinite(o).all(), f"{what}: non-finite output"
    err = np.abs(o - o_ref).max()
    assert err <= tol, f"{what}: o max-abs {err:.3e} > {tol}"
    if lse_gpu is not None:
        lse = lse_gpu.double().cpu().numpy() if torch.is_tensor(lse_gpu) else lse_gpu
        fin = np.isfinite(lse_ref)
        assert np.array_equal(np.isfinite(lse), fin), f"{what}: lse finiteness differs"
        err_l = np.abs(lse[fin] - lse_ref[fin]).max() if fin.any() else 0.0
        assert err_l <= tol, f"{what}: lse max-abs {err_l:.3e} > {tol}"
    return err


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
    e_merge = check_output(o_m, lse_m if check_lse else None, o_ref, lse_ref, w.tol, w.name + " merge")
    o_f, lse_f = cb.cascade_attn_sharded(plan, q, k, v, w.scale)
    e_fused = check_output(o_f, lse_f if check_lse else None, o_ref, lse_ref, w.tol, w.name + " fused")
    # both routes are within tol of the exact result, hence within 2 tol of each other
    d = (o_f.double() - o_m.double()).abs().max().item()
    assert d <= 2 * w.tol, f"{w.name}: fused vs merge(partials) {d:.3e}"
    assert plan.device_status() == 0
    plan.destroy()
    return errs, e_merge, e_fused


def sampled_parity(w, per_shard=2, partial_shards=None):
    """Full-size run on the GPU; the oracle evaluates a stratified sample of query rows (all heads)."""
    q, k, v = to_device(w)
    plan = make_plan(w)
    oplan = oracle_plan(w)
    assert np.array_equal(plan.get("vis")[0], oplan.vis)
    rows = wl.sample_rows(w, per_shard)
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
    e_merge = check_output(o_m[:, rt], lse_m[:, rt], o_ref, lse_ref, w.tol, w.name + " merge (sampled rows)")
    del o_part, m_part, l_part
    o_f, lse_f = cb.cascade_attn_sharded(plan, q, k, v, w.scale)
    e_fused = check_output(o_f[:, rt], lse_f[:, rt], o_ref, lse_ref, w.tol, w.name + " fused (sampled rows)")
    # properties that hold at any size: finite everywhere, fused == merge(partials) on every row
    assert torch.isfinite(o_f.float()).all() and torch.isfinite(lse_f).all()
    d = (o_f.float() - o_m.float()).abs().max().item()  # each within tol of the exact result
    assert d <= 2 * w.tol, f"{w.name}: fused vs merge(partials) over all rows {d:.3e}"
    assert plan.device_status() == 0
    plan.destroy()
    return errs, e_merge, e_fused
