"""The multi-rank form of the path on one GPU: every rank's share is run in turn in one process (no kernel waits on
another), the stage-B all-to-all is delivered in-process, and each rank's post-pass is compared with the oracle.

Per rank: K/V rows of its own shards only (cascade_shard_plan_resident), partials against every query row
(cascade_attn_partials), rows routed to their owner (exchange.StageB), cascade_merge on what arrived."""
import numpy as np
import pytest
import torch

import oracle
from paper_2507_05228_b200 import exchange as ex
from paper_2507_05228_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def gu():
    import gpu_util
    return gpu_util


def _run_ranks(gu, w, world):
    q, k, v = gu.to_device(w)
    oplan = oracle.shard_plan(w.q_shard_of, w.kv_shard_of, w.n_q_shards, w.n_kv_shards, w.q_pos_offset, w.causal)
    u_ref, m_ref, e_ref = oracle.attn_pass(w.q, w.k, w.v, w.scale, oplan)
    o_ref, lse_ref = oracle.attention_unsharded(w.q, w.k, w.v, w.scale, causal=w.causal, q_pos_offset=w.q_pos_offset)
    ranks = [ex.RankAttention(w.q_shard_of, w.kv_shard_of, w.n_q_shards, w.n_kv_shards, r, world, w.q_pos_offset,
                              w.causal) for r in range(world)]
    packed, sent = [], 0
    for r, ra in enumerate(ranks):
        tok = torch.from_numpy(ra.tokens.astype(np.int64)).cuda()
        k_res, v_res = k[:, tok].contiguous(), v[:, tok].contiguous()  # the rows this rank keeps, nothing else
        o_part, m_part, l_part = ra.partials(q, k_res, v_res, w.scale)
        torch.cuda.synchronize()
        mine = ex.owned_shards(w.n_kv_shards, r, world)
        gu.check_partials((o_part.double().cpu().numpy(), m_part.double().cpu().numpy(), l_part.double().cpu().numpy()),
                          (u_ref[:, mine], m_ref[:, mine], e_ref[:, mine]), w.tol, f"{w.name} rank {r}/{world} partials")
        packed.append(ra.stage.pack(o_part, m_part, l_part))
        sent += sum(t.numel() * t.element_size() for t in packed[-1][:2])
        assert ra.plan.device_status() == 0
    es = 2 if w.dtype == "bf16" else 4
    assert sent == ex.stage_b_bytes(w.B, w.n_kv_shards, w.n_q, w.H, w.d, es)
    got = ex.deliver_in_process([ra.stage for ra in ranks], packed, w.B, w.H, w.d)
    sources = [ra.parts for ra in ranks]  # every rank's partial buffers, left where they were written
    seen = []
    for r, ra in enumerate(ranks):
        o, lse = ra.combine(*got[r])
        rows = ra.owned_tokens
        # the one-kernel form of stage B + post-pass reads the same parts in place: same arithmetic, same result
        o_d, lse_d = ra.combine_in_place(sources)
        assert o_d.shape == o.shape
        if rows.size:
            gu.check_output(o_d, lse_d, o_ref[:, rows], lse_ref[:, rows], w.tol, f"{w.name} rank {r}/{world} in place",
                            stored_partials=True)
            assert (o_d.float() - o.float()).abs().max().item() <= 2.0 ** -6  # summation order differs at most
        gu.check_output(o, lse, o_ref[:, rows], lse_ref[:, rows], w.tol, f"{w.name} rank {r}/{world} post-pass",
                        stored_partials=True)
        seen.append(rows)
        ra.destroy()
    assert np.array_equal(np.sort(np.concatenate(seen)), np.arange(w.n_q))


@pytest.mark.parametrize("world", [1, 2, 3])
def test_ranks_with_resident_kv_on_the_tensor_core_route(gu, world):
    _run_ranks(gu, wl.config("c2_prefill_8b", n_q=768, n_kv=768, H=8, Hkv=2, n_q_shards=6, n_kv_shards=6), world)


def test_ranks_on_the_other_routes(gu):
    _run_ranks(gu, wl.config("c1_tiny_f32"), 2)
    _run_ranks(gu, wl.make_workload("decode_ranks", 3, 1, 900, 8, 2, 128, "bf16", "round_robin", "random", 1, 6, seed=61), 3)
    _run_ranks(gu, wl.make_workload("bidir_ranks", 1, 200, 200, 4, 4, 128, "bf16", "random", "random", 4, 5, seed=62,
                                    causal=False), 2)
