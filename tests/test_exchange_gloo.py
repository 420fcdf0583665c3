"""Stage-B exchange on two CPU ranks (gloo): the routing of partial rows to their owner, on the oracle's partials.

Each rank is given the (u, m, e) columns of its own KV shards (taken from the oracle: this test is about the routing,
not about a kernel), runs the all-to-all, and checks that
  * it receives exactly the rows of its query shards, parts in global KV-shard order, rows in shard-major order,
  * the bytes handed to the collective, summed over ranks, equal the closed form of the paper's communication
    analysis: beta (d + 2) H N elements per sequence,
  * the post-pass of what arrived equals unsharded attention on the rows it owns.
"""
import os
import socket

import numpy as np
import torch
import torch.multiprocessing as mp


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


CASES = [
    # name, B, n, H, Hkv, d, q shards, kv shards, map kinds
    ("symmetric_perm", 2, 96, 4, 2, 16, 4, 4, "random"),
    ("odd_counts", 1, 75, 3, 3, 8, 3, 5, "random"),
    ("block_rr", 1, 128, 2, 1, 32, 6, 6, "block_rr"),
]


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    import oracle
    from paper_2507_05228_b200 import dist as cd
    from paper_2507_05228_b200 import exchange as ex
    from paper_2507_05228_b200 import workloads as wl
    cd.init("gloo")
    results = []
    for name, B, n, H, Hkv, d, J, P, kind in CASES:
        w = wl.make_workload(name, B, n, n, H, Hkv, d, "f32", kind, kind, J, P, seed=70 + J, block=8)
        plan = oracle.shard_plan(w.q_shard_of, w.kv_shard_of, J, P)
        u, m, e = oracle.attn_pass(w.q, w.k, w.v, w.scale, plan)  # [B, P, n, H, d], [B, P, n, H]
        mine = ex.owned_shards(P, rank, world)
        stage = ex.StageB(plan.q_off, P, rank, world)
        got_u, got_m, got_e, nbytes = stage.exchange(torch.from_numpy(u[:, mine]).contiguous(),
                                                     torch.from_numpy(m[:, mine]).contiguous(),
                                                     torch.from_numpy(e[:, mine]).contiguous())
        # exactly my rows, all parts, in order
        slots = np.concatenate([np.arange(plan.q_off[j], plan.q_off[j + 1]) for j in range(rank, J, world)])
        assert np.array_equal(stage.my_slots, slots)
        assert np.array_equal(got_u.numpy(), u[:, :, slots]) and np.array_equal(got_m.numpy(), m[:, :, slots])
        assert np.array_equal(got_e.numpy(), e[:, :, slots])
        # post-pass of what arrived == unsharded attention on the rows this rank owns
        o, lse = oracle.post_pass(got_u.numpy(), got_m.numpy(), got_e.numpy())
        tokens = plan.q_idx[slots]
        o_ref, lse_ref = oracle.attention_unsharded(w.q, w.k, w.v, w.scale, rows=tokens.astype(np.int32))
        assert np.abs(o - o_ref).max() < 1e-12 and np.abs(lse - lse_ref).max() < 1e-12
        total = cd.sum_over_ranks(float(nbytes))
        results.append((name, total, ex.stage_b_elements(B, P, n, H, d) * 8, slots.size))
    out.put((rank, results))
    cd.finalize()


def test_two_rank_stage_b_exchange_routes_rows_and_matches_closed_form():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = dict(out.get(timeout=300) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for (name, total, closed, rows0), (_, total1, _, rows1), case in zip(res[0], res[1], CASES):
        # fp64 payload here: 8 bytes per element, (d + 2) elements per (part, row, head)
        assert total == total1 == closed, (name, total, closed)
        assert rows0 + rows1 == case[2]


def test_routing_tables_cover_every_row_once_and_byte_forms_agree():
    from paper_2507_05228_b200 import exchange as ex
    q_off = np.array([0, 5, 5, 12, 20, 21])
    for world in (1, 2, 3, 5):
        stages = [ex.StageB(q_off, 7, r, world) for r in range(world)]
        allslots = np.sort(np.concatenate([s.my_slots for s in stages]))
        assert np.array_equal(allslots, np.arange(21))
        assert sum(s.n_local_of[s.rank] for s in stages) == 7
    # bytes: bf16 u, fp32 m and e
    assert ex.stage_b_bytes(2, 4, 10, 3, 128, 2) == 2 * 4 * 10 * 3 * (256 + 8)
    assert ex.stage_b_elements(2, 4, 10, 3, 128) == 2 * 4 * 130 * 3 * 10


def test_in_process_delivery_equals_the_collective_layout():
    """deliver_in_process (all ranks played by one process) hands every rank what the all-to-all would."""
    from paper_2507_05228_b200 import exchange as ex
    rng = np.random.Generator(np.random.PCG64(3))
    B, n, H, d, J, P, world = 2, 23, 3, 4, 5, 7, 3
    q_off = np.array([0, 4, 9, 9, 17, 23])
    u = rng.standard_normal((B, P, n, H, d)).astype(np.float32)
    m = rng.standard_normal((B, P, n, H)).astype(np.float32)
    l = rng.uniform(1, 2, (B, P, n, H)).astype(np.float32)
    stages = [ex.StageB(q_off, P, r, world) for r in range(world)]
    packed = []
    for r in range(world):
        mine = ex.owned_shards(P, r, world)
        packed.append(stages[r].pack(torch.from_numpy(u[:, mine]).contiguous(), torch.from_numpy(m[:, mine]).contiguous(),
                                     torch.from_numpy(l[:, mine]).contiguous()))
    got = ex.deliver_in_process(stages, packed, B, H, d)
    for r in range(world):
        s = stages[r].my_slots
        assert np.array_equal(got[r][0].numpy(), u[:, :, s]) and np.array_equal(got[r][1].numpy(), m[:, :, s])
        assert np.array_equal(got[r][2].numpy(), l[:, :, s])
