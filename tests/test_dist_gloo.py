"""The N>1 host logic (unit sharding, barrier, max-over-ranks timing) under gloo with two CPU processes."""
import os
import socket

import torch.multiprocessing as mp


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    from paper_2507_05228_b200 import dist as cd
    r, w, _ = cd.init("gloo")
    units = list(cd.shard_units(7, r, w))
    cd.barrier()
    t_max = cd.max_over_ranks(1.0 + r)
    total = cd.sum_over_ranks(len(units))
    out.put((r, units, t_max, total))
    cd.finalize()


def test_two_rank_gloo_sharding_and_reductions():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, u0, t0, s0), (r1, u1, t1, s1) = res
    assert u0 == [0, 1, 2, 3] and u1 == [4, 5, 6]
    assert t0 == t1 == 2.0 and s0 == s1 == 7.0


def test_shard_units_cover_exactly_once():
    from paper_2507_05228_b200 import dist as cd
    for n in (0, 1, 5, 8, 64):
        for w in (1, 2, 3, 8):
            got = [u for r in range(w) for u in cd.shard_units(n, r, w)]
            assert got == list(range(n))
