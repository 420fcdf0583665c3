"""Host-side shard-map generators and shard-safety measures of the library against the oracle (bit-exact; no GPU)."""
import os

import numpy as np
import pytest

from oracle import sharding

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "sharding_example_n18.txt")


@pytest.fixture(scope="module")
def cb():
    from paper_2507_05228_b200 import build
    build.build_library()
    from paper_2507_05228_b200 import binding
    return binding


def _golden():
    out = {}
    for line in open(GOLDEN):
        line = line.strip()
        if line and not line.startswith("#"):
            name, vals = line.split(":")
            out[name.strip()] = [int(x) for x in vals.split()]
    return out


def _flags(n, members):
    h = np.zeros(n, np.uint8)
    h[np.asarray(members, dtype=np.int64)] = 1
    return h


def test_paper_example_through_the_library(cb):
    """Section 6.4: alpha = 3, c = 2, delta = 6, N = 18, m = 2 (the paper's ids are 1-based)."""
    g = _golden()
    r_of, alpha = cb.cascade_cdelta_shard_map(18, 2, 6)
    assert alpha == 3
    for i in range(3):
        assert (np.flatnonzero(r_of == i) + 1).tolist() == g[f"R_{i + 1}"]
    s_of = cb.cascade_msplit_shard_map(r_of, 3, 2)
    for i in range(3):
        for x in range(2):
            assert (np.flatnonzero(s_of == 2 * i + x) + 1).tolist() == g[f"R_{i + 1},{x + 1}"]
    # every listed AttnNode token set has the oracle's clusters and gaps
    for name, toks in g.items():
        held = _flags(18, [t - 1 for t in toks])
        assert cb.cascade_index_set_gaps(held) == sharding.index_set_gaps([t - 1 for t in toks]), name
    assert cb.cascade_index_set_gaps(_flags(18, [t - 1 for t in g["R_1"]]))["min_gap"] == 4  # delta - c
    R1 = _flags(18, [t - 1 for t in g["R_1"]])
    assert cb.cascade_kl_gaps(R1, r_of, 3).tolist() == [-1, 2, 2]
    assert cb.cascade_kl_gaps(R1, s_of, 6).tolist() == [-1, -1, 1, 1, 1, 1]


@pytest.mark.parametrize("n,c,delta", [(0, 1, 1), (1, 1, 1), (100, 3, 10), (512, 8, 64), (1000, 8, 96), (77, 5, 5),
                                        (4096, 1, 16), (33, 7, 30)])
def test_generators_match_the_oracle(cb, n, c, delta):
    r_of, alpha = cb.cascade_cdelta_shard_map(n, c, delta)
    assert alpha == sharding.alpha_of(c, delta)
    assert np.array_equal(r_of, sharding.cdelta_shard_of(n, c, delta))
    for m in (1, 2, 3, 4, 8):
        assert np.array_equal(cb.cascade_msplit_shard_map(r_of, alpha, m), sharding.m_split_shard_of(r_of, m))


def test_measures_match_the_oracle_on_random_sets_and_colluding_unions(cb):
    rng = np.random.default_rng(3)
    for trial in range(200):
        n = int(rng.integers(0, 60))
        held = (rng.random(n) < rng.random()).astype(np.uint8)
        assert cb.cascade_index_set_gaps(held) == sharding.index_set_gaps(np.flatnonzero(held))
        ns = int(rng.integers(1, 5))
        s_of = rng.integers(0, ns, n).astype(np.int32)
        assert np.array_equal(cb.cascade_kl_gaps(held, s_of, ns), sharding.kl_gaps(np.flatnonzero(held), s_of, ns))
    # colluding CompNodes of a (8, 64)-sharding: the union of shards i and i+1 has gaps 64 - 16, of i and i+4 gaps 24
    r_of, alpha = cb.cascade_cdelta_shard_map(1024, 8, 64)
    two = np.isin(r_of, [2, 3])
    assert cb.cascade_index_set_gaps(two) == {"n_indices": 256, "n_clusters": 16, "min_gap": 48, "max_gap": 48}
    far = np.isin(r_of, [0, 4])
    assert cb.cascade_index_set_gaps(far) == sharding.index_set_gaps(np.flatnonzero(far))
    assert cb.cascade_index_set_gaps(far)["min_gap"] == 24
    # all alpha nodes colluding hold everything: one cluster, no gap (the whole prompt is revealed)
    assert cb.cascade_index_set_gaps(np.ones(1024)) == {"n_indices": 1024, "n_clusters": 1, "min_gap": -1, "max_gap": -1}


def test_maps_feed_the_plan_builder(cb):
    r_of, alpha = cb.cascade_cdelta_shard_map(640, 8, 64)
    s_of = cb.cascade_msplit_shard_map(r_of, alpha, 4)
    plan = cb.cascade_shard_plan_host(s_of, s_of, 4 * alpha, 4 * alpha)
    q_off = plan.get("q_off")[0]
    assert np.array_equal(np.diff(q_off), np.bincount(s_of, minlength=4 * alpha))
    q_idx = plan.get("q_idx")[0]
    assert np.array_equal(q_idx[q_off[5]:q_off[6]], np.flatnonzero(s_of == 5))
    plan.destroy()


def test_argument_checks(cb):
    L = cb.lib()
    buf = np.zeros(8, np.int32)
    p = buf.ctypes.data_as(__import__("ctypes").c_void_p)
    assert L.cascade_cdelta_shard_map(8, 0, 4, p, None) == 1
    assert L.cascade_cdelta_shard_map(8, 5, 4, p, None) == 1
    assert L.cascade_cdelta_shard_map(8, 2, 4, None, None) == 1
    assert L.cascade_msplit_shard_map(8, p, 1, 0, p) == 1
    bad = np.array([0, 1, 7, 0, 0, 0, 0, 0], np.int32)
    assert L.cascade_msplit_shard_map(8, bad.ctypes.data_as(__import__("ctypes").c_void_p), 2, 2, p) == 2
    assert b"r_shard_of[2] = 7" in L.cascade_last_error()
    assert L.cascade_index_set_gaps(8, None, None, None, None, None) == 1
    assert L.cascade_kl_gaps(8, p, p, 0, p) == 1
