"""The communication closed forms against the numbers the paper prints.

Section 7.1 gives CommBytes = beta F (2 d H + 2 d H_KV + 2 H) N per layer (stage A: beta d (H + 2 H_KV) N elements,
stage B: beta (d + 2) H N elements; derived in the appendix "Communication Analysis"), and Section 7.2 says the
measured totals are within 2 % of it and prints them for Bert-Base and Bert-Large at alpha = 1, 4, 8
(tests/golden/comm_bytes_table.txt).  The paper does not state F; with F = 2 bytes per element and GB = 1e9 bytes the
formula, summed over the layers, lands on all six printed values within their rounding and the stated 2 % (F = 4, a
dropped stage or a missing factor beta would miss every row) - which pins the stage-A / stage-B element counts that
the exchange tests and the benchmark compare their byte counters with.  (The "+ 2" of stage B, m and e per row, is
0.8 % of the total and is not resolved by a three-decimal table; it is fixed by the appendix's derivation.)"""
import os

import numpy as np

from paper_2507_05228_b200 import exchange as ex

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "comm_bytes_table.txt")
MODELS = {"base": dict(layers=12, H=12, d=64), "large": dict(layers=24, H=16, d=64)}


def _rows():
    with open(GOLDEN) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                a, base, large = line.split()
                yield int(a), float(base), float(large)


def test_layer_formula_reproduces_the_printed_communication_table():
    n_rows = 0
    for alpha, gb_base, gb_large in _rows():
        for name, printed in (("base", gb_base), ("large", gb_large)):
            m = MODELS[name]
            total = m["layers"] * ex.layer_comm_bytes(alpha, 2, m["d"], m["H"], m["H"], 128)
            # printed to three decimals (half a unit of the last place) and measured within 2 % of the formula
            assert abs(total / 1e9 - printed) <= 0.0005 + 0.02 * printed, (alpha, name, total)
        n_rows += 1
    assert n_rows == 3
    # the pin has teeth: four-byte elements or a forgotten stage miss the table
    m = MODELS["large"]
    assert abs(24 * ex.layer_comm_bytes(8, 4, 64, 16, 16, 128) / 1e9 - 0.203) > 0.1
    assert abs(24 * 2 * ex.stage_a_elements(1, 8, 128, 16, 16, 64) / 1e9 - 0.203) > 0.05


def test_stages_add_up_to_the_layer_formula_and_scale_linearly_in_beta():
    for beta, F, d, H, Hkv, N in ((1, 2, 64, 12, 12, 128), (4, 4, 128, 32, 8, 2048), (32, 2, 128, 64, 8, 32768)):
        a = ex.stage_a_elements(1, beta, N, H, Hkv, d)
        b = ex.stage_b_elements(1, beta, N, H, d)
        assert a == beta * d * (H + 2 * Hkv) * N and b == beta * (d + 2) * H * N
        assert ex.layer_comm_bytes(beta, F, d, H, Hkv, N) == beta * F * (2 * d * H + 2 * d * Hkv + 2 * H) * N
        assert ex.layer_comm_bytes(2 * beta, F, d, H, Hkv, N) == 2 * ex.layer_comm_bytes(beta, F, d, H, Hkv, N)
    # the partial buffers of cascade_attn_partials ARE the stage-B payload: u in the I/O type, m and l in fp32
    assert ex.stage_b_bytes(1, 32, 32768, 64, 128, 2) == 32 * 32768 * 64 * (128 * 2 + 8)
