"""The index-checking build of the library (-DCASCADE_DEBUG) on small cases of every route.

In that build every row index a kernel takes out of a plan array is checked against the tensor it indexes before an
address is formed; a violation is recorded in the plan's status word instead of becoming a stray access.  The cases run
in a child process that loads libcascade_b200_debug.so in place of the release library (CASCADE_B200_LIB) and must end
with parity against the oracle and a clean status word.  This is the stand-in for a device memory checker."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
CHILD = r"""
import sys
sys.path.insert(0, %(root)r); sys.path.insert(0, %(tests)r)
import numpy as np, torch
from paper_2507_05228_b200 import binding as cb, workloads as wl
import gpu_util as gu
assert cb.LIB_PATH.endswith("libcascade_b200_debug.so"), cb.LIB_PATH
cases = [wl.config("c2_prefill_8b", n_q=512, n_kv=512, H=8, Hkv=2), wl.config("c1_tiny_f32"),
         wl.config("c5_decode", B=3, n_kv=1500),
         wl.make_workload("dbg_ragged", 2, 333, 333, 4, 1, 128, "bf16", "random", "contiguous", 2, 7, seed=95),
         wl.make_workload("dbg_chunk", 1, 96, 400, 8, 2, 128, "bf16", "random", "random", 3, 7, seed=96)]
for w in cases:
    gu.full_parity(w)   # plan arrays, partials, merge, fused; asserts the status word is 0
print("debug build: %%d cases clean" %% len(cases))
"""


def test_small_cases_run_clean_on_the_index_checking_build():
    from paper_2507_05228_b200 import build
    lib = build.build_library(debug=True)  # compiles only if the library is missing or older than its sources
    env = dict(os.environ, CASCADE_B200_LIB=lib)
    out = subprocess.run([sys.executable, "-c", CHILD % {"root": ROOT, "tests": os.path.join(ROOT, "tests")}], env=env,
                         capture_output=True, text=True, timeout=900)
    assert out.returncode == 0, out.stdout[-2000:] + out.stderr[-4000:]
    assert "cases clean" in out.stdout
