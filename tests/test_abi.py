"""The C-ABI library loads, exports every symbol the header declares, and rejects bad arguments on the host
(no GPU needed: nothing here launches a kernel)."""
import ctypes
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def binding():
    from paper_2507_05228_b200 import build
    build.build_library()
    from paper_2507_05228_b200 import binding as b
    return b


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "cascade.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(cascade_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(binding):
    names = _declared_functions()
    assert {"cascade_shard_plan", "cascade_attn_partials", "cascade_merge", "cascade_attn_sharded"} <= set(names)
    L = binding.lib()
    for n in names:
        assert hasattr(L, n), n
    assert set(binding.EXPORTS) == set(names)
    assert binding.cascade_version() >= 100


def test_library_does_not_import_or_link_the_oracle():
    pkg = os.path.join(ROOT, "paper_2507_05228_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in src.lower() or f == "workloads.py", f
    src = open(os.path.join(pkg, "workloads.py")).read()
    assert "import oracle" not in src and "from oracle" not in src


def test_host_side_argument_checks(binding):
    L = binding.lib()
    out = ctypes.c_void_p()
    good = np.zeros(8, np.int32)
    p = good.ctypes.data_as(ctypes.c_void_p)
    assert L.cascade_shard_plan_host(1, 8, 8, None, p, 1, 1, 0, 1, ctypes.byref(out)) == 1
    assert L.cascade_shard_plan_host(1, 0, 8, p, p, 1, 1, 0, 1, ctypes.byref(out)) == 1
    bad = np.array([0, 1, 2, 5, 0, 1, 2, 0], np.int32)
    assert L.cascade_shard_plan_host(1, 8, 8, bad.ctypes.data_as(ctypes.c_void_p), p, 3, 1, 0, 1,
                                     ctypes.byref(out)) == 2
    assert b"q_shard_of[3] = 5" in L.cascade_last_error()
    neg = np.array([0, -1], np.int32)
    assert L.cascade_shard_plan_host(1, 2, 2, neg.ctypes.data_as(ctypes.c_void_p), p, 1, 1, 0, 1,
                                     ctypes.byref(out)) == 2
    # merge: null pointers / unsupported shapes are refused before any CUDA call
    S = binding.Strides(0, 0, 0)
    assert L.cascade_merge(1, 1, 2, 4, 2, 128, None, None, None, None, 0, None, S, None, None) == 1
    assert L.cascade_merge(1, 1, 2, 4, 2, 96, 256, 256, 256, None, 0, 256, S, None, None) == 3
    assert L.cascade_merge(7, 1, 2, 4, 2, 128, 256, 256, 256, None, 0, 256, S, None, None) == 3
    assert L.cascade_merge(1, 1, 2, 4, 2, 128, 264, 256, 256, None, 0, 256, S, None, None) == 1  # misaligned
    # a host-only plan is readable but cannot be used by the attention calls
    plan = binding.cascade_shard_plan_host(good, good, 1, 1)
    assert plan.get("q_idx").tolist() == [list(range(8))]
    S4 = binding.Strides(1024, 128, 128)
    rc = L.cascade_attn_partials(plan.handle, 1, 1, 1, 1, 128, 1.0, 256, S4, 256, S4, 256, S4, 256, 256, 256,
                                 None, 0, None)
    assert rc == 1 and b"cascade_shard_plan_host" in L.cascade_last_error()
    # the host-buffer call refuses null pointers and a host-only plan before touching CUDA; its workspace size is
    # staging for q, k, v, o plus one head group's scratch
    hb = np.zeros(16, np.uint8).ctypes.data_as(ctypes.c_void_p)
    assert L.cascade_attn_sharded_host(plan.handle, 1, 1, 4, 2, 128, 1.0, None, hb, hb, hb, hb, 0, None) == 1
    assert L.cascade_attn_sharded_host(plan.handle, 1, 1, 4, 2, 128, 1.0, hb, hb, hb, hb, hb, 0, None) == 1
    assert b"cascade_shard_plan_host" in L.cascade_last_error()
    nbytes = ctypes.c_size_t()
    assert L.cascade_workspace_bytes(plan.handle, 2, 1, 1, 4, 2, 128, ctypes.byref(nbytes)) == 0
    q_b, kv_b = 8 * 4 * 128 * 2, 8 * 2 * 128 * 2
    assert nbytes.value >= 2 * q_b + 2 * kv_b and nbytes.value % 256 == 0
    assert L.cascade_workspace_bytes(plan.handle, 0, 1, 1, 4, 3, 128, ctypes.byref(nbytes)) == 1
    assert L.cascade_workspace_bytes(plan.handle, 9, 1, 1, 4, 2, 128, ctypes.byref(nbytes)) == 1
    plan.destroy()
