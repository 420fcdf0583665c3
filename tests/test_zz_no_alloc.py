"""cascade_attn_decode_static: the decode entry point that never allocates.

It exists for callers that have no scratch memory to pass and may not create any (a server whose allocator owns
all free HBM, a latency-critical decode loop, a plug-in that only sees raw pointers).  The test calls it through
the C ABI twice in a row, with different inputs, and checks each result against cascade_attn_sharded (which takes
a caller workspace) and against the oracle, so a result that depended on what the previous call left in the shared
scratch array would be caught.  The file name makes pytest collect it last.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2507_05228_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def test_decode_static_matches_workspace_path_on_two_calls_in_a_row():
    import gpu_util as gu
    from paper_2507_05228_b200 import binding as cb

    first = wl.make_workload("static_a", 6, 1, 3000, 32, 8, 128, "bf16", "round_robin", "random", 1, 16, seed=41)
    # second call: fewer shards and heads, so only part of the scratch is rewritten
    second = wl.make_workload("static_b", 3, 1, 777, 8, 2, 128, "bf16", "round_robin", "random", 1, 5, seed=42)
    for w in (first, second):
        q, k, v = gu.to_device(w)
        plan = gu.make_plan(w)
        o_ws, lse_ws = cb.cascade_attn_sharded(plan, q, k, v, w.scale)
        o_st, lse_st = cb.cascade_attn_decode_static(plan, q, k, v, w.scale)
        torch.cuda.synchronize()
        o_ref, lse_ref = oracle.attention_unsharded(w.q, w.k, w.v, w.scale, q_pos_offset=w.q_pos_offset)
        gu.check_output(o_st, lse_st, o_ref, lse_ref, w.tol, w.name + " static scratch")
        # same kernels, same inputs: the two entry points agree to well within the parity tolerance
        assert (o_st.float() - o_ws.float()).abs().max().item() <= w.tol
        assert (lse_st - lse_ws).abs().max().item() <= w.tol
        plan.destroy()


def test_decode_static_allocates_no_device_memory():
    """After a first call (which loads the module and looks the scratch array up), a raw C-ABI call with outputs the
    caller already owns leaves the device's free memory and torch's allocator exactly where they were."""
    import gpu_util as gu
    from paper_2507_05228_b200 import binding as cb

    L = cb.lib()
    S = cb._strides
    w = wl.make_workload("static_mem", 4, 1, 1024, 16, 4, 128, "bf16", "round_robin", "random", 1, 8, seed=44)
    q, k, v = gu.to_device(w)
    plan = gu.make_plan(w)
    o = torch.empty_like(q)
    lse = torch.empty((w.B, 1, w.H), dtype=torch.float32, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream

    def call():
        rc = L.cascade_attn_decode_static(plan.handle, w.B, w.H, w.Hkv, w.scale, q.data_ptr(), S(q), k.data_ptr(), S(k),
                                          v.data_ptr(), S(v), o.data_ptr(), S(o), lse.data_ptr(), stream)
        assert rc == 0, L.cascade_last_error()

    call()  # warm-up: module load, address look-up
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    alloc0, reserved0 = torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
    for _ in range(3):
        call()
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0, (free0, free1)
    assert torch.cuda.memory_allocated() == alloc0 and torch.cuda.memory_reserved() == reserved0
    o_ref, lse_ref = oracle.attention_unsharded(w.q, w.k, w.v, w.scale, q_pos_offset=w.q_pos_offset)
    gu.check_output(o, lse, o_ref, lse_ref, w.tol, "static scratch, raw call")
    plan.destroy()


def test_decode_static_rejects_oversized_and_unsupported_problems():
    import gpu_util as gu
    from paper_2507_05228_b200 import binding as cb

    L = cb.lib()
    S = cb._strides
    w = wl.make_workload("static_big", 2, 1, 64, 8, 2, 128, "bf16", "round_robin", "random", 1, 4, seed=43)
    q, k, v = gu.to_device(w)
    plan = gu.make_plan(w)
    # claim a batch whose partials cannot fit in the 16 MiB array: refused on the host, nothing is launched
    rc = L.cascade_attn_decode_static(plan.handle, 60000, 8, 2, w.scale, q.data_ptr(), S(q), k.data_ptr(), S(k),
                                      v.data_ptr(), S(v), q.data_ptr(), S(q), None, None)
    assert rc == 4 and b"16777216" in L.cascade_last_error()
    plan.destroy()
    # a prefill plan (n_q > 1) is not a decode step
    pre = wl.make_workload("static_pre", 1, 8, 64, 8, 2, 128, "bf16", "random", "random", 2, 2, seed=45)
    qp, kp, vp = gu.to_device(pre)
    plan = gu.make_plan(pre)
    rc = L.cascade_attn_decode_static(plan.handle, 1, 8, 2, pre.scale, qp.data_ptr(), S(qp), kp.data_ptr(), S(kp),
                                      vp.data_ptr(), S(vp), qp.data_ptr(), S(qp), None, None)
    assert rc == 3
    plan.destroy()
