"""The host-buffer entry point (upload, fused attention and download pipelined over the KV heads) against the oracle
and against the device entry point, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from paper_2507_05228_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def gu():
    import gpu_util
    return gpu_util


@pytest.fixture(scope="module")
def cb():
    from paper_2507_05228_b200 import binding
    return binding


def _host(w, a):
    if w.dtype == "bf16":
        return torch.from_numpy(wl.bf16_bits(a).view(np.int16)).view(torch.bfloat16).pin_memory()
    return torch.from_numpy(a).pin_memory()


@pytest.mark.parametrize("case", [
    dict(B=2, n_q=600, n_kv=600, H=8, Hkv=2, d=128, dtype="bf16", q_map="random", kv_map="random", n_q_shards=5,
         n_kv_shards=5),                                                     # tensor-core route, two sequences
    dict(B=1, n_q=256, n_kv=256, H=8, Hkv=8, d=64, dtype="f32", q_map="round_robin", kv_map="round_robin",
         n_q_shards=4, n_kv_shards=4),                                       # fp32 ALU route, no head sharing
    dict(B=3, n_q=1, n_kv=1000, H=16, Hkv=4, d=128, dtype="bf16", q_map="round_robin", kv_map="random", n_q_shards=1,
         n_kv_shards=7),                                                     # decode route
])
def test_host_call_matches_oracle_and_device_call(cb, gu, case):
    w = wl.make_workload("host_call", seed=31, **case)
    plan = gu.make_plan(w)
    code = cb.BF16 if w.dtype == "bf16" else cb.F32
    hq, hk, hv = _host(w, w.q), _host(w, w.k), _host(w, w.v)
    ho = torch.empty_like(hq).pin_memory()
    need = cb.cascade_workspace_bytes(plan, cb.CALL_SHARDED_HOST, code, w.B, w.H, w.Hkv, w.d)
    assert need >= 2 * hq.numel() * hq.element_size() + 2 * hk.numel() * hk.element_size()
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    o_ref, _ = oracle.attention_unsharded(w.q, w.k, w.v, w.scale, causal=w.causal, q_pos_offset=w.q_pos_offset)
    for _ in range(2):  # the second call reuses the streams, events and the workspace
        ho.zero_()
        cb.cascade_attn_sharded_host(plan, hq, hk, hv, w.scale, ho, ws)
        torch.cuda.current_stream().synchronize()
        gu.check_output(ho.double().numpy(), None, o_ref, None, w.tol, "host call")
    q, k, v = gu.to_device(w)
    o_dev, _ = cb.cascade_attn_sharded(plan, q, k, v, w.scale)
    assert torch.equal(o_dev.cpu(), ho)  # head groups are independent: the same kernels on the same data
    with pytest.raises(cb.CascadeError) as ei:
        cb.cascade_attn_sharded_host(plan, hq, hk, hv, w.scale, ho, ws[: need - 256])
    assert ei.value.status == 4
    assert plan.device_status() == 0
    plan.destroy()
