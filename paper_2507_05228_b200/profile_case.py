"""Runs one workload through one route a few times, for profiling with ncu or quick timing.

    python -m paper_2507_05228_b200.profile_case <workload> <route> [--launches N] [--override k=v ...]

workload: c1_tiny_f32 | c2_prefill_8b | c3_batched | c4_long_70b | c5_decode
route:    fused | fused_rope | partials | merge | decode
Prints the median CUDA-event time per launch (L2 flushed between launches).
"""
from __future__ import annotations

import argparse
import statistics

import numpy as np
import torch

from . import binding as cb
from . import workloads as wl


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("workload")
    ap.add_argument("route", choices=["fused", "fused_rope", "partials", "merge", "decode"])
    ap.add_argument("--launches", type=int, default=3)
    ap.add_argument("--override", nargs="*", default=[])
    args = ap.parse_args()
    over = {}
    for kv in args.override:
        k, v = kv.split("=")
        over[k] = int(v)
    w = wl.config(args.workload, **over)
    up = lambda a: (torch.from_numpy(wl.bf16_bits(a).view(np.int16)).cuda().view(torch.bfloat16)
                    if w.dtype == "bf16" else torch.from_numpy(a).cuda())
    q, k, v = up(w.q), up(w.k), up(w.v)
    plan = cb.cascade_shard_plan(w.q_shard_of, w.kv_shard_of, w.n_q_shards, w.n_kv_shards, w.q_pos_offset, w.causal)
    o = torch.empty_like(q)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    parts = None
    ws = None
    if w.n_q > 1:
        nb = cb.cascade_workspace_bytes(plan, cb.CALL_SHARDED, cb.BF16 if w.dtype == "bf16" else cb.F32, w.B, w.H, w.Hkv,
                                        w.d)
        ws = torch.empty(max(nb, 1), dtype=torch.uint8, device="cuda")
    if args.route in ("partials", "merge", "decode"):
        parts = cb.cascade_attn_partials(plan, q, k, v, w.scale, workspace=ws)
    table = cb.cascade_rope_table(max(w.q_pos_offset + w.n_q, w.n_kv), w.d, 500000.0) if args.route == "fused_rope" else None
    fn = {
        "fused_rope": lambda: cb.cascade_attn_sharded_rope(plan, q, k, v, w.scale, table, out=o, want_lse=False,
                                                           workspace=ws),
        "fused": lambda: cb.cascade_attn_sharded(plan, q, k, v, w.scale, out=o, want_lse=False, workspace=ws),
        "partials": lambda: cb.cascade_attn_partials(plan, q, k, v, w.scale, out=parts, workspace=ws),
        "decode": lambda: cb.cascade_attn_partials(plan, q, k, v, w.scale, out=parts),
        "merge": lambda: cb.cascade_merge(*parts, plan.dev_ptr("q_idx") if w.n_q > 1 else 0, out=o, want_lse=False),
    }[args.route]
    if args.route == "fused" and w.n_q == 1:
        ws = torch.empty(cb.cascade_workspace_bytes(plan, cb.CALL_SHARDED, cb.BF16, w.B, w.H, w.Hkv, w.d),
                         dtype=torch.uint8, device="cuda")
        fn = lambda: cb.cascade_attn_sharded(plan, q, k, v, w.scale, out=o, want_lse=False, workspace=ws)
    ms = []
    for _ in range(args.launches):
        flush.fill_(1)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        fn()
        b.record()
        torch.cuda.synchronize()
        ms.append(a.elapsed_time(b))
    print(f"{args.workload} {args.route}: median {statistics.median(ms):.4f} ms over {args.launches} launches; "
          f"{w.flops() / 1e12:.3f} TFLOP algorithmic, {w.kv_bytes() / 1e9:.3f} GB K+V; status {plan.device_status()}")
    plan.destroy()


if __name__ == "__main__":
    main()
