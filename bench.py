#!/usr/bin/env python
"""Benchmark of the sequence-sharded attention hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--no-extras]

One step = one pass of the hot path over one batch of the headline workload (the Llama-8B-shaped prefill
layer: 2048 tokens, 32 query / 8 KV heads, head_dim 128, bf16, 8 x 8 random shards): the fused call
``cascade_attn_sharded`` (gather, QK^T, mask, streaming statistics, PV and the post-pass combine in one launch).
``value`` is algorithmic TFLOP/s = 4 * d * H * (visible query-key pairs) / time, inputs resident in HBM; the
unfused route (``cascade_attn_partials`` + ``cascade_merge``) and the other workloads are reported next to it.
Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "sharded-attn TFLOP/s (prefill)"
HEADLINE = "c2_prefill_8b"
L2_FLUSH_BYTES = 256 << 20

# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel, from the ncu captures summarised
# under profiles/ (None until a capture exists for that workload).
NCU_TRAFFIC_BYTES = {"c2_prefill_8b": 25463552}  # profiles/attn_tc_kernel_c2_headline.md


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples while the timed region runs (read-only query)."""

    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.tmp = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={gpu_index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=self.tmp, stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.tmp.flush()
        self.tmp.seek(0)
        sm, smax, reasons = [], [], set()
        for line in self.tmp.read().splitlines():
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                sm.append(float(parts[1]))
                smax.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"),
                                 parts[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        self.tmp.close()
        os.unlink(self.tmp.name)
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(smax), reasons=sorted(reasons), samples=len(sm))
        return out


def _upload(w, torch, wl):
    ts = []
    for a in (w.q, w.k, w.v):
        if w.dtype == "bf16":
            ts.append(torch.from_numpy(wl.bf16_bits(a).view(np.int16)).cuda().view(torch.bfloat16))
        else:
            ts.append(torch.from_numpy(a).cuda())
    return ts


def _time_steps(torch, fn, steps, warmup, flush, after_warmup=None):
    """Per-step CUDA-event timing on the current stream, L2 flushed between steps.  Returns ms list."""
    for _ in range(warmup):
        flush.fill_(1)
        fn()
    torch.cuda.synchronize()
    if after_warmup is not None:
        after_warmup()
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    for a, b in evs:
        flush.fill_(1)  # evict the previous step's inputs and outputs from the 126 MB L2
        a.record()
        fn()
        b.record()
    torch.cuda.synchronize()
    return [a.elapsed_time(b) for a, b in evs]


def _steps_then_kernel(torch, cb, fn, steps, warmup, flush):
    """Times `steps` steps as a user runs them, then the attention kernel alone in a second pass of the same steps.
    The library brackets the kernel with events on the launch stream while kernel timing is on; the event between
    the gather and the attention launch serialises the two, which otherwise overlap (the attention grid is launched as a
    programmatic dependent of the gather grid), so the step time must not be taken from that pass.
    Returns (ms per step list, kernel ms per launch, kernel launches timed)."""
    ms = _time_steps(torch, fn, steps, warmup, flush)
    _time_steps(torch, fn, steps, 1, flush, after_warmup=cb.cascade_kernel_timing_begin)
    k_ms, k_n = cb.cascade_kernel_timing_end()
    return ms, k_ms / max(k_n, 1), k_n


def run_ours(args):
    import torch
    from paper_2507_05228_b200 import binding as cb
    from paper_2507_05228_b200 import dist as cd
    from paper_2507_05228_b200 import workloads as wl

    rank, world, local = cd.init()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the attention path has no CPU fallback")
    torch.cuda.set_device(local)
    cb.lib()  # fail loudly if the CUDA library is missing
    peaks = _peaks()
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device="cuda")

    # ---- headline workload; with N ranks every rank runs its own sequence (independent problems, no exchange)
    w = wl.config(HEADLINE, seed=1 + rank)
    q, k, v = _upload(w, torch, wl)
    plan = cb.cascade_shard_plan(w.q_shard_of, w.kv_shard_of, w.n_q_shards, w.n_kv_shards, w.q_pos_offset, w.causal)
    o = torch.empty_like(q)
    lse = None
    flops = w.flops()

    ws = torch.empty(cb.cascade_workspace_bytes(plan, cb.CALL_SHARDED, cb.BF16, w.B, w.H, w.Hkv, w.d),
                     dtype=torch.uint8, device="cuda")  # shard-major K/V copies, allocated once

    def step_fused():
        cb.cascade_attn_sharded(plan, q, k, v, w.scale, out=o, want_lse=False, workspace=ws)

    parts = None

    def step_unfused():
        nonlocal parts
        parts = cb.cascade_attn_partials(plan, q, k, v, w.scale, out=parts, workspace=ws)
        cb.cascade_merge(*parts, plan.dev_ptr("q_idx"), out=o, want_lse=False)

    step_unfused()  # allocate the partial buffers once
    torch.cuda.synchronize()

    sampler = ClockSampler(local) if rank == 0 else None
    cd.barrier()
    torch.cuda.synchronize()
    launches0 = cb.cascade_launch_count()
    wall0 = time.perf_counter()
    ms = _time_steps(torch, step_fused, args.steps, args.warmup, flush)
    torch.cuda.synchronize()
    cd.barrier()
    wall = time.perf_counter() - wall0
    launches = (cb.cascade_launch_count() - launches0) * args.steps // (args.steps + args.warmup)
    # the same steps once more with the library's event pairs around every launch of the attention kernel
    _time_steps(torch, step_fused, args.steps, 1, flush, after_warmup=cb.cascade_kernel_timing_begin)
    kernel_ms_total, kernel_launches = cb.cascade_kernel_timing_end()
    clocks = sampler.stop() if sampler else None
    total_ms = cd.max_over_ranks(sum(ms))
    ms_per_step = total_ms / args.steps
    value = world * flops / (ms_per_step * 1e-3) / 1e12

    # ---- end to end through the public call with host buffers: H2D of q, k, v, the fused call, D2H of o
    hq, hk, hv = (t.cpu().pin_memory() for t in (q, k, v))
    ho = torch.empty_like(hq).pin_memory()

    ws_host = torch.empty(cb.cascade_workspace_bytes(plan, cb.CALL_SHARDED_HOST, cb.BF16, w.B, w.H, w.Hkv, w.d),
                          dtype=torch.uint8, device="cuda")

    def step_e2e():
        # the library's host-buffer call: uploads q, k, v from pinned memory, runs the fused route and downloads o,
        # one KV head group after another with the copies in both directions and the compute overlapped
        cb.cascade_attn_sharded_host(plan, hq, hk, hv, w.scale, ho, ws_host)

    e2e_steps = max(3, min(args.steps, 50))
    ms_e2e = _time_steps(torch, step_e2e, e2e_steps, 3, flush)
    e2e_ms = cd.max_over_ranks(sum(ms_e2e)) / e2e_steps
    h2d = sum(t.numel() * t.element_size() for t in (hq, hk, hv))
    d2h = ho.numel() * ho.element_size()

    ms_unfused = _time_steps(torch, step_unfused, max(3, min(args.steps, 50)), 3, flush)
    status = plan.device_status()
    routes = {
        "fused": {"ms": statistics.median(ms), "ms_min": min(ms), "tflops": flops / (statistics.median(ms) * 1e-3) / 1e12},
        "partials_merge": {"ms": statistics.median(ms_unfused), "ms_min": min(ms_unfused),
                           "tflops": flops / (statistics.median(ms_unfused) * 1e-3) / 1e12},
    }
    # Two launches per step: the shard gather of K/V (HBM-bound, a few microseconds) and the attention kernel, which
    # dominates.  Its own duration comes from the event pairs the library recorded around it in a second pass of the
    # same steps, under the same clock sampling: in the timed steps the two launches overlap (programmatic dependent
    # launch), and an event between them would take that overlap away.
    kernel_ms = kernel_ms_total / max(kernel_launches, 1)
    achieved = flops / (kernel_ms * 1e-3) / 1e12
    roofline = {"bound": "tensor", "kernel": "attn_tc_kernel (fused route)", "achieved": achieved,
                "peak": peaks["bf16_tflops"], "peak_source": peaks["source"] + " burst bf16 (cuBLAS)",
                "unit": "TFLOP/s", "frac": achieved / peaks["bf16_tflops"],
                "frac_of_sustained": achieved / peaks["bf16_tflops_sustained"], "frac_of_nominal_2250": achieved / 2250.0,
                "kernel_ms": kernel_ms, "kernel_launches_timed": kernel_launches,
                "timed": "second pass of the same steps, event pair around each attention launch",
                "traffic": NCU_TRAFFIC_BYTES.get(HEADLINE)}
    if rank == 0 and world == 1 and not args.no_extras:
        routes["fused_rope"] = _rope_record(torch, cb, w, plan, q, k, v, o, ws, flush, routes["fused"]["ms"], kernel_ms,
                                            steps=max(args.steps, 20))
    plan.destroy()
    del q, k, v, o, parts

    extras = {}
    if rank == 0 and world == 1 and not args.no_extras:
        extras = run_extras(torch, cb, wl, flush, peaks)

    cpu = None
    if rank == 0 and world == 1:
        cpu = cpu_baseline(wl.config(HEADLINE, seed=1))

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": HEADLINE + ": batch 1 per GPU, 2048 tokens, 32 q / 8 kv heads, head_dim 128, "
                                              "8x8 random token shards, causal", "route": "cascade_attn_sharded (fused)",
                       "l2": "flushed between steps (256 MiB write)", "sequences_per_gpu": 1},
            "clocks": clocks,
            "e2e": {"value": world * flops / (e2e_ms * 1e-3) / 1e12, "unit": "TFLOP/s", "ms_per_step": e2e_ms,
                    "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "call": "cascade_attn_sharded_host (pinned host buffers; copies and compute pipelined over KV heads)"},
            "gpu_launches": int(launches),
            "roofline": roofline,
            "cpu_baseline": cpu,
            "routes": routes,
            "other_workloads": extras,
            "device_status": status,
            "wall_s_timed_region": wall,
        }
        print(json.dumps(line))
    cd.finalize()


ROPE_BASE = 500000.0  # rotary base of the model family the prefill shapes are taken from


def _rope_record(torch, cb, w, plan, q, k, v, o, ws, flush, plain_ms, plain_kernel_ms, steps=5):
    """The fused route with the rotary step of the pre-pass folded into the staging of Q and K rows: what the extra
    arithmetic costs over the same call on rotated inputs (a separate rotary pass would read and write Q and K once)."""
    table = cb.cascade_rope_table(max(w.q_pos_offset + w.n_q, w.n_kv), w.d, ROPE_BASE)
    ms, k_ms, k_n = _steps_then_kernel(torch, cb, lambda: cb.cascade_attn_sharded_rope(
        plan, q, k, v, w.scale, table, out=o, want_lse=False, workspace=ws), steps, 3, flush)
    med = statistics.median(ms)
    qk_bytes = 2 * (w.B * w.n_q * w.H + w.B * w.n_kv * w.Hkv) * w.d * 2  # one read + one write of Q and K
    return {"rope_fused_ms": med, "rope_attn_kernel_ms": k_ms, "rope_extra_ms": med - plain_ms,
            "rope_attn_kernel_extra_ms": k_ms - plain_kernel_ms,
            "separate_rotary_pass_bytes": qk_bytes}


def run_extras(torch, cb, wl, flush, peaks):
    """The other prefill workloads (tensor-bound) and the decode step and merge (HBM-bound), a few steps each."""
    out = {}
    for name in ("c3_batched", "c4_long_70b"):
        w = wl.config(name)
        q, k, v = _upload(w, torch, wl)
        plan = cb.cascade_shard_plan(w.q_shard_of, w.kv_shard_of, w.n_q_shards, w.n_kv_shards, w.q_pos_offset, w.causal)
        o = torch.empty_like(q)
        ws = torch.empty(cb.cascade_workspace_bytes(plan, cb.CALL_SHARDED, cb.BF16, w.B, w.H, w.Hkv, w.d),
                         dtype=torch.uint8, device="cuda")
        ms, k_ms, k_n = _steps_then_kernel(torch, cb, lambda: cb.cascade_attn_sharded(
            plan, q, k, v, w.scale, out=o, want_lse=False, workspace=ws), 5, 3, flush)
        tf = w.flops() / (statistics.median(ms) * 1e-3) / 1e12
        ktf = w.flops() / (k_ms * 1e-3) / 1e12  # attention kernel alone (without the K/V shard gather)
        rec = {"fused_ms": statistics.median(ms), "fused_tflops": tf, "frac_of_burst_peak": tf / peaks["bf16_tflops"],
               "frac_of_sustained_peak": tf / peaks["bf16_tflops_sustained"], "frac_of_nominal_2250": tf / 2250.0,
               "attn_kernel_ms": k_ms, "attn_kernel_tflops": ktf,
               "attn_kernel_frac_of_burst_peak": ktf / peaks["bf16_tflops"]}
        rec.update(_rope_record(torch, cb, w, plan, q, k, v, o, ws, flush, rec["fused_ms"], rec["attn_kernel_ms"]))
        # unfused route: partials (tensor) then merge (HBM)
        parts = cb.cascade_attn_partials(plan, q, k, v, w.scale, workspace=ws)
        ms_p = _time_steps(torch, lambda: cb.cascade_attn_partials(plan, q, k, v, w.scale, out=parts, workspace=ws), 3, 2,
                           flush)
        ms_m = _time_steps(torch, lambda: cb.cascade_merge(*parts, plan.dev_ptr("q_idx"), out=o, want_lse=False), 5, 3,
                           flush)
        rows = w.B * w.n_q * w.H
        merge_bytes = w.n_kv_shards * rows * (w.d * 2 + 8) + rows * w.d * 2
        gbs = merge_bytes / (statistics.median(ms_m) * 1e-3) / 1e9
        rec.update(partials_ms=statistics.median(ms_p),
                   partials_tflops=w.flops() / (statistics.median(ms_p) * 1e-3) / 1e12,
                   merge_ms=statistics.median(ms_m), merge_gbs=gbs, merge_frac_of_hbm=gbs / peaks["hbm_gbs"],
                   merge_frac_of_8tbs=gbs / 8000.0)
        out[name] = rec
        plan.destroy()
        del q, k, v, o, parts, ws
        torch.cuda.empty_cache()
    w = wl.config("c5_decode")
    q, k, v = _upload(w, torch, wl)
    plan = cb.cascade_shard_plan(w.q_shard_of, w.kv_shard_of, w.n_q_shards, w.n_kv_shards, w.q_pos_offset, w.causal)
    parts = cb.cascade_attn_partials(plan, q, k, v, w.scale)
    ms_d = _time_steps(torch, lambda: cb.cascade_attn_partials(plan, q, k, v, w.scale, out=parts), 20, 3, flush)
    o = torch.empty_like(q)
    nbytes = cb.cascade_workspace_bytes(plan, cb.CALL_SHARDED, cb.BF16, w.B, w.H, w.Hkv, w.d)
    ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    ms_f = _time_steps(torch, lambda: cb.cascade_attn_sharded(plan, q, k, v, w.scale, out=o, want_lse=False,
                                                             workspace=ws), 20, 3, flush)
    # a decode-loop step as a serving loop runs it: advance the plan to the new token's position, then decode + merge
    pos = [w.n_kv - 1]

    def step_loop():
        plan.advance(pos[0])
        cb.cascade_attn_sharded(plan, q, k, v, w.scale, out=o, want_lse=False, workspace=ws)

    ms_l = _time_steps(torch, step_loop, 20, 3, flush)
    gbs = w.kv_bytes() / (statistics.median(ms_d) * 1e-3) / 1e9
    out["c5_decode"] = {"decode_step_with_plan_advance_ms": statistics.median(ms_l),
                        "partials_ms": statistics.median(ms_d), "kv_gbs": gbs, "frac_of_hbm": gbs / peaks["hbm_gbs"],
                        "frac_of_8tbs": gbs / 8000.0, "decode_plus_merge_ms": statistics.median(ms_f),
                        "decode_plus_merge_kv_gbs": w.kv_bytes() / (statistics.median(ms_f) * 1e-3) / 1e9}
    plan.destroy()
    del q, k, v, o, parts, ws
    # The shape of the paper's own latency tables: one BERT-Base layer's attention, 128-token prompt, bidirectional
    # mask, fp32, (c, delta) = (8, 16) sharding over alpha = 2 nodes (launch-latency-bound at this size).
    r_of, alpha = cb.cascade_cdelta_shard_map(128, 8, 16)
    w = wl.make_workload("bert_base_n128", 1, 128, 128, 12, 12, 64, "f32", "round_robin", "round_robin", alpha, alpha,
                         seed=5, causal=False)
    q, k, v = _upload(w, torch, wl)
    plan = cb.cascade_shard_plan(r_of, r_of, alpha, alpha, 0, False)
    o = torch.empty_like(q)
    ms_b = _time_steps(torch, lambda: cb.cascade_attn_sharded(plan, q, k, v, w.scale, out=o, want_lse=False), 20, 3,
                       flush)
    parts = cb.cascade_attn_partials(plan, q, k, v, w.scale)
    ms_bp = _time_steps(torch, lambda: (cb.cascade_attn_partials(plan, q, k, v, w.scale, out=parts),
                                        cb.cascade_merge(*parts, plan.dev_ptr("q_idx"), out=o, want_lse=False)), 20, 3,
                        flush)
    out["bert_base_n128_noncausal_f32"] = {"fused_ms": statistics.median(ms_b),
                                           "partials_plus_merge_ms": statistics.median(ms_bp),
                                           "sharding": "(c, delta) = (8, 16), alpha = 2"}
    plan.destroy()
    return out


def cpu_baseline(w, budget_s: float = 20.0):
    """The fp64 oracle as it stands, timed on this machine's host cores on a bounded sample of the workload."""
    import oracle
    cores = oracle.num_threads()
    probe = np.arange(w.n_q - 32, w.n_q, dtype=np.int32)  # 32 of the most expensive rows
    t0 = time.perf_counter()
    oracle.attention_unsharded(w.q, w.k, w.v, w.scale, causal=w.causal, q_pos_offset=w.q_pos_offset, rows=probe)
    t_probe = time.perf_counter() - t0
    pairs_probe = float(np.clip(probe + w.q_pos_offset + 1, 0, w.n_kv).sum())
    rate = pairs_probe / max(t_probe, 1e-6)  # visible pairs per second (all heads)
    total_pairs = w.visible_pairs() / w.B
    if total_pairs / rate <= budget_s:
        rows = np.arange(w.n_q, dtype=np.int32)
        sample = f"all {w.n_q} query rows of {w.name}, all heads"
    else:
        n = max(8, int(w.n_q * budget_s * rate / total_pairs))
        rows = np.unique(np.linspace(0, w.n_q - 1, n).astype(np.int32))
        sample = f"{rows.size} evenly spaced query rows of {w.name}, all heads"
    t0 = time.perf_counter()
    oracle.attention_unsharded(w.q, w.k, w.v, w.scale, causal=w.causal, q_pos_offset=w.q_pos_offset, rows=rows)
    dt = time.perf_counter() - t0
    pairs = float(np.clip(rows.astype(np.int64) + w.q_pos_offset + 1, 0, w.n_kv).sum()) * w.B
    fl = 4.0 * w.d * w.H * pairs
    return {"value": fl / dt / 1e12, "unit": "TFLOP/s", "cores": cores, "kind": "oracle", "sample": sample,
            "seconds": dt}


def run_reference(args):
    """Reference arm: the CPU oracle on the headline workload.  Each step evaluates a bounded sample of query rows
    sized so that the whole run ends within a few minutes."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    from paper_2507_05228_b200 import workloads as wl
    w = wl.config(HEADLINE, seed=1)
    cores = oracle.num_threads()
    probe = np.arange(w.n_q - 16, w.n_q, dtype=np.int32)
    t0 = time.perf_counter()
    oracle.attention_unsharded(w.q, w.k, w.v, w.scale, rows=probe)
    rate = float((probe + 1).sum()) / max(time.perf_counter() - t0, 1e-6)
    budget = 120.0 / max(1, args.steps + args.warmup)
    pairs_per_row = (w.n_q + 1) / 2.0
    n_rows = int(max(4, min(w.n_q, budget * rate / pairs_per_row)))
    rows = np.unique(np.linspace(0, w.n_q - 1, n_rows).astype(np.int32))
    pairs = float((rows.astype(np.int64) + 1).sum())
    fl = 4.0 * w.d * w.H * pairs
    for _ in range(args.warmup):
        oracle.attention_unsharded(w.q, w.k, w.v, w.scale, rows=rows)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle.attention_unsharded(w.q, w.k, w.v, w.scale, rows=rows)
    dt = (time.perf_counter() - t0) / args.steps
    value = fl / dt / 1e12
    sample = f"{rows.size} evenly spaced query rows of {w.name} per step, all heads"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": HEADLINE + " (fp64 CPU oracle, unsharded definition)", "sample": sample},
        "cpu_baseline": {"value": value, "unit": "TFLOP/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-extras", action="store_true", help="skip the other workloads (c3, c4, c5)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
