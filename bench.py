#!/usr/bin/env python
"""Benchmark of the sequence-sharded attention hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--no-extras]

One step = one pass of the hot path over one batch of the headline workload, the largest single-GPU prefill
configuration (the 70B-shaped long-context layer: 32768 tokens, 64 query / 8 KV heads, head_dim 128, bf16, 32 x 32
random token shards): the fused call ``cascade_attn_sharded`` (shard gather, QK^T, mask, streaming statistics, PV and
the post-pass combine).  ``value`` is algorithmic TFLOP/s = 4 * d * H * (visible query-key pairs) / time with the
inputs resident in HBM; the unfused route (``cascade_attn_partials`` + ``cascade_merge``), the other prefill
configurations, the decode step and the merge are reported next to it, each with its own roofline record.
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
HEADLINE = "c4_long_70b"
HEADLINE_TEXT = ("c4_long_70b: batch 1 per GPU, 32768 tokens, 64 q / 8 kv heads, head_dim 128, bf16, 32x32 random token "
                 "shards, causal")
L2_FLUSH_BYTES = 256 << 20
MIN_STEPS = 20  # timed launches behind every record

# dram__bytes_read.sum + dram__bytes_write.sum per launch of each record's dominant kernel, from one ncu capture per
# kernel and workload ((bytes of the captured case, launches of the captured size that make one full-size launch); None =
# no capture of the kernel as it stands).  The prefill kernel's traffic grows with batch * KV heads (each (sequence, KV
# head) streams its own K/V and writes its own output rows), the decode and merge kernels' with the batch.
NCU_TRAFFIC = {
    "c2_prefill_8b/attn_tc_kernel": (25478656, 1),
    "c3_batched/attn_tc_kernel": (136032256, 4),        # captured on one of the four sequences
    "c4_long_70b/attn_tc_kernel": (1212214016, 1),
    "c3_batched/attn_tc_kernel/partials": (1257771264, 4),
    "c4_long_70b/attn_tc_kernel/partials": (4671739904, 4),  # captured with a quarter of the heads
    "c5_decode/decode_kernel": (545430528, 8),          # captured with batch 8 of 64
    "c3_batched/merge_kernel": (1135894528, 4),
}


def _traffic(key):
    rec = NCU_TRAFFIC.get(key)
    return None if rec is None else rec[0] * rec[1]


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
        sm, smax, power, reasons = [], [], [], set()
        for line in self.tmp.read().splitlines():
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                sm.append(float(parts[1]))
                smax.append(float(parts[2]))
                power.append(float(parts[3]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"),
                                 parts[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        self.tmp.close()
        os.unlink(self.tmp.name)
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(smax), reasons=sorted(reasons), samples=len(sm),
                       sm_mhz_min=min(sm), power_w_max=max(power))
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


def _tensor_roofline(peaks, kernel, flops, kernel_ms, steps, traffic, power_capped=False):
    """The dense bf16 peak a launch is held against: the burst figure (a GEMM timed alone) unless the clock samples
    taken during the timed region show the board's power cap active, i.e. the kernel ran inside a long step at the
    clocks a seconds-long GEMM loop gets too; then the sustained figure.  Both fractions are always reported."""
    achieved = flops / (kernel_ms * 1e-3) / 1e12
    burst, sustained = peaks["bf16_tflops"], peaks["bf16_tflops_sustained"]
    peak = sustained if power_capped else burst
    which = ("sustained bf16 (cuBLAS back to back for seconds; sw_power_cap was active in the timed region)"
             if power_capped else "burst bf16 (cuBLAS, timed alone)")
    return {"bound": "tensor", "kernel": kernel, "achieved": achieved, "peak": peak,
            "peak_source": peaks["source"] + " " + which, "unit": "TFLOP/s", "frac": achieved / peak,
            "frac_of_burst": achieved / burst, "frac_of_sustained": achieved / sustained,
            "frac_of_nominal_2250": achieved / 2250.0, "kernel_ms": kernel_ms, "steps": steps, "traffic": traffic}


def _hbm_roofline(peaks, kernel, nbytes, kernel_ms, steps, traffic):
    achieved = nbytes / (kernel_ms * 1e-3) / 1e9
    return {"bound": "hbm", "kernel": kernel, "achieved": achieved, "peak": peaks["hbm_gbs"],
            "peak_source": peaks["source"] + " copy bandwidth", "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"],
            "frac_of_8tbs": achieved / 8000.0, "kernel_ms": kernel_ms, "steps": steps, "traffic": traffic,
            "algorithmic_bytes": nbytes}


def plan_statistics(plan, w):
    """Host-side counts from the plan: how much tensor work the tiling executes per unit of causal work, and the
    EMPTY / PARTIAL / FULL classes of the (query shard, KV shard) pairs (what pair-class skipping can use)."""
    vis = plan.get("vis")[0].astype(np.int64)  # [n_q, P]
    q_off = plan.get("q_off")[0]
    G = w.H // w.Hkv
    gp = 1
    while gp < 8 and G % (2 * gp) == 0:
        gp *= 2
    rows_per_cta = 2 * (128 // gp)  # two sub-tiles of 128 MMA rows, gp heads stacked per slot
    executed = 0
    for j in range(w.n_q_shards):
        for r0 in range(q_off[j], q_off[j + 1], rows_per_cta):
            n = min(rows_per_cta, q_off[j + 1] - r0)
            need = vis[r0 + n - 1]  # the tile's last row has the longest prefix of every shard
            keys = int((-(-need // 32) * 32).sum())  # every shard's prefix rounded up to 32-key chunks
            n_sub = 2 if n > rows_per_cta // 2 else 1
            executed += keys * n_sub * (128 // gp)  # MMA rows are (slot, head) pairs: 128 / gp slots per sub-tile
    causal = int(vis.sum())
    pc = plan.get("pair_class")[0]
    return {"mma_pairs_executed_over_causal": executed / max(causal, 1),
            "pair_classes": {"empty": int((pc == 0).sum()), "partial": int((pc == 1).sum()), "full": int((pc == 2).sum())}}


ROPE_BASE = 500000.0  # rotary base of the model family the prefill shapes are taken from


def measure_prefill(torch, cb, wl, name, flush, peaks, steps, warmup, seed=None, with_rope=True):
    """Every route of one prefill workload.  Returns (record, context) where context keeps the device tensors alive
    for callers that go on with the same workload."""
    w = wl.config(name) if seed is None else wl.config(name, seed=seed)
    q, k, v = _upload(w, torch, wl)
    plan = cb.cascade_shard_plan(w.q_shard_of, w.kv_shard_of, w.n_q_shards, w.n_kv_shards, w.q_pos_offset, w.causal)
    o = torch.empty_like(q)
    ws = torch.empty(cb.cascade_workspace_bytes(plan, cb.CALL_SHARDED, cb.BF16, w.B, w.H, w.Hkv, w.d),
                     dtype=torch.uint8, device="cuda")  # shard-major K/V copies, allocated once
    flops = w.flops()

    def step_fused():
        cb.cascade_attn_sharded(plan, q, k, v, w.scale, out=o, want_lse=False, workspace=ws)

    launches0 = cb.cascade_launch_count()
    ms, k_ms, k_n = _steps_then_kernel(torch, cb, step_fused, steps, warmup, flush)
    launches_per_step = (cb.cascade_launch_count() - launches0) // (2 * steps + warmup + 1)
    med = statistics.median(ms)
    rec = {"fused": {"ms": med, "ms_min": min(ms), "tflops": flops / (med * 1e-3) / 1e12, "steps": steps,
                     "launches_per_step": int(launches_per_step),
                     "roofline": _tensor_roofline(peaks, "attn_tc_kernel (fused route)", flops, k_ms, k_n,
                                                  _traffic(name + "/attn_tc_kernel"))}}
    if with_rope:
        table = cb.cascade_rope_table(max(w.q_pos_offset + w.n_q, w.n_kv), w.d, ROPE_BASE)
        ms_r, k_ms_r, _ = _steps_then_kernel(torch, cb, lambda: cb.cascade_attn_sharded_rope(
            plan, q, k, v, w.scale, table, out=o, want_lse=False, workspace=ws), MIN_STEPS, 3, flush)
        med_r = statistics.median(ms_r)
        rec["fused_rope"] = {"ms": med_r, "attn_kernel_ms": k_ms_r, "extra_ms": med_r - med, "steps": MIN_STEPS,
                             "separate_rotary_pass_bytes":
                                 2 * (w.B * w.n_q * w.H + w.B * w.n_kv * w.Hkv) * w.d * 2}
        del table
    # unfused route: the attention-pass of every pair (tensor-bound, plus the partial writes), then the post-pass (HBM)
    parts = cb.cascade_attn_partials(plan, q, k, v, w.scale, workspace=ws)
    ms_p, kp_ms, kp_n = _steps_then_kernel(torch, cb, lambda: cb.cascade_attn_partials(
        plan, q, k, v, w.scale, out=parts, workspace=ws), MIN_STEPS, 2, flush)
    ms_m = _time_steps(torch, lambda: cb.cascade_merge(*parts, plan.dev_ptr("q_idx"), out=o, want_lse=False), MIN_STEPS,
                       3, flush)
    rows = w.B * w.n_q * w.H
    part_bytes = w.n_kv_shards * rows * (w.d * 2 + 8)
    merge_bytes = part_bytes + rows * w.d * 2
    med_p, med_m = statistics.median(ms_p), statistics.median(ms_m)
    rec["partials"] = {"ms": med_p, "tflops": flops / (med_p * 1e-3) / 1e12, "steps": MIN_STEPS,
                       "partial_write_gbs": part_bytes / (kp_ms * 1e-3) / 1e9,
                       "roofline": _tensor_roofline(peaks, "attn_tc_kernel (one CTA per query tile walks all KV shards)",
                                                    flops, kp_ms, kp_n, _traffic(name + "/attn_tc_kernel/partials"))}
    rec["merge"] = {"ms": med_m, "steps": MIN_STEPS,
                    "roofline": _hbm_roofline(peaks, "merge_kernel", merge_bytes, med_m, MIN_STEPS,
                                              _traffic(name + "/merge_kernel"))}
    rec["partials_plus_merge_ms"] = med_p + med_m
    rec["plan"] = plan_statistics(plan, w)
    rec["device_status"] = plan.device_status()
    del parts
    return rec, (w, plan, q, k, v, o, ws, ms)


def measure_decode(torch, cb, wl, flush, peaks):
    w = wl.config("c5_decode")
    q, k, v = _upload(w, torch, wl)
    plan = cb.cascade_shard_plan(w.q_shard_of, w.kv_shard_of, w.n_q_shards, w.n_kv_shards, w.q_pos_offset, w.causal)
    parts = cb.cascade_attn_partials(plan, q, k, v, w.scale)
    steps = 2 * MIN_STEPS
    ms_d, k_ms, k_n = _steps_then_kernel(torch, cb, lambda: cb.cascade_attn_partials(plan, q, k, v, w.scale, out=parts),
                                         steps, 3, flush)
    o = torch.empty_like(q)
    ws = torch.empty(cb.cascade_workspace_bytes(plan, cb.CALL_SHARDED, cb.BF16, w.B, w.H, w.Hkv, w.d),
                     dtype=torch.uint8, device="cuda")
    ms_f = _time_steps(torch, lambda: cb.cascade_attn_sharded(plan, q, k, v, w.scale, out=o, want_lse=False,
                                                             workspace=ws), steps, 3, flush)
    # a decode-loop step as a serving loop runs it: advance the plan to the new token's position, then decode + merge
    pos = [w.n_kv - 1]

    def step_loop():
        plan.advance(pos[0])
        cb.cascade_attn_sharded(plan, q, k, v, w.scale, out=o, want_lse=False, workspace=ws)

    ms_l = _time_steps(torch, step_loop, steps, 3, flush)
    rows = w.B * w.n_kv_shards * w.H
    merge_bytes = rows * (w.d * 2 + 8) + w.B * w.H * w.d * 2
    med_f = statistics.median(ms_f)
    rec = {"partials_ms": statistics.median(ms_d), "decode_plus_merge_ms": med_f,
           "decode_plus_merge_kv_gbs": w.kv_bytes() / (med_f * 1e-3) / 1e9,
           "decode_step_with_plan_advance_ms": statistics.median(ms_l), "steps": steps,
           "merge_bytes": merge_bytes, "device_status": plan.device_status(),
           "roofline": _hbm_roofline(peaks, "decode_kernel<4>", w.kv_bytes(), k_ms, k_n,
                                     _traffic("c5_decode/decode_kernel"))}
    plan.destroy()
    return rec


def measure_small_cases(torch, cb, wl, flush):
    """The shape of the paper's own latency tables, and the host cost of moving a prefill chunk along a cache."""
    out = {}
    # one BERT-Base layer's attention, 128-token prompt, bidirectional mask, fp32, (c, delta) = (8, 16) sharding over
    # alpha = 2 nodes (launch-latency-bound at this size)
    r_of, alpha = cb.cascade_cdelta_shard_map(128, 8, 16)
    w = wl.make_workload("bert_base_n128", 1, 128, 128, 12, 12, 64, "f32", "round_robin", "round_robin", alpha, alpha,
                         seed=5, causal=False)
    q, k, v = _upload(w, torch, wl)
    plan = cb.cascade_shard_plan(r_of, r_of, alpha, alpha, 0, False)
    o = torch.empty_like(q)
    ms_b = _time_steps(torch, lambda: cb.cascade_attn_sharded(plan, q, k, v, w.scale, out=o, want_lse=False),
                       MIN_STEPS, 3, flush)
    parts = cb.cascade_attn_partials(plan, q, k, v, w.scale)
    ms_bp = _time_steps(torch, lambda: (cb.cascade_attn_partials(plan, q, k, v, w.scale, out=parts),
                                        cb.cascade_merge(*parts, plan.dev_ptr("q_idx"), out=o, want_lse=False)),
                        MIN_STEPS, 3, flush)
    out["bert_base_n128_noncausal_f32"] = {"fused_ms": statistics.median(ms_b),
                                           "partials_plus_merge_ms": statistics.median(ms_bp), "steps": MIN_STEPS,
                                           "sharding": "(c, delta) = (8, 16), alpha = 2"}
    plan.destroy()
    # chunked prefill over a preallocated cache: a 512-row query block moved along 8192 cache rows, 16 KV shards
    w = wl.config("c3_batched", B=1, n_q=512, H=8, Hkv=2, outlier_frac=0.0, q_pos_offset=0)
    plan = cb.cascade_shard_plan(w.q_shard_of, w.kv_shard_of, w.n_q_shards, w.n_kv_shards, 0, True)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    n_adv = 0
    for off in range(0, w.n_kv - w.n_q + 1, w.n_q):
        plan.advance(off)
        n_adv += 1
    torch.cuda.synchronize()
    # wall clock per call with the device drained at the end: two small kernels per advance, nothing on the host
    out["plan_advance_sliding_chunk"] = {"ms_per_advance": (time.perf_counter() - t0) * 1e3 / n_adv,
                                         "chunk_rows": w.n_q, "cache_rows": w.n_kv, "kv_shards": w.n_kv_shards}
    plan.destroy()
    return out


def measure_exchange(torch, cb, cd, wl, flush, rank, world):
    """The multi-rank form of the path: resident K/V per rank, partials, stage-B all-to-all, local post-pass, on one
    sequence of the 8B-shaped prefill shape.  With one rank the all-to-all is a local copy (no wire)."""
    from paper_2507_05228_b200 import exchange as ex
    w = wl.config("c2_prefill_8b", n_q=8192, n_kv=8192, n_q_shards=16, n_kv_shards=16, seed=11)  # same on every rank
    q, k, v = _upload(w, torch, wl)
    ra = ex.RankAttention(w.q_shard_of, w.kv_shard_of, w.n_q_shards, w.n_kv_shards, rank, world)
    tok = torch.from_numpy(ra.tokens.astype(np.int64)).cuda()
    k_res, v_res = k[:, tok].contiguous(), v[:, tok].contiguous()
    del k, v
    sent = [0]

    def step():
        _, _, sent[0] = ra.run(q, k_res, v_res, w.scale)

    ms = _time_steps(torch, step, MIN_STEPS, 3, flush)
    total_ms = cd.max_over_ranks(sum(ms)) / MIN_STEPS
    direct_ms = None
    if world == 1:
        # the one-kernel form of stage B + post-pass (cascade_merge_peers reads the parts where they were written);
        # with several ranks the sources would be the peers' buffers mapped into this process, which is not wired here
        def step_direct():
            ra.combine_in_place([ra.partials(q, k_res, v_res, w.scale)], want_lse=True)

        direct_ms = statistics.median(_time_steps(torch, step_direct, MIN_STEPS, 3, flush))
    wire = cd.sum_over_ranks(float(sent[0]))
    rec = {"workload": "one 8B-shaped sequence of 8192 tokens, 16 x 16 random shards, KV shards dealt round-robin to "
                       "the ranks", "world": world, "ms_per_layer": total_ms, "steps": MIN_STEPS,
           "tflops": w.flops() / (total_ms * 1e-3) / 1e12, "stage_b_bytes_sent": wire,
           "stage_b_bytes_closed_form": ex.stage_b_bytes(w.B, w.n_kv_shards, w.n_q, w.H, w.d, 2),
           "wire": "nccl all_to_all_single" if world > 1 else "none (one rank: local copy)",
           "ms_per_layer_parts_read_in_place": direct_ms,
           "device_status": ra.plan.device_status()}
    ra.destroy()
    return rec


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
    w = wl.config(HEADLINE, seed=3 + rank)
    q, k, v = _upload(w, torch, wl)
    plan = cb.cascade_shard_plan(w.q_shard_of, w.kv_shard_of, w.n_q_shards, w.n_kv_shards, w.q_pos_offset, w.causal)
    o = torch.empty_like(q)
    flops = w.flops()
    ws = torch.empty(cb.cascade_workspace_bytes(plan, cb.CALL_SHARDED, cb.BF16, w.B, w.H, w.Hkv, w.d),
                     dtype=torch.uint8, device="cuda")

    def step_fused():
        cb.cascade_attn_sharded(plan, q, k, v, w.scale, out=o, want_lse=False, workspace=ws)

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
    # Two launches per step: the shard gather of K/V (HBM-bound, tens of microseconds) and the attention kernel, which
    # dominates.  Its own duration comes from the event pairs the library records around it in a second pass of the
    # same steps, under the same clock sampling: in the timed steps the two launches overlap (programmatic dependent
    # launch), and an event between them would take that overlap away.
    _time_steps(torch, step_fused, args.steps, 1, flush, after_warmup=cb.cascade_kernel_timing_begin)
    kernel_ms_total, kernel_launches = cb.cascade_kernel_timing_end()
    clocks = sampler.stop() if sampler else None
    total_ms = cd.max_over_ranks(sum(ms))
    ms_per_step = total_ms / args.steps
    value = world * flops / (ms_per_step * 1e-3) / 1e12
    kernel_ms = kernel_ms_total / max(kernel_launches, 1)
    capped = bool(clocks) and any("power_cap" in r for r in (clocks.get("reasons") or []))
    roofline = _tensor_roofline(peaks, "attn_tc_kernel (fused route)", flops, kernel_ms, kernel_launches,
                                _traffic(HEADLINE + "/attn_tc_kernel"), power_capped=capped)
    roofline["timed"] = "second pass of the same steps, event pair around each attention launch"
    status = plan.device_status()

    # ---- end to end through the public call with host buffers: H2D of q, k, v, the fused call, D2H of o
    hq, hk, hv = (t.cpu().pin_memory() for t in (q, k, v))
    ho = torch.empty_like(hq).pin_memory()
    ws_host = torch.empty(cb.cascade_workspace_bytes(plan, cb.CALL_SHARDED_HOST, cb.BF16, w.B, w.H, w.Hkv, w.d),
                          dtype=torch.uint8, device="cuda")

    def step_e2e():
        # the library's host-buffer call: uploads q, k, v from pinned memory, runs the fused route and downloads o,
        # one KV head group after another with the copies in both directions and the compute overlapped
        cb.cascade_attn_sharded_host(plan, hq, hk, hv, w.scale, ho, ws_host)

    e2e_steps = max(3, min(args.steps, MIN_STEPS))
    ms_e2e = _time_steps(torch, step_e2e, e2e_steps, 3, flush)
    e2e_ms = cd.max_over_ranks(sum(ms_e2e)) / e2e_steps
    h2d = sum(t.numel() * t.element_size() for t in (hq, hk, hv))
    d2h = ho.numel() * ho.element_size()
    del hq, hk, hv, ho, ws_host
    plan_stats = plan_statistics(plan, w)
    plan.destroy()
    del q, k, v, o, ws
    torch.cuda.empty_cache()

    exchange = None
    if not args.no_extras:
        exchange = measure_exchange(torch, cb, cd, wl, flush, rank, world)

    workloads = {}
    if rank == 0 and world == 1 and not args.no_extras:
        for name, steps in (("c4_long_70b", MIN_STEPS), ("c3_batched", 2 * MIN_STEPS), ("c2_prefill_8b", 10 * MIN_STEPS)):
            rec, ctx = measure_prefill(torch, cb, wl, name, flush, peaks, steps, 3)
            ctx[1].destroy()
            del ctx
            torch.cuda.empty_cache()
            workloads[name] = rec
        workloads["c5_decode"] = measure_decode(torch, cb, wl, flush, peaks)
        workloads.update(measure_small_cases(torch, cb, wl, flush))

    cpu = None
    if rank == 0 and world == 1:
        cpu = cpu_baseline(w)  # rank 0's own sequence: the arrays the GPU steps ran on

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": HEADLINE_TEXT, "route": "cascade_attn_sharded (fused)",
                       "l2": "flushed between steps (256 MiB write); inputs are 1.2 GB", "sequences_per_gpu": 1,
                       "plan": plan_stats},
            "clocks": clocks,
            "e2e": {"value": world * flops / (e2e_ms * 1e-3) / 1e12, "unit": "TFLOP/s", "ms_per_step": e2e_ms,
                    "steps": e2e_steps, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "call": "cascade_attn_sharded_host (pinned host buffers; copies and compute pipelined over KV heads)"},
            "gpu_launches": int(launches),
            "roofline": roofline,
            "cpu_baseline": cpu,
            "ms_median": statistics.median(ms), "ms_min": min(ms),
            "exchange": exchange,
            "other_workloads": workloads,
            "device_status": status,
            "wall_s_timed_region": wall,
        }
        print(json.dumps(line))
    cd.finalize()


def _oracle_rows(w, n_rows):
    """Evenly spaced query rows (token ids) of the workload, the last row included."""
    return np.unique(np.linspace(0, w.n_q - 1, max(2, n_rows)).astype(np.int32))


def _pairs(w, rows):
    return float(np.clip(rows.astype(np.int64) + w.q_pos_offset + 1, 0, w.n_kv).sum()) * w.B


def cpu_baseline(w, budget_s: float = 20.0):
    """The fp64 oracle as it stands, timed on this machine's host cores on a bounded sample of the workload: evenly
    spaced query rows (all heads), as many as the budget allows.  `value` is the rate on that sample; the time the
    whole workload would take at that rate is given as an extrapolation."""
    import oracle
    cores = oracle.num_threads()
    probe = np.arange(w.n_q - 16, w.n_q, dtype=np.int32)  # 16 of the most expensive rows
    t0 = time.perf_counter()
    oracle.attention_unsharded(w.q, w.k, w.v, w.scale, causal=w.causal, q_pos_offset=w.q_pos_offset, rows=probe)
    rate = _pairs(w, probe) / max(time.perf_counter() - t0, 1e-6)  # visible pairs per second (all heads)
    total_pairs = float(w.visible_pairs())
    n = int(min(w.n_q, max(8, w.n_q * budget_s * rate / total_pairs)))
    rows = _oracle_rows(w, n)
    t0 = time.perf_counter()
    oracle.attention_unsharded(w.q, w.k, w.v, w.scale, causal=w.causal, q_pos_offset=w.q_pos_offset, rows=rows)
    dt = time.perf_counter() - t0
    pairs = _pairs(w, rows)
    fl = 4.0 * w.d * w.H * pairs
    sample = (f"all {w.n_q} query rows" if rows.size == w.n_q else f"{rows.size} evenly spaced query rows") + \
             f" of {w.name}, all heads"
    return {"value": fl / dt / 1e12, "unit": "TFLOP/s", "cores": cores, "kind": "oracle", "sample": sample,
            "seconds": dt, "whole_workload_seconds_extrapolated": dt * total_pairs / pairs}


def run_reference(args):
    """Reference arm: the CPU oracle on the headline workload.  Each step evaluates a bounded sample of query rows
    sized so that the whole run ends within a few minutes."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    from paper_2507_05228_b200 import workloads as wl
    w = wl.config(HEADLINE, seed=3)
    cores = oracle.num_threads()
    probe = np.arange(w.n_q - 16, w.n_q, dtype=np.int32)
    t0 = time.perf_counter()
    oracle.attention_unsharded(w.q, w.k, w.v, w.scale, rows=probe)
    rate = _pairs(w, probe) / max(time.perf_counter() - t0, 1e-6)
    budget = 100.0 / max(1, args.steps + args.warmup)
    n_rows = int(max(4, min(w.n_q, w.n_q * budget * rate / float(w.visible_pairs()))))
    rows = _oracle_rows(w, n_rows)
    fl = 4.0 * w.d * w.H * _pairs(w, rows)
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
        "config": {"workload": HEADLINE_TEXT, "arm": "fp64 CPU oracle, unsharded definition", "sample": sample},
        "cpu_baseline": {"value": value, "unit": "TFLOP/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=60)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-extras", action="store_true", help="skip the other workloads and routes")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
