#!/usr/bin/env python
"""Benchmark of the KVReviver hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

One "step" is one pass of the whole hot path over one batch of seeded synthetic input: compress
every layer of the workload (score, select, gather, sketch insert), then run all of the
workload's decode steps (reconstruct + attention over retained and reconstructed tokens, one
kernel launch per layer per decode step, replayed through a CUDA graph).  The metric is decode
tokens per second of the whole job.  Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2512_17917_b200 import dist as kdist  # noqa: E402
from paper_2512_17917_b200 import synth  # noqa: E402

METRIC = "decode_attention_tokens_per_s"
UNIT = "tokens/s"
DEFAULT_WORKLOAD = "32k_llama3_8b"
FALLBACK_HBM_GBS = 6650.0


# ------------------------------------------------------------------------------------------ util
def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """nvidia-smi clocks / throttle reasons sampled every 200 ms while the timed region runs."""

    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_id: str):
        self.gpu = gpu_id
        self.proc = None
        self.path = None

    def start(self):
        try:
            f = tempfile.NamedTemporaryFile("w", suffix=".csv", delete=False)
            self.path = f.name
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "200", "-i", str(self.gpu)], stdout=f, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        time.sleep(0.25)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        try:
            for line in open(self.path):
                c = [x.strip() for x in line.split(",")]
                if len(c) < 9:
                    continue
                try:
                    sm.append(float(c[1]))
                    mx.append(float(c[2]))
                except ValueError:
                    continue
                for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), c[5:9]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))
        return out


def config_of(w) -> dict:
    """The workload as both arms print it (same keys, so that the two lines can be matched)."""
    return {"workload": w.name, "batch": w.batch, "layers": w.n_layers, "kv_heads": w.n_kv_heads,
            "q_heads": w.n_q_heads, "head_dim": w.head_dim, "context": w.context, "budget": w.budget,
            "sketch_rows": 3, "sketch_width": w.b, "obs_window": w.obs_window,
            "decode_steps_per_step": w.decode_steps, "kv_dtype": w.dtype, "launch": "per_layer_cuda_graph",
            "l2": "inputs larger than L2 (each decode step streams %.2f GB)"
                  % (decode_bytes_per_launch(w, w.n_layers * w.batch * w.n_kv_heads) / 1e9)}


def host_cores() -> int:
    """Cores this process may run on (the oracle's OpenMP team is sized from the same mask)."""
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


def decode_bytes_per_launch(w, n_inst_launch: int, entry_bytes: int = 8) -> int:
    """Algorithmic HBM bytes of one decode-attention launch over n_inst head-instances: retained
    K and V rows, the fp32 sketch (keys + values) once, the list of compressed tokens (8-byte
    entries for the staged kernel, 4-byte for the split kernel), the queries and the fp32 output."""
    R, N, b, D = w.budget, w.context, w.b, w.head_dim
    G = w.n_q_heads // w.n_kv_heads
    per = R * D * 2 * 2 + 3 * b * 2 * D * 4 + (N - R) * entry_bytes + (b + 1) * 4 + G * D * 2 + G * D * 4
    return per * n_inst_launch


def compress_bytes_per_layer(w, n_inst_layer: int) -> int:
    """Algorithmic HBM bytes of compressing one layer: K and V read once (scoring, copies and
    insertion share them through L2), the retained copies written, the fp32 sketch written."""
    R, N, b, D = w.budget, w.context, w.b, w.head_dim
    return (N * D * 2 * 2 + R * D * 2 * 2 + 3 * b * 2 * D * 4) * n_inst_layer


def smem_cell_bytes_per_launch(w, n_inst_launch: int) -> int:
    """Shared-memory bytes of cell data one staged launch reads: every reconstructed token takes two
    of its three cells (keys and values, fp32) from shared memory; the third sits in registers."""
    return (w.context - w.budget) * 2 * 2 * w.head_dim * 4 * n_inst_launch


def minmax_ops_per_launch(w, n_inst_launch: int) -> int:
    """fp32 min/max lane-operations one launch cannot avoid: the element-wise median of three
    (4 two-input min/max) for the D key and D value channels of every reconstructed token."""
    return (w.context - w.budget) * 2 * w.head_dim * 4 * n_inst_launch


# ------------------------------------------------------------------------------- the GPU arm
def run_gpu(args, w, rank, world, local):
    import paper_2512_17917_b200 as kvr

    dev = torch.device(f"cuda:{local}")
    torch.cuda.set_device(dev)
    L, B, H, Hq, D, N, R, W, S = (w.n_layers, w.batch, w.n_kv_heads, w.n_q_heads, w.head_dim, w.context,
                                  w.budget, w.obs_window, w.decode_steps)
    dt = w.torch_dtype
    seed_shift = 1_000_003 * rank          # every rank draws its own batch (weak scaling)
    seeds = synth.hash_seeds(w.seed + 3)
    sk = kvr.kvr_sketch_create(b=w.b, batch=B, n_layers=L, n_kv_heads=H, n_q_heads=Hq, max_context=N,
                               kv_dtype=dt, hash_seeds=seeds, device=dev)
    kvr.kvr_sketch_set_decode_kernel(sk, {"auto": kvr.KVR_DECODE_AUTO, "split": kvr.KVR_DECODE_SPLIT,
                                          "staged": kvr.KVR_DECODE_STAGED}[args.decode_kernel])
    if args.combine == "mean":
        kvr.kvr_sketch_set_combine(sk, kvr.KVR_COMBINE_MEAN)
    Kall = torch.empty((L, B, H, N, D), dtype=dt, device=dev)
    Vall = torch.empty_like(Kall)
    Qall = torch.empty((L, B, Hq, W, D), dtype=dt, device=dev)
    ws = dataclasses.replace(w, seed=w.seed + seed_shift)
    for layer in range(L):
        Kall[layer], Vall[layer], Qall[layer] = synth.layer_inputs(ws, layer, dev)
    qs = torch.stack([synth.decode_queries(ws, s, dev) for s in range(S)])          # [S, L, B, Hq, D]
    Kr = torch.empty((L, B, H, R, D), dtype=dt, device=dev)
    Vr = torch.empty_like(Kr)
    ret = torch.empty((L, B, H, R), dtype=torch.int32, device=dev)
    outs = torch.empty((S, L, B, Hq, D), dtype=torch.float32, device=dev)

    def compress_all():
        for layer in range(L):
            kvr.kvr_compress(sk, layer, Kall[layer], Vall[layer], Qall[layer], R, w.n_recent, Kr=Kr[layer], Vr=Vr[layer],
                             ret_idx=ret[layer])

    def decode_all():
        for s in range(S):
            for layer in range(L):
                kvr.kvr_decode_attention(sk, layer, qs[s, layer], Kr[layer], Vr[layer], ret[layer], out=outs[s, layer])

    # ---- untimed set-up: grow workspaces, then capture all decode launches of a step in a graph ----
    compress_all()
    kvr.kvr_decode_attention(sk, 0, qs[0, 0], Kr[0], Vr[0], ret[0], out=outs[0, 0])
    torch.cuda.synchronize()
    side = torch.cuda.Stream(device=dev)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            decode_all()
    torch.cuda.synchronize()
    decode_launches_per_step = S * L

    stream = torch.cuda.current_stream()
    launches0 = None
    ev_c, ev_d, ev_e = [], [], []
    try:
        gpu_id = "GPU-" + str(torch.cuda.get_device_properties(dev).uuid)
    except Exception:
        gpu_id = str(local)
    sampler = ClockSampler(gpu_id)
    clocks = None
    for step in range(args.warmup + args.steps):
        if step == args.warmup:
            torch.cuda.synchronize()
            kdist.barrier()
            torch.cuda.synchronize()
            launches0 = kvr.kvr_launch_count(sk)
            if rank == 0:
                sampler.start()
        a, b_, c = (torch.cuda.Event(enable_timing=True) for _ in range(3))
        a.record(stream)
        compress_all()
        b_.record(stream)
        graph.replay()
        c.record(stream)
        if step >= args.warmup:
            ev_c.append(a), ev_d.append(b_), ev_e.append(c)
    torch.cuda.synchronize()
    kdist.barrier()
    torch.cuda.synchronize()
    if rank == 0:
        clocks = sampler.stop()
    total_ms = ev_c[0].elapsed_time(ev_e[-1])
    compress_ms = sum(x.elapsed_time(y) for x, y in zip(ev_c, ev_d)) / args.steps
    decode_ms = sum(x.elapsed_time(y) for x, y in zip(ev_d, ev_e)) / args.steps
    eager_launches = kvr.kvr_launch_count(sk) - launches0
    gpu_launches = eager_launches + args.steps * decode_launches_per_step
    total_ms = kdist.max_over_ranks(total_ms, dev)
    ms_per_step = total_ms / args.steps
    value = world * B * S / (ms_per_step * 1e-3)

    # ---- roofline of the dominant kernel: the decode-attention launch (one per layer per decode step) ----
    peak, peak_kind = measured_peaks()
    launch_ms = decode_ms / decode_launches_per_step
    staged = kvr.kvr_last_decode_kernel(sk) == kvr.KVR_DECODE_STAGED
    kernel_name = "decode_staged_kernel" if staged else "decode_split_kernel"
    bytes_launch = decode_bytes_per_launch(w, B * H, 8 if staged else 4)
    ach = bytes_launch / (launch_ms * 1e-3) / 1e9
    roofline = {"kernel": kernel_name, "bound": "hbm", "achieved": round(ach, 1), "peak": peak,
                "peak_kind": peak_kind, "unit": "GB/s", "frac": round(ach / peak, 4),
                "frac_of_nominal_8TBs": round(ach / 8000.0, 4),
                "bytes_per_launch": bytes_launch, "avg_launch_us": round(launch_ms * 1e3, 2),
                "traffic": args.traffic}
    # The same launch against the two on-chip rates Algorithm 2 cannot avoid, both MEASURED on this
    # device a moment ago by the library's probe kernels (a register-only min/max loop and a
    # conflict-free 16-byte shared-memory load loop): the medians run on the ALU pipe, the two cells a
    # token does not keep in registers are read from shared memory once per pass.
    mm_peak, lds_peak = kvr.kvr_measure_pipe_peaks()
    alu_peak = mm_peak / 1e12                                              # T lane-ops/s
    alu_ach = minmax_ops_per_launch(w, B * H) / (launch_ms * 1e-3) / 1e12
    roofline_alu = {"kernel": kernel_name, "bound": "alu", "achieved": round(alu_ach, 3), "peak": round(alu_peak, 3),
                    "unit": "T min/max lane-ops/s", "frac": round(alu_ach / alu_peak, 4),
                    "peak_kind": "measured: register-only min/max loop (kvr_measure_pipe_peaks)"}
    smem_bytes = smem_cell_bytes_per_launch(w, B * H)
    smem_ach = smem_bytes / (launch_ms * 1e-3) / 1e9
    roofline_smem = {"kernel": kernel_name, "bound": "smem", "achieved": round(smem_ach, 1),
                     "peak": round(lds_peak / 1e9, 1), "unit": "GB/s", "frac": round(smem_ach / (lds_peak / 1e9), 4),
                     "bytes_per_launch": smem_bytes,
                     "peak_kind": "measured: 16-byte shared-memory load loop (kvr_measure_pipe_peaks)"}
    # which of the three ceilings is nearest (the largest fraction), and the time each alone would allow
    floors_us = {"hbm": bytes_launch / (peak * 1e9) * 1e6, "alu": minmax_ops_per_launch(w, B * H) / mm_peak * 1e6,
                 "smem": smem_bytes / lds_peak * 1e6}
    binding = {"nearest_ceiling": max(floors_us, key=floors_us.get),
               "floor_us": {k: round(v, 2) for k, v in floors_us.items()},
               "note": "the launch also spends instruction issue slots around these: at its instruction count the issue floor alone is about 22 us"}
    # ---- same decode work as ONE launch over all layers per decode step (upper bound on launch shape) ----
    batched = None
    if L > 1:
        o2 = torch.empty((L, B, Hq, D), dtype=torch.float32, device=dev)
        kvr.kvr_decode_attention(sk, kvr.KVR_ALL_LAYERS, qs[0], Kr, Vr, ret, out=o2)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        reps = 3
        e0.record(stream)
        for _ in range(reps):
            for s in range(S):
                kvr.kvr_decode_attention(sk, kvr.KVR_ALL_LAYERS, qs[s], Kr, Vr, ret, out=o2)
        e1.record(stream)
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / (reps * S)
        gbs = decode_bytes_per_launch(w, L * B * H, 8 if staged else 4) / (ms * 1e-3) / 1e9
        batched = {"ms_per_decode_step": round(ms, 4), "decode_tokens_per_s": round(B / (ms * 1e-3), 1),
                   "achieved_GBs": round(gbs, 1), "frac": round(gbs / peak, 4),
                   "alu_frac": round(minmax_ops_per_launch(w, L * B * H) / (ms * 1e-3) / 1e12 / alu_peak, 4)}
        # the two launch shapes cut the token lists differently: only the summation order differs
        batched["max_abs_diff_vs_per_layer"] = float((o2 - outs[S - 1]).abs().max().item())
        assert batched["max_abs_diff_vs_per_layer"] <= 5e-4, "layer-batched launch disagrees"

    # ---- end to end through the host-buffer calls: H2D of the step's inputs, D2H of its results ----
    e2e = None
    if not args.no_e2e:
        Kh, Vh, Qh = (torch.empty(x.shape, dtype=x.dtype, pin_memory=True).copy_(x) for x in (Kall, Vall, Qall))
        qh = torch.empty(qs.shape, dtype=qs.dtype, pin_memory=True).copy_(qs)
        oh = torch.empty((S, L, B, Hq, D), dtype=torch.float32, pin_memory=True)
        sk2 = kvr.kvr_sketch_create(b=w.b, batch=B, n_layers=L, n_kv_heads=H, n_q_heads=Hq, max_context=N,
                                    kv_dtype=dt, hash_seeds=seeds, device=dev)
        if args.combine == "mean":
            kvr.kvr_sketch_set_combine(sk2, kvr.KVR_COMBINE_MEAN)

        def e2e_step():
            for layer in range(L):
                kvr.kvr_compress_host(sk2, layer, Kh[layer], Vh[layer], Qh[layer], R, w.n_recent)
            for s in range(S):
                kvr.kvr_decode_attention_host(sk2, kvr.KVR_ALL_LAYERS, qh[s], oh[s])

        e2e_step()
        torch.cuda.synchronize()
        kdist.barrier()
        n_e2e = max(1, min(args.steps, 3))
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(n_e2e):
            e2e_step()
        e1.record(stream)
        torch.cuda.synchronize()
        ms = kdist.max_over_ranks(e0.elapsed_time(e1) / n_e2e, dev)
        h2d = Kh.numel() * 2 * 2 + Qh.numel() * 2 + qh.numel() * 2
        e2e = {"value": round(world * B * S / (ms * 1e-3), 2), "unit": UNIT, "ms_per_step": round(ms, 3),
               "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(oh.numel() * 4), "steps": n_e2e,
               "api": "kvr_compress_host per layer + kvr_decode_attention_host (all layers) per decode step"}
        assert float((oh.to(dev) - outs).abs().max().item()) <= 5e-4, "host-buffer path disagrees"
        kvr.kvr_sketch_destroy(sk2)
        del Kh, Vh, Qh

    checksum = float(outs.double().abs().sum().item())
    result = {
        "metric": METRIC, "value": round(value, 2), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": round(ms_per_step, 3), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": config_of(w),
        "decode_kernel": kernel_name,
        "compress_ms_per_step": round(compress_ms, 3), "decode_ms_per_step": round(decode_ms, 3),
        "compress": {"ms_per_layer": round(compress_ms / L, 4),
                     "achieved_GBs": round(compress_bytes_per_layer(w, B * H) / (compress_ms / L * 1e-3) / 1e9, 1),
                     "frac_of_measured_hbm": round(compress_bytes_per_layer(w, B * H) / (compress_ms / L * 1e-3) / 1e9 / peak, 4),
                     "bytes_per_layer": compress_bytes_per_layer(w, B * H),
                     "scoring_kernel": {kvr.KVR_SCORE_TCGEN05: "score_tc_kernel (tcgen05)",
                                        kvr.KVR_SCORE_MMA_SYNC: "score_pass_kernel (mma.sync)"}.get(kvr.kvr_last_score_kernel(sk), "?")},
        "decode_only_tokens_per_s": round(world * B * S / (decode_ms * 1e-3), 1),
        "roofline": roofline, "roofline_alu": roofline_alu, "roofline_smem": roofline_smem, "binding": binding, "layer_batched": batched, "e2e": e2e, "gpu_launches": int(gpu_launches),
        "clocks": clocks, "checksum": checksum,
        "device_bytes": kvr.kvr_sketch_device_bytes(sk),
    }
    kvr.kvr_sketch_destroy(sk)
    return result, (Kall, Vall, Qall, qs)


# ------------------------------------------------------------------- streaming generation (Algorithm 3)
def run_stream(args, w):
    """--stream T: after the compress, T generation steps; every step and layer runs the decode over
    the current storage, adds the step's attention mass to the scores of the stored rows and of the
    vague tokens (half of the steps as one call whose decode kernel keeps its logits, half as three calls
    that compute them twice), and takes the new token through Algorithm 3 (kvr_append: Recent part with Slack,
    pops into the sketch, swap loop with ReplaceRate 1.1).  One JSON line: generation tokens/s."""
    import paper_2512_17917_b200 as kvr

    dev = torch.device("cuda:0")
    torch.cuda.set_device(dev)
    L, B, H, Hq, D, N, R, T = w.n_layers, w.batch, w.n_kv_heads, w.n_q_heads, w.head_dim, w.context, w.budget, args.stream
    dt = w.torch_dtype
    r_budget = max(1, int(0.5 * R)) if w.n_recent else 64          # Recent budget (the storage-split preset keeps half)
    c_budget, slack, n_recent = R - min(r_budget, R), 32, w.n_recent
    sk = kvr.kvr_sketch_create(b=w.b, batch=B, n_layers=L, n_kv_heads=H, n_q_heads=Hq, max_context=N + T, kv_dtype=dt,
                               hash_seeds=synth.hash_seeds(w.seed + 3), device=dev)
    st = []
    for layer in range(L):
        K, V, Q = synth.layer_inputs(w, layer, dev)
        Kr, Vr, ret = kvr.kvr_compress(sk, layer, K, V, Q, R, n_recent)
        sc = torch.gather(kvr.kvr_get_scores(sk, layer), -1, ret.long()).contiguous()
        st.append([Kr, Vr, ret, sc, n_recent])
        del K, V, Q
    gen = torch.Generator(device=dev).manual_seed(w.seed + 99)
    new_k = (torch.randn((T, L, B, H, 1, D), generator=gen, device=dev)).to(dt)
    new_v = (torch.randn((T, L, B, H, 1, D), generator=gen, device=dev)).to(dt)
    qs = torch.stack([synth.decode_queries(w, s % max(1, w.decode_steps), dev) for s in range(T)])
    out = torch.empty((B, Hq, D), dtype=torch.float32, device=dev)

    def step(t, one_call):
        for layer in range(L):
            Kr, Vr, ret, sc, nr = st[layer]
            if one_call:                       # the decode kernel hands its logits to the score update
                kvr.kvr_decode_attention_scored(sk, layer, qs[t, layer], Kr, Vr, ret, sc, out=out)
            else:                              # the score update computes every logit again
                kvr.kvr_decode_attention(sk, layer, qs[t, layer], Kr, Vr, ret, out=out)
                kvr.kvr_accumulate_scores(sk, layer, qs[t, layer], Kr, sc)
                kvr.kvr_accumulate_vague_scores(sk, layer, qs[t, layer])
            Kr, Vr, ret, sc, nr, _ = kvr.kvr_append(sk, layer, Kr, Vr, ret, sc, nr, new_k[t, layer], new_v[t, layer],
                                                    r_budget, c_budget, slack, 1.1, 64)
            st[layer] = [Kr, Vr, ret, sc, nr]

    # the first half of the timed steps makes three calls per layer, the second half one: same storage sizes
    warm = min(3, T // 4)
    mid = warm + (T - warm) // 2
    for t in range(warm):
        step(t, t % 2 == 1)
    torch.cuda.synchronize()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
    ev[0].record()
    for t in range(warm, mid):
        step(t, False)
    ev[1].record()
    l0 = kvr.kvr_launch_count(sk)
    for t in range(mid, T):
        step(t, True)
    ev[2].record()
    torch.cuda.synchronize()
    ms3 = ev[0].elapsed_time(ev[1]) / max(1, mid - warm)
    ms = ev[1].elapsed_time(ev[2]) / (T - mid)
    assert kvr.kvr_sketch_device_status(sk) == 0 and torch.isfinite(out).all()
    res = {"metric": "stream_generation_tokens_per_s", "value": round(B / (ms * 1e-3), 2), "unit": UNIT, "n_gpus": 1,
           "steps": T - mid, "warmup": warm, "ms_per_step": round(ms, 3), "higher_is_better": True, "scaling": "weak",
           "vs_baseline": None, "dtype": "f32", "data": "synthetic",
           "config": dict(config_of(w), launch="eager, per layer: kvr_decode_attention_scored + kvr_append",
                          r_budget=r_budget, c_budget=c_budget, slack=slack, replace_rate=1.1),
           "three_calls": {"ms_per_step": round(ms3, 3), "steps": mid - warm,
                           "launch": "eager, per layer: decode + accumulate x2 + kvr_append"},
           "rows_after": int(st[0][0].shape[-2]), "context_after": N + T,
           "gpu_launches": int(kvr.kvr_launch_count(sk) - l0)}
    kvr.kvr_sketch_destroy(sk)
    return res


# ------------------------------------------------------------------- several queries per head
def mq_launches(rows: int) -> int:
    """Launches of one multi-query call: 64, 32 or 16 query rows per launch, as many as are left."""
    n = 0
    while rows > 0:
        rows -= 64 if rows > 32 else 32 if rows > 16 else 16
        n += 1
    return n


def run_mq(args, w):
    """--queries Qn: decode attention for Qn queries per head per call (kvr_decode_attention_mq) over the
    compressed cache of the workload, one call per layer, all layers and decode steps replayed from a
    CUDA graph.  One JSON line: query tokens per second, the time per layer call, the same bytes-based
    roofline as the single-query line (the cache is read once per call whatever Qn is), and the time
    of Qn single-query calls beside it."""
    import paper_2512_17917_b200 as kvr

    dev = torch.device("cuda:0")
    torch.cuda.set_device(dev)
    L, B, H, Hq, D, N, R, Qn = w.n_layers, w.batch, w.n_kv_heads, w.n_q_heads, w.head_dim, w.context, w.budget, args.queries
    S = max(1, min(w.decode_steps, 16))
    dt = w.torch_dtype
    sk = kvr.kvr_sketch_create(b=w.b, batch=B, n_layers=L, n_kv_heads=H, n_q_heads=Hq, max_context=N, kv_dtype=dt,
                               hash_seeds=synth.hash_seeds(w.seed + 3), device=dev)
    st = []
    for layer in range(L):
        K, V, Q = synth.layer_inputs(w, layer, dev)
        st.append(kvr.kvr_compress(sk, layer, K, V, Q, R, w.n_recent))
        del K, V, Q
    gen = torch.Generator(device=dev).manual_seed(w.seed + 77)
    qm = torch.randn((S, L, B, Hq, Qn, D), generator=gen, device=dev).to(dt)
    out = torch.empty((L, B, Hq, Qn, D), dtype=torch.float32, device=dev)
    out1 = torch.empty((L, B, Hq, D), dtype=torch.float32, device=dev)

    def graph_of(fn):
        fn()
        torch.cuda.synchronize()
        g, side = torch.cuda.CUDAGraph(), torch.cuda.Stream(device=dev)
        with torch.cuda.stream(side):
            with torch.cuda.graph(g, stream=side):
                fn()
        torch.cuda.synchronize()
        return g

    def mq_all():
        for s in range(S):
            for layer in range(L):
                kvr.kvr_decode_attention_mq(sk, layer, qm[s, layer], *st[layer], causal=False, out=out[layer])

    def single_all():
        for s in range(S):
            for layer in range(L):
                kvr.kvr_decode_attention(sk, layer, qm[s, layer, :, :, 0].contiguous(), *st[layer], out=out1[layer])

    def timed(g, reps):
        for _ in range(3):
            g.replay()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            g.replay()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps

    ms_mq = timed(graph_of(mq_all), max(1, args.steps))
    ms_1 = timed(graph_of(single_all), max(1, args.steps))
    assert kvr.kvr_sketch_device_status(sk) == 0 and torch.isfinite(out).all()
    peak, peak_kind = measured_peaks()
    call_us = ms_mq * 1e3 / (S * L)
    bytes_call = decode_bytes_per_launch(w, B * H) + B * Hq * Qn * D * 6
    res = {"metric": METRIC, "value": round(B * Qn * S / (ms_mq * 1e-3), 2), "unit": UNIT, "n_gpus": 1, "steps": args.steps,
           "warmup": 3, "ms_per_step": round(ms_mq, 3), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
           "dtype": "f32 accumulate, f16 hi+lo operands", "data": "synthetic",
           "config": dict(config_of(w), queries_per_head=Qn, decode_steps_per_step=S, launch="per_layer_cuda_graph"),
           "decode_kernel": "decode_mq_kernel", "layer_call_us": round(call_us, 2),
           "launches_per_layer_call": mq_launches(Hq // H * Qn),
           "roofline": {"kernel": "decode_mq_kernel", "bound": "hbm", "achieved": round(bytes_call / (call_us * 1e-6) / 1e9, 1),
                        "peak": peak, "peak_kind": peak_kind, "unit": "GB/s",
                        "frac": round(bytes_call / (call_us * 1e-6) / 1e9 / peak, 4), "bytes_per_launch": bytes_call,
                        "avg_launch_us": round(call_us, 2), "traffic": None},
           "single_query": {"layer_call_us": round(ms_1 * 1e3 / (S * L), 2),
                            "speedup_per_query": round(Qn * ms_1 / ms_mq, 2)},
           "gpu_launches": int(S * L * ((Hq // H * Qn + 15) // 16))}
    kvr.kvr_sketch_destroy(sk)
    return res


# ----------------------------------------------------------------------------- the CPU oracle
def oracle_sample(w, n_sample: int, decode_steps: int, inputs=None, combine: str = "median"):
    """Time the oracle, as it stands, on n_sample head-instances of layer 0: one compress and
    `decode_steps` decode steps.  Returns (compress_s, decode_s_per_step, cores)."""
    from oracle import kvr_oracle as orc

    H, Hq, N, D, W, R = w.n_kv_heads, w.n_q_heads, w.context, w.head_dim, w.obs_window, w.budget
    G = Hq // H
    if inputs is None:
        K, V, Q = synth.layer_inputs(w, 0, "cpu")
        qd = torch.stack([synth.decode_queries(w, s, "cpu")[0] for s in range(decode_steps)])
    else:
        K, V, Q = (x[0].cpu() for x in inputs[:3])
        qd = inputs[3][:decode_steps, 0].cpu()
    n_sample = min(n_sample, w.batch * H)
    Kc = K.float().reshape(-1, N, D).numpy()[:n_sample]
    Vc = V.float().reshape(-1, N, D).numpy()[:n_sample]
    Qc = Q.float().reshape(w.batch, H, G, W, D).reshape(-1, G * W, D).numpy()[:n_sample]
    seeds = synth.hash_seeds(w.seed + 3)
    orc.lib()
    t0 = time.perf_counter()
    c = orc.compress(Qc, Kc, Vc, R, w.n_recent, seeds, w.b)
    t1 = time.perf_counter()
    for s in range(decode_steps):
        qc = qd[s].float().reshape(-1, G, D).numpy()[:n_sample]
        orc.decode(qc, c["Kr"], c["Vr"], c["ret_idx"], c["cells"], N, seeds, combine=combine)
    t2 = time.perf_counter()
    return t1 - t0, (t2 - t1) / decode_steps, min(orc.max_threads(), n_sample), n_sample


def oracle_throughput(w, compress_s, decode_s, n_sample):
    """Whole-job tokens/s extrapolated from the sample (instances are independent and alike)."""
    scale = w.n_inst / n_sample
    step_s = scale * (compress_s + w.decode_steps * decode_s)
    return w.batch * w.decode_steps / step_s, step_s


def run_reference(args, w):
    """--impl reference: the CPU oracle on the host cores, each step a bounded sample."""
    cores = host_cores()
    n_sample = max(1, min(cores, w.batch * w.n_kv_heads))
    dsteps = 1
    vals, step_ms = [], []
    for i in range(args.warmup + args.steps):
        cs, ds, used, ns = oracle_sample(w, n_sample, dsteps, combine=args.combine)
        if i >= args.warmup:
            v, step_s = oracle_throughput(w, cs, ds, ns)
            vals.append(v)
            step_ms.append(step_s * 1e3)
    v = float(np.mean(vals))
    sample = (f"{n_sample} head-instances of layer 0 (of {w.n_inst}): one compress + {dsteps} decode step; "
              f"extrapolated x{w.n_inst / n_sample:.0f} instances and x{w.decode_steps} decode steps")
    return {
        "impl": "reference", "metric": METRIC, "value": round(v, 4), "unit": UNIT, "n_gpus": 1, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": round(float(np.mean(step_ms)), 1), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_of(w),
        "cpu_baseline": {"value": round(v, 4), "unit": UNIT, "cores": used, "kind": "oracle", "sample": sample},
        "e2e": {"value": round(v, 4), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(synth.WORKLOADS))
    ap.add_argument("--impl", default="kvr", choices=["kvr", "reference"])
    ap.add_argument("--all-workloads", action="store_true",
                    help="one JSON line per benchmark workload (the budget x width sweep of 8k_qwen3_8b_batch8 included); "
                         "no end-to-end and no CPU-baseline leg")
    ap.add_argument("--stream", type=int, default=0, help="time T generation steps with Algorithm 3 (kvr_append) instead")
    ap.add_argument("--queries", type=int, default=0, help="time decode attention with this many queries per head per call instead")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--layers", type=int, default=0, help="override the workload's layer count (profiling a small case)")
    ap.add_argument("--decode-steps", type=int, default=0, help="override the workload's decode steps per step")
    ap.add_argument("--budget-ratio", type=float, default=0.0, help="override the workload's retained fraction (sweeps)")
    ap.add_argument("--width-mult", type=float, default=0.0, help="override the sketch width multiplier (sweeps)")
    ap.add_argument("--preset", default="top_budget", choices=["top_budget", "paper"],
                    help="top_budget: the whole budget is exact top-scored rows, the sketch on top (the benchmark's "
                         "reading); paper: Recent 0.45 / Candidate 0.45 / Vague 0.10 of the budget, sketch inside it")
    ap.add_argument("--combine", default="median", choices=["median", "mean"],
                    help="what the query makes of a token's three cells: the paper's element-wise median, or their mean "
                         "(an option of the library; shows the launch time without the min/max arithmetic)")
    ap.add_argument("--decode-kernel", default="auto", choices=["auto", "split", "staged"],
                    help="force one of the two decode kernels (default: the library chooses)")
    ap.add_argument("--structured", action="store_true",
                    help="inputs with four sink tokens per head (peaked scores) instead of plain Gaussian keys")
    ap.add_argument("--traffic", type=float, default=None,
                    help="ncu dram bytes per decode launch to report in roofline.traffic (from profiles/)")
    args = ap.parse_args()
    if args.all_workloads:
        if not torch.cuda.is_available():
            raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback of the hot path)")
        rank, world, local = kdist.init_from_env()
        args.no_e2e = args.no_cpu_baseline = True
        args.warmup = max(args.warmup, 3)
        points = [(n, 0.0, 0.0) for n in ("2k_single_layer", "2k_llama3_8b", "32k_llama3_8b", "32k_llama3_8b_batch16")]
        points += [("8k_qwen3_8b_batch8", r, m) for r in (0.05, 0.10, 0.25, 0.50) for m in (0.5, 1.0, 2.0)]
        for name, ratio, mult in points:
            w = synth.WORKLOADS[name]
            if ratio:
                w = dataclasses.replace(w, budget_ratio=ratio, width_mult=mult, name=f"{name}[budget={ratio},width={mult}]")
            result, inputs = run_gpu(args, w, rank, world, local)
            del inputs
            torch.cuda.empty_cache()
            if rank == 0:
                print(json.dumps(result), flush=True)
        kdist.finalize()
        return
    w = synth.WORKLOADS[args.workload]
    if args.layers or args.decode_steps:
        w = dataclasses.replace(w, n_layers=args.layers or w.n_layers, decode_steps=args.decode_steps or w.decode_steps,
                                name=f"{w.name}[layers={args.layers or w.n_layers},decode_steps={args.decode_steps or w.decode_steps}]")

    if args.structured:
        w = dataclasses.replace(w, structured=True, name=f"{w.name}[sink tokens]")
    if args.preset == "paper":
        ratio = args.budget_ratio or w.budget_ratio
        if args.impl == "reference":
            from oracle import kvr_oracle as orc
            exact, n_recent, b_cells = orc.paper_split(w.context, ratio)
        else:
            import paper_2512_17917_b200 as kvr
            exact, n_recent, b_cells = kvr.kvr_paper_storage_split(w.context, ratio)
        w = dataclasses.replace(w, budget_ratio=ratio, budget_rows=exact, n_recent=n_recent, b_cells=b_cells,
                                name=f"{w.name}[paper split {ratio}: recent {n_recent}, candidate {exact - n_recent}, b {b_cells}]")
    elif args.budget_ratio or args.width_mult:
        w = dataclasses.replace(w, budget_ratio=args.budget_ratio or w.budget_ratio, width_mult=args.width_mult or w.width_mult,
                                name=f"{w.name}[budget={args.budget_ratio or w.budget_ratio},width={args.width_mult or w.width_mult}]")

    if args.combine != "median":
        w = dataclasses.replace(w, name=f"{w.name}[combine={args.combine}]")
    if args.impl == "reference":
        rank = int(os.environ.get("RANK", "0"))
        if rank == 0:
            print(json.dumps(run_reference(args, w)), flush=True)
        return

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback of the hot path)")
    if args.stream > 0:
        print(json.dumps(run_stream(args, w)), flush=True)
        return
    if args.queries > 0:
        print(json.dumps(run_mq(args, w)), flush=True)
        return
    if args.warmup < 3:
        args.warmup = 3
    rank, world, local = kdist.init_from_env()
    result, inputs = run_gpu(args, w, rank, world, local)
    if rank == 0:
        if not args.no_cpu_baseline:
            cores = host_cores()
            cs, ds, used, ns = oracle_sample(w, max(1, min(cores, w.batch * w.n_kv_heads)), 1, inputs, combine=args.combine)
            v, _ = oracle_throughput(w, cs, ds, ns)
            result["cpu_baseline"] = {
                "value": round(v, 4), "unit": UNIT, "cores": used, "kind": "oracle",
                "sample": (f"{ns} head-instances of layer 0 (of {w.n_inst}): one compress ({cs:.2f} s) + one decode "
                           f"step ({ds:.2f} s), extrapolated to all instances and {w.decode_steps} decode steps")}
        if result["roofline"]["traffic"] is None:
            result["roofline"]["traffic"] = default_traffic(w, result["roofline"]["kernel"])
        print(json.dumps(result), flush=True)
    kdist.finalize()


def default_traffic(w, kernel_name):
    """dram bytes per decode launch measured by ncu (one line per capture in profiles/decode_traffic.txt:
    workload, kernel, bytes), or None when no capture of this workload with this kernel is recorded."""
    p = os.path.join(ROOT, "profiles", "decode_traffic.txt")
    try:
        for line in open(p):
            f = line.split()
            if len(f) >= 3 and not line.startswith("#") and f[0] == w.name and f[1] == kernel_name:
                return float(f[2])
    except Exception:
        pass
    return None


if __name__ == "__main__":
    main()
