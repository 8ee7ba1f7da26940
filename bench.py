#!/usr/bin/env python
"""Benchmark of the ConfLayers hot path on B200: decode tokens/s at the 7B shape (bf16, batch 1).

A "step" is one whole pass of the hot path over one batch of synthetic input: from a prefilled
512-token context, generate 256 greedy tokens with self-speculative cycles (draft K with the
skip-masked model, one (K+1)-row verify pass, greedy accept).  Weights (13 GB) are far larger than
L2, so every step streams them from HBM again.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints ONE JSON line (see the keys below).  With N > 1 (launched by torch.distributed.run) every
rank runs an independent replica of the same job ("replicas only": batch-1 decode has no
independent units to shard); value is the aggregate over ranks, time is the max over ranks.
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

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import synth  # noqa: E402

WORKLOAD = "C3"
K_DRAFT = 4
SKIP_RATIO = 0.5
TRAFFIC_RATIO = 0.992   # ncu dram bytes / algorithmic bytes of the token-step kernel (profiles/); None once stale
METRIC = "decode tokens/s at 7B-shape bf16 bs=1; achieved HBM GB/s vs ~8 TB/s roofline"


def algorithmic_bytes(shape, n_kept, ctx_len, rows=1):
    """Bytes one pass must move: kept layers' matrices + LM head + KV read of kept layers (+ KV write)."""
    d, F, V, es = shape.d_model, shape.d_ffn, shape.vocab, 2 if shape.weight_dtype == "bf16" else 4
    per_layer = es * (4 * d * d + 3 * d * F)
    kv = n_kept * (2 * es * d * ctx_len + 2 * es * d * rows)
    return n_kept * per_layer + es * V * d + kv


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        j = json.load(open(p))
        return float(j["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def reduce_over_ranks(ms_local, dist=None, device=None):
    """A timed region costs what its slowest rank took: MAX over ranks (one rank: the value itself)."""
    if dist is None:
        return float(ms_local)
    import torch
    t = torch.tensor([float(ms_local)], device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(units_per_rank, world, ms):
    """Replicas only: every rank runs the same job, the aggregate is world x units over the slowest rank's time."""
    return world * units_per_rank / (ms * 1e-3)


class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None
        try:
            self.p = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                                       "-lms", "200", "-i", str(index)], stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.p = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": []}
        if self.p is None:
            return out
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except Exception:
            self.p.kill()
        self.f.flush()
        rows = [r.strip().split(", ") for r in open(self.f.name) if r.strip()]
        os.unlink(self.f.name)
        sm, mx, reasons = [], [], set()
        for r in rows:
            if len(r) < 9:
                continue
            try:
                sm.append(float(r[1])); mx.append(float(r[2]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[5:9]):
                if v.strip().lower().startswith("active"):
                    reasons.add(name)
        if sm:
            out = {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                   "samples": len(sm)}
        return out


ORACLE_CYCLES = 8   # speculative cycles per oracle sample: about 10 s of CPU work at the 7B shape


def oracle_sample(shape, weights_host, prompt, mask, K, n_cycles=ORACLE_CYCLES):
    """n_cycles speculative cycles of the CPU oracle after a 2-token prefill; returns (tokens, seconds, threads)."""
    import oracle
    om = oracle.OracleModel(shape, weights_host)
    p = prompt[:2]
    t0, _, _ = oracle.prefill(om, p)
    ctx_len, tok, emitted = len(p), t0, 0
    t = time.perf_counter()
    for _ in range(n_cycles):
        cyc = oracle.speculative_cycle(om, mask, tok, ctx_len, K)
        emitted += len(cyc["emitted"])
        ctx_len, tok = cyc["new_ctx"], cyc["next_t0"]
    dt = time.perf_counter() - t
    om.close()
    return emitted, dt, int(os.environ.get("OMP_NUM_THREADS", os.cpu_count() or 1))


def run_reference(args, rank):
    """The reference arm for this tier is the CPU oracle, as it stands, on the host cores."""
    if rank != 0:
        return
    import torch
    w = synth.WORKLOADS[WORKLOAD]
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    W = synth.make_weights(w.shape, w.seed, device=dev)
    Wh = synth.weights_to(W, "cpu") if dev != "cpu" else W
    del W
    prompt = synth.make_prompt(w.seed, w.prompt_len, w.shape.vocab)
    n_skip = synth.n_skip_for_ratio(w.lo, w.hi, SKIP_RATIO)
    mask = synth.layers_to_mask(synth.uniform_skip_layers(w.lo, w.hi, n_skip), w.shape.n_layers)
    for _ in range(args.warmup):
        oracle_sample(w.shape, Wh, prompt, mask, K_DRAFT)
    toks, secs, cores = 0, 0.0, 1
    for _ in range(args.steps):
        n, dt, cores = oracle_sample(w.shape, Wh, prompt, mask, K_DRAFT)
        toks += n
        secs += dt
    val = toks / secs
    sample = f"{ORACLE_CYCLES} draft-{K_DRAFT}/verify/accept cycles of {WORKLOAD} after a 2-token prefill per step"
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": "tokens/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * secs / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32 (f64 reductions)", "data": "synthetic",
            "config": {"workload": f"{WORKLOAD}: 7B-shape Llama decoder, bf16 weights, K={K_DRAFT}, "
                                   f"uniform {int(SKIP_RATIO * 100)}% skip set"},
            "cpu_baseline": {"value": val, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip the oracle timing (profiling runs)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--layers", type=int, default=0, help="fewer layers of the same shape (profiling captures only)")
    ap.add_argument("--gen", type=int, default=0, help="fewer generated tokens per step (profiling captures only)")
    ap.add_argument("--workload", default="C3", choices=["C3", "C4"],
                    help="C3 (7B shape, K=4, 50%% skip) is the configuration the metric is quoted on; C4 = the 13B shape "
                         "(K=6, 40%% skip) as an extra measurement")
    args = ap.parse_args()
    global WORKLOAD, K_DRAFT, SKIP_RATIO
    if args.workload == "C4":
        WORKLOAD, K_DRAFT, SKIP_RATIO = "C4", 6, 0.4
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank)
        return
    args.warmup = max(args.warmup, 3)

    import torch
    import paper_2604_14612_b200 as cl
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    w = synth.WORKLOADS[WORKLOAD]
    if args.layers:
        w = synth.reduced(w, n_layers=args.layers, prompt_len=w.prompt_len, gen_len=w.gen_len, max_seq=w.shape.max_seq)
    if args.gen:
        w = dataclasses.replace(w, gen_len=args.gen)
    shape = w.shape
    W = synth.make_weights(shape, w.seed, device="cuda")
    ctx = cl.Context.from_shape(shape)
    ctx.cl_load(W)
    prompt = synth.make_prompt(w.seed, w.prompt_len, shape.vocab)
    n_skip = synth.n_skip_for_ratio(w.lo, w.hi, SKIP_RATIO)
    skip_layers = synth.uniform_skip_layers(w.lo, w.hi, n_skip)
    mask = synth.layers_to_mask(skip_layers, shape.n_layers)
    n_kept = shape.n_layers - len(skip_layers)
    gen = w.gen_len

    cpu_base = None
    if rank == 0 and not args.no_cpu_baseline:
        Wh = synth.weights_to(W, "cpu")
        n, dt, cores = oracle_sample(shape, Wh, prompt, mask, K_DRAFT)
        cpu_base = {"value": n / dt, "unit": "tokens/s", "cores": cores, "kind": "oracle",
                    "sample": f"{ORACLE_CYCLES} draft-{K_DRAFT}/verify/accept cycles of {w.name} after a 2-token prefill "
                              f"({n} tokens in {dt:.1f} s)"}
        del Wh
    del W
    torch.cuda.empty_cache()

    first = ctx.cl_prefill(prompt)
    ctx.cl_set_skip_set(mask)

    def step(K):
        ctx.cl_rollback(w.prompt_len, first)
        return ctx.cl_generate(K, gen)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(K, steps):
        barrier()
        s0 = ctx.cl_get_stats()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            toks, st = step(K)
        e1.record()
        barrier()
        ms = reduce_over_ranks(e0.elapsed_time(e1), dist, "cuda")
        s1 = ctx.cl_get_stats()
        return ms, s0, s1

    for _ in range(args.warmup):
        step(K_DRAFT)
    sampler = ClockSampler(local) if rank == 0 else None
    ms, s0, s1 = timed(K_DRAFT, args.steps)
    clocks = sampler.stop() if sampler else {}
    launches = int(s1.kernel_launches - s0.kernel_launches)
    cycles = int(s1.cycles - s0.cycles)
    accepted = int(s1.accepted - s0.accepted)
    drafted = int(s1.drafted - s0.drafted)
    tokens = args.steps * gen
    value = whole_job_value(tokens, world, ms)

    # bytes the timed cycles had to stream (algorithmic): K draft passes + one verify pass per cycle
    ctx_mid = w.prompt_len + gen // 2
    draft_bytes = K_DRAFT * algorithmic_bytes(shape, n_kept, ctx_mid)
    cyc_bytes = draft_bytes + algorithmic_bytes(shape, shape.n_layers, ctx_mid, rows=K_DRAFT + 1)
    cycle_gbs = cycles * cyc_bytes / (ms * 1e-3) / 1e9
    peak, peak_kind = measured_peaks()

    # the dominant kernel on its own: one launch of the token-step kernel = K draft steps with the skip set,
    # timed with CUDA events on the launching stream at the mid-run context length
    ctx.cl_rollback(ctx_mid, first)
    n_draft = 8 * max(1, args.steps)
    for _ in range(3):
        ctx.cl_draft(K_DRAFT)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(n_draft):
        ctx.cl_draft(K_DRAFT)
    e1.record()
    barrier()
    draft_ms = e0.elapsed_time(e1) / n_draft
    achieved = draft_bytes / (draft_ms * 1e-3) / 1e9
    # DRAM traffic per launch: ncu counters of the same kernel on an 8-layer case (profiles/), where
    # dram read + write bytes were 0.992 x the algorithmic bytes; traffic grows with the bytes scheduled
    traffic = TRAFFIC_RATIO * draft_bytes if TRAFFIC_RATIO else None

    # vanilla decoding with the same kernels (context for the speculative number)
    step(0)
    ms_v, _, _ = timed(0, 1)
    vanilla_tps = gen / (ms_v * 1e-3)
    vanilla_gbs = gen * algorithmic_bytes(shape, shape.n_layers, ctx_mid) / (ms_v * 1e-3) / 1e9

    # the all-layer confidence scoring workload (C5): 8 rounds of score -> select -> best, tensor-core bound
    c5 = None
    if rank == 0 and not args.layers:
        cc = synth.C5
        L5, P5, d5, V5 = cc["n_layers"], cc["positions"], cc["d_model"], cc["vocab"]
        head5 = synth.make_lm_head(cc["seed"], V5, d5, device="cuda")
        ctx5 = cl.Context(L5, d5, d5 // 128, 11008, V5, 8, "bf16", rms_eps=cc["rms_eps"])
        ctx5.cl_load(dict(lm_head=head5, final_norm=torch.ones(d5, device="cuda")), head_only=True)
        hid5 = [synth.make_hidden(cc["seed"], t, L5, P5, d5, device="cuda") for t in range(cc["iters"])]
        sc5 = synth.make_round_scores(cc["seed"], cc["iters"])
        sel5 = cl.SelectCfg.make(cc["lo"], cc["hi"], n_skip=cc["n_skip"])
        for _ in range(3):
            ctx5.cl_score_loop(sel5, hid5, sc5)
        t5 = []
        for _ in range(5):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            ctx5.cl_score_loop(sel5, hid5, sc5)
            e1.record()
            torch.cuda.synchronize()
            t5.append(e0.elapsed_time(e1))
        ms5 = statistics.median(t5)
        tf5 = cc["iters"] * 2.0 * L5 * P5 * d5 * V5 / (ms5 * 1e-3) / 1e12
        pk = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json"))) if os.path.exists(os.path.join(ROOT, "MEASURED_PEAKS.json")) else {}
        sus = float(pk.get("bf16_tflops_sustained", 1400.0))
        c5 = {"score_loop_ms": ms5, "tflops": tf5, "frac_of_bf16_sustained": tf5 / sus,
              "peak_kind": "of measured" if pk else "of fallback"}
        ctx5.close()
        del head5, hid5

    # end to end through the public API with host buffers: prompt H2D + prefill + generate + tokens D2H
    e2e = None
    if not args.no_e2e:
        barrier()
        t0 = time.perf_counter()
        n_e2e = max(1, min(args.steps, 3))
        for _ in range(n_e2e):
            ctx.cl_prefill(prompt)
            toks, _ = ctx.cl_generate(K_DRAFT, gen)
        barrier()
        dt = reduce_over_ranks(time.perf_counter() - t0, dist, "cuda")
        e2e = {"value": world * n_e2e * gen / dt, "unit": f"tokens/s (prefill of the {w.prompt_len}-token prompt included)",
               "h2d_bytes_per_step": int(4 * w.prompt_len), "d2h_bytes_per_step": int(4 * gen)}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16 weights, f32 accumulate", "data": "synthetic",
            "config": {"workload": f"{w.name}: {'13B' if WORKLOAD == 'C4' else '7B'}-shape Llama decoder (L{shape.n_layers} d{shape.d_model} "
                                   f"F{shape.d_ffn} V{shape.vocab}), prompt {w.prompt_len}, generate {gen}, K={K_DRAFT}, "
                                   f"uniform {int(SKIP_RATIO * 100)}% skip set of layers {w.lo}..{w.hi}",
                       "l2": f"{algorithmic_bytes(shape, shape.n_layers, 0) / 1e9:.0f} GB of weights per pass, far larger than L2: every pass re-streams from HBM",
                       "parallelism": "replicas only" if world > 1 else "1 GPU",
                       "alpha": accepted / drafted if drafted else None, "cycles_per_step": cycles / args.steps,
                       "vanilla_tokens_per_s": vanilla_tps, "vanilla_achieved_gbs": vanilla_gbs,
                       "vanilla_frac_of_peak": vanilla_gbs / peak, "c5_scoring": c5},
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "traffic": traffic, "peak_kind": f"of {peak_kind}", "frac_of_8TBps": achieved / 8000.0,
                         "kernel": f"k_token_steps, one launch = {K_DRAFT} draft steps over {n_kept} kept layers + LM head",
                         "ms_per_launch": draft_ms, "bytes_per_launch": draft_bytes,
                         "whole_cycle_gbs": cycle_gbs, "whole_cycle_frac": cycle_gbs / peak},
            "cpu_baseline": cpu_base, "e2e": e2e, "gpu_launches": launches, "clocks": clocks,
        }
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
