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
import hashlib
import json
import os
import re
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import synth  # noqa: E402

K_DRAFT = 4
SKIP_RATIO = 0.5
METRIC = "decode tokens/s at 7B-shape bf16 bs=1; achieved HBM GB/s vs ~8 TB/s roofline"
STEP_KERNEL_SRC = os.path.join(ROOT, "paper_2604_14612_b200", "csrc", "kernels_step.cu")
STEP_KERNEL_PROFILE = os.path.join(ROOT, "profiles", "k_token_steps_C3_8layers.txt")


def workload_string(w, K, ratio):
    """The same for both arms: names the model shape, the inputs and the loop."""
    s = w.shape
    return (f"{w.name}: {'13B' if w.name.startswith('C4') else '7B'}-shape Llama decoder (L{s.n_layers} d{s.d_model} F{s.d_ffn} "
            f"V{s.vocab}), {s.weight_dtype} weights, prompt {w.prompt_len}, generate {w.gen_len}, K={K}, "
            f"uniform {int(ratio * 100)}% skip set of layers {w.lo}..{w.hi}")


def algorithmic_bytes(shape, n_kept, ctx_len, rows=1):
    """Bytes one pass must move: kept layers' matrices + LM head + KV read of kept layers (+ KV write)."""
    d, F, V, es = shape.d_model, shape.d_ffn, shape.vocab, 2 if shape.weight_dtype != "fp32" else 4
    per_layer = es * (4 * d * d + 3 * d * F)
    kv = n_kept * (2 * es * d * ctx_len + 2 * es * d * rows)
    return n_kept * per_layer + es * V * d + kv


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        return json.load(open(p)), "measured"
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}, "fallback"


def step_kernel_traffic_ratio():
    """DRAM bytes / algorithmic bytes of the token-step kernel, from the committed ncu summary -- only while the kernel's
    source still is the one the counters were taken on (the summary records its SHA-256); None otherwise."""
    try:
        txt = open(STEP_KERNEL_PROFILE).read()
        ratio = float(re.search(r"^traffic_ratio:\s*([0-9.]+)", txt, re.M).group(1))
        sha = re.search(r"^kernels_step_sha256:\s*([0-9a-f]{64})", txt, re.M).group(1)
        now = hashlib.sha256(open(STEP_KERNEL_SRC, "rb").read()).hexdigest()
        return ratio if sha == now else None
    except Exception:
        return None


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


def oracle_sample_text(K):
    return f"{ORACLE_CYCLES} draft-{K}/verify/accept cycles of the workload after a 2-token prefill"


def run_reference(args, rank):
    """The reference arm for this tier is the CPU oracle, as it stands, on the host cores."""
    if rank != 0:
        return
    import torch
    w = synth.WORKLOADS["C3"]
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
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": "tokens/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * secs / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32 (f64 reductions)", "data": "synthetic",
            "config": {"workload": workload_string(w, K_DRAFT, SKIP_RATIO)},
            "cpu_baseline": {"value": val, "unit": "tokens/s", "cores": cores, "kind": "oracle",
                             "sample": oracle_sample_text(K_DRAFT) + " per step"},
            "e2e": {"value": val, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def c5_scoring(torch, cl, peaks, peak_kind):
    """The all-layer confidence scoring workload (C5): 8 rounds of score -> select -> best; tensor-core bound."""
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
    out = {"score_loop_ms": ms5, "tflops": tf5, "bound": "tensor", "frac_of_bf16_burst": tf5 / float(peaks["bf16_tflops"]),
           "frac_of_bf16_sustained": tf5 / float(peaks["bf16_tflops_sustained"]), "peak_kind": f"of {peak_kind}"}
    ctx5.close()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip the oracle timing (profiling runs)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-extra", action="store_true", help="skip the extra measurements under config.extra (profiling runs)")
    ap.add_argument("--layers", type=int, default=0, help="fewer layers of the same shape (profiling captures only)")
    ap.add_argument("--gen", type=int, default=0, help="fewer generated tokens per step (profiling captures only)")
    ap.add_argument("--c5-only", action="store_true", help="only the C5 scoring loop; prints its object (profiling captures)")
    args = ap.parse_args()
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
    peaks, peak_kind = measured_peaks()
    peak = float(peaks["hbm_gbs"])
    if args.c5_only:
        print(json.dumps({"c5_scoring": c5_scoring(torch, cl, peaks, peak_kind)}), flush=True)
        return

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def event_ms(fn, n):
        """Average device time of fn() over n calls, CUDA events on the stream the library launches on."""
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(n):
            fn()
        e1.record()
        barrier()
        return e0.elapsed_time(e1) / n

    def make_case(name, damp=None):
        w = synth.WORKLOADS[name]
        if args.layers:
            w = synth.reduced(w, n_layers=args.layers, prompt_len=w.prompt_len, gen_len=w.gen_len, max_seq=w.shape.max_seq)
        if args.gen:
            w = dataclasses.replace(w, gen_len=args.gen)
        W = synth.make_weights(w.shape, w.seed, device="cuda")
        if damp is not None:
            synth.damp_output_projections(W, damp[0], damp[1])
        ctx = cl.Context.from_shape(w.shape, tap_positions=64)
        ctx.cl_load(W)
        prompt = synth.make_prompt(w.seed, w.prompt_len, w.shape.vocab)
        return w, W, ctx, prompt

    def uniform_mask(w, ratio):
        n_skip = synth.n_skip_for_ratio(w.lo, w.hi, ratio)
        layers = synth.uniform_skip_layers(w.lo, w.hi, n_skip)
        return synth.layers_to_mask(layers, w.shape.n_layers), w.shape.n_layers - len(layers)

    def generate_run(ctx, w, first, K, steps):
        """steps x (rollback to the prompt, generate gen_len tokens); device time, counters."""
        def one():
            ctx.cl_rollback(w.prompt_len, first)
            return ctx.cl_generate(K, w.gen_len)
        one()
        barrier()
        s0 = ctx.cl_get_stats()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            one()
        e1.record()
        barrier()
        ms = reduce_over_ranks(e0.elapsed_time(e1), dist, "cuda")
        s1 = ctx.cl_get_stats()
        cyc, acc, dr = int(s1.cycles - s0.cycles), int(s1.accepted - s0.accepted), int(s1.drafted - s0.drafted)
        return dict(ms=ms, cycles=cyc, alpha=acc / dr if dr else None, accepted_per_cycle=acc / cyc if cyc else None,
                    launches=int(s1.kernel_launches - s0.kernel_launches), tokens=steps * w.gen_len)

    def summarize(w, r, K, n_kept):
        ctx_mid = w.prompt_len + w.gen_len // 2
        cyc_bytes = K * algorithmic_bytes(w.shape, n_kept, ctx_mid) + algorithmic_bytes(w.shape, w.shape.n_layers, ctx_mid, rows=K + 1)
        gbs = r["cycles"] * cyc_bytes / (r["ms"] * 1e-3) / 1e9
        return {"tokens_per_s": r["tokens"] / (r["ms"] * 1e-3), "alpha": r["alpha"], "accepted_per_cycle": r["accepted_per_cycle"],
                "ms_per_cycle": r["ms"] / r["cycles"], "whole_cycle_gbs": gbs, "whole_cycle_frac": gbs / peak}

    # ------------------------------------------------------------------ the workload the metric is quoted on
    w, W, ctx, prompt = make_case("C3")
    shape, gen = w.shape, w.gen_len
    mask, n_kept = uniform_mask(w, SKIP_RATIO)
    cpu_base = None
    if rank == 0 and not args.no_cpu_baseline:
        Wh = synth.weights_to(W, "cpu")
        n, dt, cores = oracle_sample(shape, Wh, prompt, mask, K_DRAFT)
        cpu_base = {"value": n / dt, "unit": "tokens/s", "cores": cores, "kind": "oracle",
                    "sample": oracle_sample_text(K_DRAFT) + f" ({n} tokens in {dt:.1f} s)"}
        del Wh
    del W
    torch.cuda.empty_cache()

    first = ctx.cl_prefill(prompt)
    ctx.cl_set_skip_set(mask)
    for _ in range(args.warmup - 1):
        ctx.cl_rollback(w.prompt_len, first)
        ctx.cl_generate(K_DRAFT, gen)
    sampler = ClockSampler(local) if rank == 0 else None
    main_run = generate_run(ctx, w, first, K_DRAFT, args.steps)   # (one more untimed step inside)
    clocks = sampler.stop() if sampler else {}
    value = whole_job_value(main_run["tokens"], world, main_run["ms"])
    main_sum = summarize(w, main_run, K_DRAFT, n_kept)

    # ------------------------------------------------------------------ the phases of a cycle, each on its own
    ctx_mid = w.prompt_len + gen // 2
    ctx.cl_rollback(ctx_mid, first)
    n_rep = 8 * max(1, min(args.steps, 5))
    for _ in range(3):
        ctx.cl_draft(K_DRAFT)
    draft_ms = event_ms(lambda: ctx.cl_draft(K_DRAFT), n_rep)
    draft_bytes = K_DRAFT * algorithmic_bytes(shape, n_kept, ctx_mid)
    achieved = draft_bytes / (draft_ms * 1e-3) / 1e9
    for _ in range(3):
        ctx.cl_verify(K_DRAFT + 1)
    verify_ms = event_ms(lambda: ctx.cl_verify(K_DRAFT + 1), n_rep)
    verify_bytes = algorithmic_bytes(shape, shape.n_layers, ctx_mid, rows=K_DRAFT + 1)

    cycle_ms = main_sum["ms_per_cycle"]
    ratio = step_kernel_traffic_ratio()
    roofline = {
        "bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
        "traffic": ratio * draft_bytes if ratio else None, "peak_kind": f"of {peak_kind}", "frac_of_8TBps": achieved / 8000.0,
        "kernel": f"k_token_steps, one launch = {K_DRAFT} draft steps over {n_kept} kept layers + LM head",
        "ms_per_launch": draft_ms, "bytes_per_launch": draft_bytes,
        "verify": {"kernel": f"k_rows_pass, one launch = the {K_DRAFT + 1}-row full-model pass", "bytes": verify_bytes, "ms": verify_ms,
                   "achieved": verify_bytes / (verify_ms * 1e-3) / 1e9, "frac": verify_bytes / (verify_ms * 1e-3) / 1e9 / peak},
        # draft and verify are timed alone, back to back; the rest of a cycle (the accept kernel, the host's read of its
        # result, the gaps between launches) is what remains of the cycle time measured in the generation loop
        "phases_ms_per_cycle": {"cycle": cycle_ms, "draft": draft_ms, "verify": verify_ms,
                                "accept_and_gaps": cycle_ms - draft_ms - verify_ms},
        "whole_cycle_gbs": main_sum["whole_cycle_gbs"], "whole_cycle_frac": main_sum["whole_cycle_frac"],
    }

    # ------------------------------------------------------------------ extra measurements (short runs)
    extra = {}
    ctx.cl_prefill(prompt)
    vr = generate_run(ctx, w, first, 0, 1)
    van_gbs = gen * algorithmic_bytes(shape, shape.n_layers, ctx_mid) / (vr["ms"] * 1e-3) / 1e9
    extra["vanilla"] = {"tokens_per_s": gen / (vr["ms"] * 1e-3), "achieved_gbs": van_gbs, "frac_of_peak": van_gbs / peak}
    if not args.no_extra:
        # the rest of the 7B matrix: K in {4, 8} x {uniform 25 %, uniform 50 %, confidence-selected}
        first_t = ctx.cl_prefill(prompt, tap_hidden=True)
        ctx.cl_layer_confidences()
        n_conf = min(w.n_skip_conf, (w.hi - w.lo + 1) // 2)
        cmask, _ = ctx.cl_select_skip_set(cl.SelectCfg.make(w.lo, w.hi, n_skip=n_conf))
        sets = {"uniform25": uniform_mask(w, 0.25), "uniform50": (mask, n_kept),
                "confidence_selected": (cmask, shape.n_layers - int(np.count_nonzero(cmask)))}
        matrix = {}
        for K in w.K:
            for sname, (m, kept) in sets.items():
                ctx.cl_set_skip_set(m)
                matrix[f"K{K}_{sname}"] = dict(summarize(w, generate_run(ctx, w, first_t, K, 1), K, kept),
                                               skipped=[int(l) for l in np.nonzero(m)[0]])
        extra["c3_matrix"] = matrix
    ctx.cl_set_skip_set(mask)

    # end to end through the public API with host buffers: prompt H2D + prefill + generate + tokens D2H
    e2e = None
    if not args.no_e2e:
        barrier()
        t0 = time.perf_counter()
        n_e2e = max(1, min(args.steps, 3))
        for _ in range(n_e2e):
            ctx.cl_prefill(prompt)
            ctx.cl_generate(K_DRAFT, gen)
        barrier()
        dt = reduce_over_ranks(time.perf_counter() - t0, dist, "cuda")
        e2e = {"value": world * n_e2e * gen / dt, "unit": "tokens/s", "h2d_bytes_per_step": int(4 * w.prompt_len),
               "d2h_bytes_per_step": int(4 * gen), "includes": f"prefill of the {w.prompt_len}-token prompt in every step"}
    ctx.close()
    torch.cuda.empty_cache()

    if rank == 0 and not args.no_extra and not args.layers:
        # a model whose skipped layers add little to the residual stream (what a trained model's skippable layers look
        # like): the same shape and kernels with drafts that are mostly accepted
        skipped = [int(l) for l in np.nonzero(mask)[0]]
        wd_, Wd, ctxd, _ = make_case("C3", damp=(skipped, 0.02))
        del Wd
        fd = ctxd.cl_prefill(prompt)
        ctxd.cl_set_skip_set(mask)
        rd = generate_run(ctxd, wd_, fd, K_DRAFT, 1)
        vd = generate_run(ctxd, wd_, fd, 0, 1)
        extra["c3_accepting_model"] = dict(summarize(wd_, rd, K_DRAFT, n_kept),
                                           model="output and down projections of the skipped layers scaled by 0.02",
                                           vanilla_tokens_per_s=gen / (vd["ms"] * 1e-3),
                                           speedup_over_vanilla=(rd["tokens"] / rd["ms"]) / (gen / vd["ms"]))
        ctxd.close()
        torch.cuda.empty_cache()
        # the 13B shape: K = 6, uniform 40 %
        w4, W4, ctx4, p4 = make_case("C4")
        del W4
        m4, kept4 = uniform_mask(w4, 0.4)
        f4 = ctx4.cl_prefill(p4)
        ctx4.cl_set_skip_set(m4)
        r4 = generate_run(ctx4, w4, f4, 6, 1)
        v4 = generate_run(ctx4, w4, f4, 0, 1)
        v4_gbs = w4.gen_len * algorithmic_bytes(w4.shape, w4.shape.n_layers, w4.prompt_len + w4.gen_len // 2) / (v4["ms"] * 1e-3) / 1e9
        extra["c4"] = dict(summarize(w4, r4, 6, kept4), workload=workload_string(w4, 6, 0.4),
                           vanilla_tokens_per_s=w4.gen_len / (v4["ms"] * 1e-3), vanilla_frac_of_peak=v4_gbs / peak)
        ctx4.close()
        torch.cuda.empty_cache()
        extra["c5_scoring"] = c5_scoring(torch, cl, peaks, peak_kind)

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": main_run["ms"] / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16 weights, f32 accumulate", "data": "synthetic",
            "config": {"workload": workload_string(w, K_DRAFT, SKIP_RATIO),
                       "l2": f"{algorithmic_bytes(shape, shape.n_layers, 0) / 1e9:.0f} GB of weights per pass, far larger than L2: every pass re-streams from HBM",
                       "parallelism": "replicas only" if world > 1 else "1 GPU",
                       "alpha": main_run["alpha"], "cycles_per_step": main_run["cycles"] / args.steps, "extra": extra},
            "roofline": roofline, "cpu_baseline": cpu_base, "e2e": e2e, "gpu_launches": main_run["launches"], "clocks": clocks,
        }
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
