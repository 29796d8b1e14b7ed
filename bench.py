#!/usr/bin/env python
"""Benchmark of the bounded self-speculative decode step (SpecBound) on B200.

One "step" = one whole generation of the workload (prefill + all draft/verify rounds) for one
synthetic prompt.  ``value`` is batch-1 decode tokens/s of the speculative path, timed on the
device (CUDA events on the library's stream around the decode phase, prompt and weights already
in HBM); ``e2e`` is the same metric through the public call with host buffers (prompt copied
host->device, prefill, decode, tokens copied device->host all inside the timed region).
The autoregressive baseline on the same GPU, the speed-up, the per-phase split, the roofline of
the verify pass and of the exit-confidence kernel, and the CPU oracle timed on the host cores
are reported in the same JSON line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--workload 7b]

With N > 1 (launched by torch.distributed.run) every rank decodes its own prompt on its own GPU:
replicas only, no data-path collective; NCCL is used for the barrier and the max-over-ranks time.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time
from pathlib import Path

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

import numpy as np
import torch

from paper_2604_12247_b200 import inputs

NOMINAL_HBM_GBS = 8000.0


def metric_name(run: "inputs.Run") -> str:
    return f"batch-1 decode tokens/s (SpecBound, {run.shape.name})"


def captured_traffic(key: str):
    """DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) from the committed ncu capture
    summaries, or None if there is none for this kernel."""
    p = ROOT / "profiles" / "traffic.json"
    try:
        return json.loads(p.read_text()).get(key)
    except Exception:
        return None


def measured_peak():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        try:
            return float(json.loads(p.read_text())["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
        except Exception:
            pass
    return 6650.0, "fallback (6.65 TB/s, earlier measurement on this pool)"


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "200",
                                          "-i", str(self.index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=lambda: self.lines.extend(self.proc.stdout), daemon=True)
            self.t.start()
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.25)
        self.proc.terminate()
        self.t.join(timeout=2)
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def aggregate_replicas(dec_ms: float, call_ms: float, steps: int, dec_tokens: int, gen_tokens: int, world: int,
                       device: str = "cuda"):
    """Replica aggregation: every rank decodes its own sequence; the job's time is the slowest rank's
    (max over ranks), its throughput the tokens of all ranks over that time.  Returns (value, e2e)."""
    t = torch.tensor([dec_ms, call_ms], dtype=torch.float64, device=device)
    if world > 1:
        import torch.distributed as dist
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dec_max, call_max = t.tolist()
    return world * steps * dec_tokens / (dec_max / 1e3), world * steps * gen_tokens / (call_max / 1e3), dec_max, call_max


def kv_bytes_per_pos(s: inputs.Shape) -> int:
    return 2 * s.n_kv_heads * s.head_dim * (4 if s.dtype == "f32" else 2)


def cpu_oracle_sample(run: inputs.Run, weights_cpu: dict, p: int = 2, g: int = 4):
    """Times the oracle's plain greedy decoding on a bounded sample: a p-token prompt and g
    generated tokens = p + g - 1 full forward passes at short context."""
    from oracle import oracle
    pr = inputs.make_prompt(run.shape, p, run.seed).numpy()
    o = oracle.Oracle(run.shape, weights_cpu, p + g + 1)
    t0 = time.perf_counter()
    o.ar_generate(pr, g)
    dt = time.perf_counter() - t0
    o.close()
    passes = p + g - 1
    cores = len(os.sched_getaffinity(0))
    return {"value": passes / dt, "unit": "tokens/s", "cores": cores, "kind": "oracle",
            "sample": f"oracle greedy decoding, {p}-token prompt + {g} tokens = {passes} full forward passes "
                      f"({run.shape.name}, {run.shape.dtype} weights, fp64 arithmetic, OpenMP over output rows), {dt:.1f} s"}, dt


def cpu_oracle_specbound_sample(run: inputs.Run, weights_cpu: dict, p: int, g: int):
    """Times the oracle's SpecBound loop (Section 3.3) on a bounded sample of the workload: a p-token prompt and g
    generated tokens with the workload's d_max, w_max, temperatures and threshold.  The decode phase is what the
    metric counts, so the prefill (the same loop asked for one token) is timed separately and taken off.
    Returns (decode tokens/s, decode seconds, total seconds, rounds)."""
    from oracle import oracle
    pr = inputs.make_prompt(run.shape, p, run.seed).numpy()
    max_seq = p + g + run.w_max + 1
    o = oracle.Oracle(run.shape, weights_cpu, max_seq)
    t0 = time.perf_counter()
    o.specbound_generate(pr, 1, run.d_max, run.w_max, run.tau, run.threshold)
    t_prefill = time.perf_counter() - t0
    o.close()
    o = oracle.Oracle(run.shape, weights_cpu, max_seq)
    t0 = time.perf_counter()
    _, rounds = o.specbound_generate(pr, g, run.d_max, run.w_max, run.tau, run.threshold)
    t_all = time.perf_counter() - t0
    o.close()
    dec = max(t_all - t_prefill, 1e-9)
    return (g - 1) / dec, dec, t_all + t_prefill, len(rounds)


def host_weights(run: inputs.Run):
    if torch.cuda.is_available():
        w = inputs.make_weights(run.shape, run.seed, device="cuda", damp_rho=run.damp_rho)
        return inputs.weights_to(w, "cpu")
    return inputs.make_weights(run.shape, run.seed, device="cpu", damp_rho=run.damp_rho)


REF_PROMPT, REF_GEN = 4, 8   # the slice of the workload one reference step decodes


def reference_arm(args, run: inputs.Run):
    """--impl reference: the CPU oracle as it stands, on the host cores, same metric (decode tokens/s of the SpecBound
    loop) and hyper-parameters; every step decodes a bounded slice of the workload (REF_PROMPT prompt tokens,
    REF_GEN generated tokens), stated in config.timed_slice, first speculatively, then autoregressively."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import oracle
    oracle.build()
    w = host_weights(run)
    for _ in range(args.warmup):
        cpu_oracle_sample(run, w, 1, 1)
    dec_s, tot_s, ar_tps, rounds = [], [], [], 0
    for _ in range(args.steps):
        _, dec, tot, rounds = cpu_oracle_specbound_sample(run, w, REF_PROMPT, REF_GEN)
        desc, dt = cpu_oracle_sample(run, w, REF_PROMPT, REF_GEN)
        dec_s.append(dec); tot_s.append(tot + dt); ar_tps.append(desc["value"])
    v = args.steps * (REF_GEN - 1) / sum(dec_s)
    cfg = workload_config(run, "cpu-oracle")
    cfg["timed_slice"] = (f"each step: {REF_PROMPT}-token prompt + {REF_GEN} generated tokens of this workload through the oracle's "
                          f"SpecBound loop (value = decode tokens/s, prefill taken off), then the same slice autoregressively; "
                          f"NOT the full {run.n_prompt} + {run.n_gen} tokens")
    cores = len(os.sched_getaffinity(0))
    base = {"value": v, "unit": "tokens/s", "cores": cores, "kind": "oracle",
            "sample": f"oracle SpecBound loop, {REF_PROMPT}-token prompt + {REF_GEN} tokens ({rounds} rounds), d_max {run.d_max}, w_max "
                      f"{run.w_max}, {run.shape.name}, {run.shape.dtype} weights, fp64 arithmetic, OpenMP over output rows; "
                      f"{sum(dec_s) / len(dec_s):.1f} s of decoding per step",
            "ar_forward_passes_per_s": sum(ar_tps) / len(ar_tps)}
    line = {"impl": "reference", "metric": metric_name(run), "value": v, "unit": "tokens/s", "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": 1e3 * sum(tot_s) / len(tot_s), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": cfg, "cpu_baseline": base,
            "e2e": {"value": v, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def workload_config(run: inputs.Run, parallelism: str) -> dict:
    s = run.shape
    return {"workload": f"{s.name}: {s.n_layers} layers, d={s.d_model}, {s.n_heads} heads/{s.n_kv_heads} kv, ffn {s.d_ffn}, "
                        f"vocab {s.vocab}, {s.dtype}, random-init N(0,0.02) head x{s.head_scale:g}"
                        + (f", damped deep layers rho={run.damp_rho}" if run.damp_rho else ""),
            "batch": 1, "prompt_tokens": run.n_prompt, "generated_tokens": run.n_gen, "d_max": run.d_max, "w_max": run.w_max,
            "tau": [round(t, 4) for t in run.tau], "threshold": run.threshold, "parallelism": parallelism,
            "l2": "inputs larger than L2 (every layer pass streams >= 400 MB of distinct weights)"}


def verify_roofline(s: inputs.Shape, stats, peak: float):
    """Achieved bandwidth of the verify pass over the unified passes of `stats`: algorithmic bytes of one layer pass =
    the layer's weights once + K,V of the positions attended over (read) / appended (written), whatever the rows."""
    wb = inputs.weight_bytes(s)
    S = lambda f: sum(getattr(st, f) for st in stats)
    uni_steps, uni_us, uni_pos = S("unified_layer_steps"), S("us_unified"), S("unified_kv_positions")
    uni_bytes = uni_steps * wb["layer"] + uni_pos * kv_bytes_per_pos(s)
    ach = uni_bytes / (uni_us * 1e-6) / 1e9 if uni_us > 0 else 0.0
    return ach, uni_bytes, uni_steps, uni_us


def oracle_check(ctx, run: inputs.Run, weights_cpu: dict, n_prompt: int, n_gen: int) -> dict:
    """Accepted tokens against the oracle: the GPU decodes n_gen tokens from a short prompt with the workload's own
    weights and hyper-parameters (speculatively and autoregressively), and the oracle makes ONE teacher-forced pass
    over prompt + GPU tokens, reporting for every generated position its own top-1, the top-2 margin and how far the
    GPU's token lies below the top-1 logit.  A GPU token is correct if it is the oracle's top-1 or the margin at that
    position is below the logit tolerance (2e-2 for bf16 storage, 1e-4 for fp32); such positions are counted.  (A
    teacher-forced pass over the workload's full prompt would take the host cores tens of minutes.)"""
    from oracle import oracle
    tol = 2e-2 if run.shape.dtype == "bf16" else 1e-4
    pr = inputs.make_prompt(run.shape, n_prompt, run.seed + 5).numpy()
    sp = ctx.generate(pr, n_gen, run.d_max, run.w_max, run.tau, run.threshold)
    ar = ctx.generate_ar(pr, n_gen)
    toks = np.concatenate([pr, sp["tokens"]]).astype(np.int32)
    t0 = time.perf_counter()
    o = oracle.Oracle(run.shape, weights_cpu, len(toks) + 1)
    top1, _, margin, deficit = o.teacher_forced(toks, n_prompt)
    off = top1 != sp["tokens"]
    # How far the free-running GPU state has drifted from the oracle's at the position with the smallest margin (or the
    # first one that is not the oracle's top-1): the row that decides that token is run again on both sides layer by
    # layer (the oracle's cache holds the earlier positions from the pass above), and the ORACLE's head is applied to
    # both final hidden states.  The drift comes from K/V cache entries that land on a neighbouring bf16 value on one
    # side; it grows with depth and says how large a margin a legitimate difference can flip.
    j = int(np.nonzero(off)[0][0]) if off.any() else int(np.argmin(margin))
    drift = None
    if j >= 1:
        pos = n_prompt + j - 1
        ctx.reset()
        ctx.prefill(toks[:pos])
        ctx.draft_push(int(toks[pos]))
        ctx.draft_advance(run.shape.n_layers)
        h_gpu = ctx.read_hidden(0).astype(np.float64)
        ctx.reset()
        h_orc = o.embed(int(toks[pos]))[None, :]
        for l in range(1, run.shape.n_layers + 1):
            h_orc = o.layer_forward(l, h_orc, pos)
        z_o, z_g = o.final_logits(h_orc[0]), o.final_logits(h_gpu)
        drift = {"generated_index": j, "margin_there": float(margin[j]),
                 "hidden_rel_err_last_layer": float(np.abs(h_gpu - h_orc[0]).max() / np.abs(h_orc[0]).max()),
                 "logit_diff_rms": float(np.sqrt(np.mean((z_g - z_o) ** 2))), "logit_diff_max": float(np.abs(z_g - z_o).max())}
    o.close()
    dt = time.perf_counter() - t0
    return {"prompt_tokens": n_prompt, "positions": int(n_gen), "not_top1": int(off.sum()),
            "near_ties": int((margin < 2 * tol).sum()), "wrong": int((off & (margin >= 2 * tol)).sum()),
            "worst_deficit": float(deficit.min()), "logit_tolerance": tol, "smallest_margin": float(margin.min()),
            "tokens_equal_ar": bool(np.array_equal(sp["tokens"], ar["tokens"])), "oracle_seconds": dt,
            "free_running_drift": drift,
            "what": "teacher-forced oracle pass over a short-prompt generation of this workload (same weights, d_max, w_max, "
                    "tau, threshold); wrong = GPU token differs from the oracle's top-1 at a position whose top-2 margin is "
                    "not below twice the tolerance; free_running_drift = the oracle's head applied to the GPU's and to the "
                    "oracle's final hidden state of the row that decides the token with the smallest margin"}


def side_arm(args, workload: str, peak: float, masked: bool = False, steps: int = 3) -> dict:
    """Another workload measured the same way as the main one, for a few steps, as extra keys of the default run's
    line: `7b-damped` (damped deep layers: the synthetic stand-in for trained exit heads, with the paper's own
    hyper-parameters -- the configuration in which drafts get accepted; also with the probe-layer mask that did best in
    the hyper-parameter study) and the other full-size shapes (`l3-8b`, `13b`) at their own lengths."""
    from paper_2604_12247_b200 import binding
    run = inputs.RUNS[workload]
    s = run.shape
    w = inputs.make_weights(s, run.seed, device="cuda", damp_rho=run.damp_rho)
    prompt = inputs.make_prompt(s, run.n_prompt, run.seed).numpy()
    ctx = binding.Context(s, w, run.n_prompt + run.n_gen + run.w_max + 8, kv_page=64)
    steps = max(1, min(args.steps, steps))
    ctx.generate(prompt, run.n_gen, run.d_max, run.w_max, run.tau, run.threshold)
    ctx.generate_ar(prompt, 32)
    stats = [ctx.generate(prompt, run.n_gen, run.d_max, run.w_max, run.tau, run.threshold) for _ in range(steps)]
    ars = [ctx.generate_ar(prompt, run.n_gen) for _ in range(steps)]
    dec_tok = run.n_gen - 1
    value = steps * dec_tok / (sum(r["stats"].us_decode_dev for r in stats) * 1e-6)
    ar_value = steps * dec_tok / (sum(r["stats"].us_decode_dev for r in ars) * 1e-6)
    ach, _, uni_steps, uni_us = verify_roofline(s, [r["stats"] for r in stats], peak)
    st = stats[-1]["stats"]
    wb = inputs.weight_bytes(s)
    probe_us = sum(r["stats"].us_probe_kernels for r in stats) / max(sum(r["stats"].probes_timed for r in stats), 1)
    out = {"workload": workload_config(run, "single GPU"), "steps": steps, "value": value, "unit": "tokens/s",
           "ar_tokens_per_s": ar_value, "speedup_vs_ar": value / ar_value,
           "tokens_equal_ar": bool(np.array_equal(stats[-1]["tokens"], ars[-1]["tokens"])),
           "emitted_per_round": st.emitted / max(st.rounds, 1), "accepted_drafts_per_round": st.accepted_drafts / max(st.rounds, 1),
           "probes_per_step": st.probes, "exit_hist": list(st.exit_hist[:run.d_max + 1]), "width_hist": list(st.width_hist),
           "ttft_ms": st.us_prefill / 1e3,
           "roofline_frac": ach / peak, "verify_us_per_layer": uni_us / max(uni_steps, 1),
           "roofline_exit_frac": wb["head"] / (probe_us * 1e-6) / 1e9 / peak if probe_us > 0 else None}
    if masked:   # only every second layer is tested for an exit
        tau_m = [t if l % 2 == 0 else 0.0 for l, t in enumerate(run.tau, start=1)]
        ctx.generate(prompt, run.n_gen, run.d_max, run.w_max, tau_m, run.threshold)
        runs = [ctx.generate(prompt, run.n_gen, run.d_max, run.w_max, tau_m, run.threshold) for _ in range(steps)]
        m_value = steps * dec_tok / (sum(r["stats"].us_decode_dev for r in runs) * 1e-6)
        mst = runs[-1]["stats"]
        out["every_second_layer_probed"] = {"value": m_value, "speedup_vs_ar": m_value / ar_value,
                                            "tokens_equal_ar": bool(np.array_equal(runs[-1]["tokens"], ars[-1]["tokens"])),
                                            "emitted_per_round": mst.emitted / max(mst.rounds, 1), "probes_per_step": mst.probes,
                                            "tau": [round(t, 4) for t in tau_m]}
    ctx.close()
    return out


def product_arm(args, run: inputs.Run):
    import torch.distributed as dist
    from paper_2604_12247_b200 import binding, build
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU fallback)"
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if rank == 0:
        build.build()
    if world > 1:
        dist.barrier()
    s = run.shape
    w = inputs.make_weights(s, run.seed, device="cuda", damp_rho=run.damp_rho)
    prompt = inputs.make_prompt(s, run.n_prompt, run.seed + 17 * rank).numpy()
    ctx = binding.Context(s, w, run.n_prompt + run.n_gen + run.w_max + 8, kv_page=64)
    gen = lambda: ctx.generate(prompt, run.n_gen, run.d_max, run.w_max, run.tau, run.threshold)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        gen()
    ctx.generate_ar(prompt, min(run.n_gen, 64))
    sampler = ClockSampler(local)
    barrier()
    sampler.start()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    stats, call_ms = [], []
    barrier()
    t_region = time.perf_counter()
    for _ in range(args.steps):
        ev0.record()
        res = gen()
        ev1.record()
        ev1.synchronize()
        call_ms.append(ev0.elapsed_time(ev1))
        stats.append(res["stats"])
    barrier()
    t_region = time.perf_counter() - t_region
    clocks = sampler.stop()
    spec_tokens = res["tokens"]

    ar_stats = []
    for _ in range(args.steps):
        ar = ctx.generate_ar(prompt, run.n_gen)
        ar_stats.append(ar["stats"])
    tokens_equal = bool(np.array_equal(ar["tokens"], spec_tokens))

    dec_tok = run.n_gen - 1                          # the first token comes out of prefill
    dec_ms = sum(st.us_decode_dev for st in stats) / 1e3
    value, e2e, dec_ms_max, call_ms_max = aggregate_replicas(dec_ms, sum(call_ms), args.steps, dec_tok, run.n_gen, world)
    ar_ms = sum(st.us_decode_dev for st in ar_stats) / 1e3
    ar_value = args.steps * dec_tok / (ar_ms / 1e3)

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    peak, peak_src = measured_peak()
    wb = inputs.weight_bytes(s)
    S = lambda f: sum(getattr(st, f) for st in stats)
    ach, uni_bytes, uni_steps, uni_us = verify_roofline(s, stats, peak)
    roofline = {"kernel": "verify pass: one decoder layer for w<=8 rows (weight-streaming GEMMs + paged-KV attention), "
                          "averaged over the unified passes of the event-bracketed rounds (one round in four) of the timed region",
                "bound": "hbm", "achieved": ach, "peak": peak, "unit": "GB/s", "frac": ach / peak,
                "peak_source": peak_src, "frac_of_nominal_8TBs": ach / NOMINAL_HBM_GBS,
                "bytes_per_launch": uni_bytes / max(uni_steps, 1), "us_per_launch": uni_us / max(uni_steps, 1),
                "launches": uni_steps, "traffic": captured_traffic(f"layer_pass:{s.name}")}
    probes, probe_us = S("probes_timed"), S("us_probe_kernels")   # one probe in 32 is bracketed by events
    ach_p = probes * wb["head"] / (probe_us * 1e-6) / 1e9 if probe_us > 0 else 0.0
    roofline_exit = {"kernel": "exit-confidence kernel (final RMSNorm'd row x LM head, fused temperature softmax max/argmax)",
                     "bound": "hbm", "achieved": ach_p, "peak": peak, "unit": "GB/s", "frac": ach_p / peak,
                     "frac_of_nominal_8TBs": ach_p / NOMINAL_HBM_GBS, "bytes_per_launch": wb["head"],
                     "us_per_launch": probe_us / max(probes, 1), "launches": probes,
                     "traffic": captured_traffic(f"exit_confidence:{s.name}")}
    st0 = stats[-1]
    line = {
        "metric": metric_name(run), "value": value, "unit": "tokens/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": dec_ms_max / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "storage_dtype": s.dtype, "data": "synthetic",
        "config": workload_config(run, f"replicas x{world}" if world > 1 else "single GPU"),
        "ar_tokens_per_s": ar_value, "speedup_vs_ar": (value / world) / ar_value,
        "tokens_equal_ar": tokens_equal,
        "ar_frac_of_weight_stream_bound": ar_value / (peak * 1e9 / wb["model"]),
        "e2e": {"value": e2e, "unit": "tokens/s", "h2d_bytes_per_step": int(st0.h2d_bytes), "d2h_bytes_per_step": int(st0.d2h_bytes),
                "note": "sb_generate with host prompt/token buffers: prompt H2D + prefill + decode + result D2H"},
        "gpu_launches": int(S("kernel_launches")),
        "rounds_per_step": st0.rounds, "emitted_per_round": st0.emitted / max(st0.rounds, 1),
        "accepted_drafts_per_round": st0.accepted_drafts / max(st0.rounds, 1), "probes_per_step": st0.probes,
        "exit_hist": list(st0.exit_hist[:run.d_max + 1]), "width_hist": list(st0.width_hist),
        "ttft_ms": statistics.median(st.us_prefill for st in stats) / 1e3,
        "ttft_note": "time to first token through sb_generate: prompt host->device, prefill of all prompt tokens (wide passes), "
                     "first token device->host; host wall clock, median over the timed steps",
        "phase_ms_per_step": {"prefill_host": st0.us_prefill / 1e3, "decode_dev": st0.us_decode_dev / 1e3,
                              # the library brackets one round in four with events (rounds_timed) and one probe in 32
                              # (probes_timed): scaled to all rounds / probes of the step
                              "draft_dev": st0.us_draft / 1e3 * st0.rounds / max(st0.rounds_timed, 1),
                              "verify_dev": st0.us_verify / 1e3 * st0.rounds / max(st0.rounds_timed, 1),
                              "unified_dev": st0.us_unified / 1e3 * st0.rounds / max(st0.rounds_timed, 1),
                              "probe_kernels_dev": st0.us_probe_kernels / 1e3 * st0.probes / max(st0.probes_timed, 1),
                              "rounds_timed": st0.rounds_timed, "probes_timed": st0.probes_timed},
        "roofline": roofline, "roofline_exit": roofline_exit, "clocks": clocks,
        "paper_context": "paper reports up to 2.33x wall-time speed-up over AR on 1x H800 with trained exit heads "
                         "(Table 1); random-init weights here give near-chance draft acceptance",
        "timed_region_wall_s": t_region,
    }
    if world == 1 and not args.no_cpu_baseline:
        from oracle import oracle
        oracle.build()
        wc = inputs.weights_to(w, "cpu")
        line["cpu_baseline"], _ = cpu_oracle_sample(run, wc, 4, 40)   # 43 forward passes: about 10-30 s of CPU work
        if args.oracle_check_tokens > 0:
            line["oracle_check"] = oracle_check(ctx, run, wc, 16, args.oracle_check_tokens)
        del wc
    ctx.close()
    if world == 1 and args.workload == "7b" and not args.no_damped:
        line["damped"] = side_arm(args, "7b-damped", peak, masked=True)
        if not args.no_other_shapes:
            line["other_shapes"] = {name: side_arm(args, name, peak, steps=1) for name in ("l3-8b", "13b")}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def sweep_arm(args, run: inputs.Run):
    """Hyper-parameter study in the spirit of the paper's ablations (Section 4.4: confidence threshold gamma, annealing
    strength alpha, depth bound d_max, width bound w_max; without ACT / without d_max / without w_max), on the
    synthetic workload given by --workload at its own prompt and generation lengths (--sweep-short: at most 256 + 256
    tokens).  Every point reports decode tokens/s of SpecBound, the speed-up over autoregressive decoding with the same
    kernels, tokens emitted per round, whether the tokens equal the autoregressive ones, and what Eq. 5 predicts from
    the measured per-draft acceptance rate.  Also: the decoding strategies of Section 4.3 / Table 2, a probe-layer
    mask study (layers whose exit test rarely passes are not tested), and a least-squares fit of the round-cost model
    T = t_layer * layer_steps + t_probe * probes + t_round * rounds to all measured points (Eq. 3 is this with
    t_probe = t_round = 0 and every draft charged d_max layers).  One JSON line."""
    from paper_2604_12247_b200 import binding, build
    build.build()
    torch.cuda.set_device(0)
    s = run.shape
    L = s.n_layers
    w = inputs.make_weights(s, run.seed, device="cuda", damp_rho=run.damp_rho)
    short = getattr(args, "sweep_short", False)
    n_prompt, n_gen = (min(run.n_prompt, 256), min(run.n_gen, 256)) if short else (run.n_prompt, run.n_gen)
    pr = inputs.make_prompt(s, n_prompt, run.seed).numpy()
    ctx = binding.Context(s, w, n_prompt + n_gen + 16, kv_page=64 if n_prompt + n_gen > 1024 else 16)
    ar = None
    for _ in range(2):
        ar = ctx.generate_ar(pr, n_gen)
    ar_tps = (n_gen - 1) / (ar["stats"].us_decode_dev * 1e-6)
    alpha0 = (run.tau[0] - 1.0) / (1.0 - 1.0 / L) if run.tau[0] > 1.0 else 0.0   # Eq. 1 strength of the workload's schedule
    eq1 = abs(run.tau[-1] - (1.0 + alpha0 * (1.0 - run.d_max / L))) < 1e-6        # the workload's schedule is Eq. 1

    def tau_for(d_max, alpha=None):
        if alpha is not None:
            return [1.0 + alpha * (1.0 - l / L) for l in range(1, d_max + 1)]
        if eq1:
            return [1.0 + alpha0 * (1.0 - l / L) for l in range(1, d_max + 1)]
        return list(inputs.tau_linear(d_max, run.tau[0], run.tau[-1]))

    def measure(label, d_max, w_max, thr, tau, **extra):
        ctx.generate(pr, n_gen, d_max, w_max, tau, thr)   # warm-up (descriptor cache)
        sp = ctx.generate(pr, n_gen, d_max, w_max, tau, thr)
        st = sp["stats"]
        tps = (n_gen - 1) / (st.us_decode_dev * 1e-6)
        drafts = sum(st.exit_hist[1:])                      # rows that produced a draft
        acc = st.accepted_drafts / drafts if drafts else 0.0
        pt = {"point": label, "d_max": d_max, "w_max": w_max, "threshold": thr, "tokens_per_s": tps, "speedup_vs_ar": tps / ar_tps,
              "tokens_equal_ar": bool((sp["tokens"] == ar["tokens"]).all()), "rounds": st.rounds,
              "emitted_per_round": st.emitted / max(st.rounds, 1), "mean_width": st.rows / max(st.rounds, 1),
              "draft_acceptance": acc,
              "eq5_speedup_at_that_acceptance": binding.model_speedup(L, min(acc, 0.999), w_max, d_max),
              "probes": st.probes, "layer_steps": st.layer_steps, "decode_us": st.us_decode_dev,
              "exit_hist": list(st.exit_hist[:d_max + 1])}
        pt.update(extra)
        return pt

    depths = [int(x) for x in args.depths.split(",")] if getattr(args, "depths", None) else \
        [d for d in (1, 2, 4, 6, 8, 10, 12) if d < L]
    widths = [int(x) for x in args.widths.split(",")] if getattr(args, "widths", None) else [2, 4, 8]
    points = [measure("bounds", d, wm, run.threshold, tau_for(d)) for d in depths for wm in widths]
    points += [measure("threshold", run.d_max, run.w_max, th, tau_for(run.d_max))
               for th in (0.3, 0.4, 0.5, 0.6, 0.7, 0.8, 0.9) if th != run.threshold]
    # annealing strength of Eq. 1 (alpha = 0 is decoding without ACT: every layer tested at temperature 1)
    alphas = [measure("alpha", run.d_max, run.w_max, run.threshold, tau_for(run.d_max, a), alpha=a)
              for a in (0.0, 0.1, 0.2, 0.4, 0.8, 1.6)]
    # component ablation (Section 4.4): the full method, then one component off at a time
    base = measure("full", run.d_max, run.w_max, run.threshold, list(run.tau[:run.d_max]))
    ablation = [base,
                measure("without ACT (tau = 1 at every layer)", run.d_max, run.w_max, run.threshold, [1.0] * run.d_max),
                measure("without d_max (drafting may go to layer L-1)", L - 1, run.w_max, run.threshold, tau_for(L - 1)),
                measure("without w_max (the library's row limit, 8)", run.d_max, 8, run.threshold, list(run.tau[:run.d_max]))]
    # probe-layer mask from the exit histogram of the full method: layers that catch fewer than 2 % of the drafted rows
    # are walked but not tested; also: test every second layer only
    hist = base["exit_hist"]
    rows = max(sum(hist), 1)
    keep = [hist[l] / rows >= 0.02 for l in range(1, run.d_max + 1)]
    masks = [("full schedule", [True] * run.d_max), ("layers catching >= 2 % of the rows", keep),
             ("every second layer", [l % 2 == 0 for l in range(1, run.d_max + 1)]),
             ("last layer only", [l == run.d_max for l in range(1, run.d_max + 1)])]
    mask_points = []
    for label, m in masks:
        if not any(m):
            continue
        tau = [t if on else 0.0 for t, on in zip(run.tau[:run.d_max], m)]
        mask_points.append(measure(label, run.d_max, run.w_max, run.threshold, tau, probed_layers=[l + 1 for l, on in enumerate(m) if on]))
    # least-squares fit of the round-cost model to every measured point
    allp = points + alphas + ablation + mask_points
    A = np.array([[p["layer_steps"], p["probes"], p["rounds"]] for p in allp], dtype=np.float64)
    y = np.array([p["decode_us"] for p in allp])
    coef, *_ = np.linalg.lstsq(A, y, rcond=None)
    pred = A @ coef
    wb = inputs.weight_bytes(s)
    fit = {"model": "decode_us = t_layer * layer_steps + t_probe * probes + t_round * rounds (a layer step carries 1..w rows; "
                    "t_round = final head on w rows + acceptance + the host's look at the result)",
           "t_layer_us": float(coef[0]), "t_probe_us": float(coef[1]), "t_round_us": float(coef[2]),
           "probe_over_layer_fitted": float(coef[1] / coef[0]) if coef[0] else None,
           "probe_over_layer_bytes": wb["head"] / wb["layer"],
           "max_rel_residual": float(np.max(np.abs(pred - y) / y)), "points": len(allp),
           "ar_token_us_measured": 1e6 / ar_tps, "ar_token_us_from_fit": float(coef[0] * L + coef[2])}
    # decoding strategies (Section 4.3, Table 2): greedy, temperature and top-p sampling at the workload's own setting;
    # under sampling the baseline is autoregressive sampling with the same temperature and seed
    strategies = []
    tau = list(run.tau[:run.d_max])
    for name, temp, top_p in (("greedy", 0.0, 1.0), ("temperature 0.3", 0.3, 1.0), ("temperature 1.0", 1.0, 1.0),
                              ("top-p 0.9", 1.0, 0.9)):
        if getattr(args, "no_strategies", False):
            break
        ctx.set_sampling(temp, run.seed, top_p)
        for _ in range(2):
            a = ctx.generate_ar(pr, n_gen)
            sp = ctx.generate(pr, n_gen, run.d_max, run.w_max, tau, run.threshold)
        a_tps = (n_gen - 1) / (a["stats"].us_decode_dev * 1e-6)
        tps = (n_gen - 1) / (sp["stats"].us_decode_dev * 1e-6)
        st = sp["stats"]
        drafts = sum(st.exit_hist[1:])
        strategies.append({"strategy": name, "ar_tokens_per_s": a_tps, "tokens_per_s": tps, "speedup_vs_ar": tps / a_tps,
                           "tokens_equal_ar": bool((sp["tokens"] == a["tokens"]).all()),
                           "emitted_per_round": st.emitted / max(st.rounds, 1),
                           "draft_acceptance": st.accepted_drafts / drafts if drafts else 0.0})
    ctx.set_sampling(0.0, 0)
    out = {"mode": "sweep", "workload": workload_config(run, "single GPU")["workload"], "prompt_tokens": n_prompt,
           "generated_tokens": n_gen, "ar_tokens_per_s": ar_tps, "points": points, "alpha_sweep": alphas,
           "ablation": ablation, "probe_mask": mask_points, "cost_model_fit": fit, "decoding_strategies": strategies}
    if getattr(args, "oracle_check_tokens", 0) > 0 and not getattr(args, "no_cpu_baseline", True):
        from oracle import oracle
        oracle.build()
        wc = inputs.weights_to(w, "cpu")
        out["oracle_check"] = oracle_check(ctx, run, wc, 16, args.oracle_check_tokens)
    ctx.close()
    print(json.dumps(out), flush=True)


def micro_arm(args):
    """Kernel micro-benchmarks (bf16, 7B-shaped layer): the verify pass of one layer for w rows over
    a KV cache of S positions, and the exit-confidence kernel against LM heads of two vocabulary
    sizes.  L2 is defeated by rotating over distinct weight copies totalling more than 1 GB."""
    from paper_2604_12247_b200 import binding, build
    build.build()
    torch.cuda.set_device(0)
    peak, peak_src = measured_peak()
    base = inputs.RUNS[args.workload].shape            # --workload picks the layer's geometry (default: the 7B shape)
    if base.dtype != "bf16":
        raise SystemExit("--micro needs a bf16 workload")
    s = inputs.scaled(base, n_layers=1)
    out = {"mode": "micro", "shape": base.name, "peak_gbs": peak, "peak_source": peak_src, "iters": args.iters, "layer": [], "exit": []}
    ev = lambda: torch.cuda.Event(enable_timing=True)
    cases = [c for c in args.micro_case.split(",") if c] if args.micro_case else None

    def want(name):
        return cases is None or name in cases

    n_copies = 4
    layers = None
    chain_layers = None
    n_chain = 32     # distinct layer weight sets run back to back in the chained mode: 13 GB, the L2 defeat of a real pass
    for S in (512, 2048, 8192):
        for w in (1, 2, 4, 6, 8):
            name = f"layer:w={w}:S={S}"
            if not want(name):
                continue
            if layers is None:
                layers = [inputs.make_weights(s, 100 + i, device="cuda")["layers"][0] for i in range(n_copies)]
                lws = [binding.layer_weights(lw) for lw in layers]
            cfg = binding.make_config(s, S + 16, 64)
            kvd = s.n_kv_heads * s.head_dim
            n_pages = (S + 16 + 63) // 64
            kc = torch.randn((n_pages, 64, kvd), device="cuda").to(torch.bfloat16)
            vc = torch.randn((n_pages, 64, kvd), device="cuda").to(torch.bfloat16)
            pt = torch.arange(n_pages, dtype=torch.int32, device="cuda")
            sc = binding.KernelScratch(cfg)
            h0 = torch.randn((w, s.d_model), device="cuda")
            h = h0.clone()
            for i in range(3):
                binding.k_layer(cfg, lws[i % n_copies], h, kc, vc, pt, S, sc)
            torch.cuda.synchronize()
            times = []
            for i in range(args.iters):
                h.copy_(h0)
                e0, e1 = ev(), ev()
                e0.record()
                binding.k_layer(cfg, lws[i % n_copies], h, kc, vc, pt, S, sc)
                e1.record()
                e1.synchronize()
                times.append(e0.elapsed_time(e1) * 1e3)
            us = statistics.median(times)
            nbytes = inputs.weight_bytes(s)["layer"] + (S + 2 * w) * kv_bytes_per_pos(s)
            row = {"w": w, "S": S, "us": us, "us_min": min(times), "bytes": nbytes, "gbs": nbytes / us / 1e3,
                   "frac": nbytes / us / 1e3 / peak, "frac_of_nominal_8TBs": nbytes / us / 1e3 / NOMINAL_HBM_GBS}
            if not args.no_chained:
                # steady state: n_chain distinct layers (own weights, own K/V cache) back to back in ONE launch sequence
                # inside one event bracket, with the rotation-angle table a context would have: every kernel overlaps
                # its predecessor's tail and requests its first weight tiles early, as inside sb_generate
                if chain_layers is None:
                    chain_layers = [inputs.make_weights(s, 200 + i, device="cuda")["layers"][0] for i in range(n_chain)]
                kcs = [kc] + [torch.randn((n_pages, 64, kvd), device="cuda").to(torch.bfloat16) for _ in range(n_chain - 1)]
                vcs = [vc] + [torch.randn((n_pages, 64, kvd), device="cuda").to(torch.bfloat16) for _ in range(n_chain - 1)]
                chain = binding.LayerChain(chain_layers, kcs, vcs)
                tab = binding.k_rope_table(cfg)
                for _ in range(2):
                    h.copy_(h0)
                    binding.k_layer_chain(cfg, chain, h, pt, S, sc, tab)
                torch.cuda.synchronize()
                ctimes = []
                for i in range(max(args.iters // 4, 5)):
                    h.copy_(h0)
                    e0, e1 = ev(), ev()
                    e0.record()
                    binding.k_layer_chain(cfg, chain, h, pt, S, sc, tab)
                    e1.record()
                    e1.synchronize()
                    ctimes.append(e0.elapsed_time(e1) * 1e3 / n_chain)
                cus = statistics.median(ctimes)
                row.update({"chained_us": cus, "chained_us_min": min(ctimes), "chained_gbs": nbytes / cus / 1e3,
                            "chained_frac": nbytes / cus / 1e3 / peak, "chained_layers": n_chain})
                del kcs, vcs, chain
            out["layer"].append(row)
    del chain_layers
    del layers
    for V in (32000, 128256):
        for m in (1, 4, 8):
            name = f"exit:m={m}:V={V}"
            if not want(name):
                continue
            sh = inputs.scaled(s, vocab=V)
            cfg = binding.make_config(sh, 64, 64)
            copies = 4 if V == 32000 else 2
            heads = [(torch.randn((V, sh.d_model), device="cuda") * 0.08).to(torch.bfloat16) for _ in range(copies)]
            gain = torch.ones(sh.d_model, device="cuda", dtype=torch.bfloat16)
            sc = binding.KernelScratch(cfg)
            h = torch.randn((m, sh.d_model), device="cuda")
            for i in range(3):
                binding.k_exit_confidence(cfg, h, gain, heads[i % copies], 1.4, sc)
            torch.cuda.synchronize()
            times = []
            for i in range(args.iters):
                e0, e1 = ev(), ev()
                e0.record()
                binding.k_exit_confidence(cfg, h, gain, heads[i % copies], 1.0 + 0.2 * (i % 6), sc)
                e1.record()
                e1.synchronize()
                times.append(e0.elapsed_time(e1) * 1e3)
            us = statistics.median(times)
            nbytes = V * sh.d_model * 2
            row = {"m": m, "V": V, "us": us, "us_min": min(times), "bytes": nbytes, "gbs": nbytes / us / 1e3,
                   "frac": nbytes / us / 1e3 / peak, "frac_of_nominal_8TBs": nbytes / us / 1e3 / NOMINAL_HBM_GBS,
                   "note": "the whole stateless call: the RMSNorm launch and the exit kernel, starting cold"}
            if not args.no_chained:
                # steady state: 8 calls over rotating heads inside one event bracket (each kernel overlaps its predecessor)
                ctimes = []
                for i in range(max(args.iters // 4, 5)):
                    e0, e1 = ev(), ev()
                    e0.record()
                    for k in range(8):
                        binding.k_exit_confidence(cfg, h, gain, heads[(i + k) % copies], 1.0 + 0.2 * (k % 6), sc)
                    e1.record()
                    e1.synchronize()
                    ctimes.append(e0.elapsed_time(e1) * 1e3 / 8)
                cus = statistics.median(ctimes)
                row.update({"chained_us": cus, "chained_us_min": min(ctimes), "chained_gbs": nbytes / cus / 1e3,
                            "chained_frac": nbytes / cus / 1e3 / peak, "chained_calls": 8})
            out["exit"].append(row)
            del heads
    # sampling kernel (decoding strategies of Section 4.3): latency of one launch on m rows of L2-resident logits;
    # not a bandwidth-bound kernel (one CTA per row, fp64 exponentials), reported in microseconds only
    for V in (32000, 128256):
        for m, top_p in ((1, 1.0), (8, 1.0), (1, 0.9), (8, 0.9)):
            name = f"sample:m={m}:V={V}:top_p={top_p}"
            if not want(name):
                continue
            z = torch.randn((m, V), device="cuda") * 2.5
            for i in range(3):
                binding.k_sample(z, 1.0, 1, i, top_p=top_p)
            torch.cuda.synchronize()
            times = []
            for i in range(args.iters):
                e0, e1 = ev(), ev()
                e0.record()
                for k in range(8):   # 8 calls per timing: the queue hides the host's issue time if the kernels are longer
                    binding.k_sample(z, 1.0, 1, 64 * i + 8 * k, top_p=top_p)
                e1.record()
                e1.synchronize()
                times.append(e0.elapsed_time(e1) * 1e3 / 8)
            out.setdefault("sample", []).append({"m": m, "V": V, "top_p": top_p, "us": statistics.median(times),
                                                 "us_min": min(times)})
    print(json.dumps(out), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="7b", choices=sorted(inputs.RUNS))
    ap.add_argument("--n-gen", type=int, default=None, help="override the number of generated tokens")
    ap.add_argument("--n-prompt", type=int, default=None, help="override the prompt length (profiling small cases)")
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip the legs that run the CPU oracle (cpu_baseline, oracle_check)")
    ap.add_argument("--no-damped", action="store_true", help="skip the extra workloads of the default run (7b-damped, l3-8b, 13b)")
    ap.add_argument("--no-other-shapes", action="store_true", help="skip the l3-8b and 13b measurements of the default run")
    ap.add_argument("--oracle-check-tokens", type=int, default=96,
                    help="tokens of the short-prompt generation the oracle checks teacher-forced (0 = skip)")
    ap.add_argument("--micro", action="store_true", help="kernel micro-benchmarks instead of the generation benchmark")
    ap.add_argument("--sweep", action="store_true", help="hyper-parameter study on --workload (one JSON line)")
    ap.add_argument("--sweep-short", action="store_true", help="--sweep at no more than 256 + 256 tokens")
    ap.add_argument("--depths", default=None, help="--sweep: comma list of d_max values (default 1,2,4,6,8,10,12 below the layer count)")
    ap.add_argument("--widths", default=None, help="--sweep: comma list of w_max values (default 2,4,8)")
    ap.add_argument("--no-strategies", action="store_true", help="--sweep: skip the sampling-strategy rows")
    ap.add_argument("--micro-case", default="", help="comma list, e.g. layer:w=4:S=512,exit:m=1:V=32000 (default: all)")
    ap.add_argument("--iters", type=int, default=40)
    ap.add_argument("--no-chained", action="store_true", help="--micro: isolated calls only (skip the chained steady-state mode)")
    ap.add_argument("--tune", action="append", default=[], metavar="KEY=VALUE",
                    help="library option set before the run (sb_set_default_option), e.g. 6=10; for tuning sweeps")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    run = inputs.RUNS[args.workload]
    if args.n_gen or args.n_prompt:
        run = inputs.Run(run.shape, args.n_prompt or run.n_prompt, args.n_gen or run.n_gen, run.d_max, run.w_max, run.tau,
                         run.threshold, run.seed, run.damp_rho)
    if args.tune and args.impl == "ours":
        from paper_2604_12247_b200 import binding, build
        build.build()
        for kv in args.tune:
            k, v = kv.split("=")
            assert binding.lib().sb_set_default_option(int(k), int(v)) == 0, kv
    if args.sweep:
        sweep_arm(args, run)
    elif args.micro:
        micro_arm(args)
    elif args.impl == "reference":
        reference_arm(args, run)
    else:
        product_arm(args, run)


if __name__ == "__main__":
    main()
