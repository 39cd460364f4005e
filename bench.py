#!/usr/bin/env python
"""Benchmark of the SpecDec draft -> verify -> commit path on B200.

One step = one call of specdec_generate (encode + every draft/verify/commit round
until the sequences finish) on one batch of the translation-shaped workload
(Transformer-base verifier 6+6, drafter 12+2, d=512, vocab 32768, k=25, beta=3,
tau=1.0; sources of 20..40 Zipf ids at batch 1).  The default run also carries the
metric's second half in the same line: `roofline` = one verify step at (batch 1,
k = 25, 64 committed tokens) against the HBM roofline, and `batch128` = tokens/s
on the padded batch of 128 (sources of 10..80 ids) with its verify step against
the bf16 tensor roofline.  The timed region repeats the K-step stream until it is
at least two seconds long.  Random-init models almost never
agree, so the acceptance pattern of the paper's regime is imposed through the
library's scripted-draft hook: the drafter runs in full, then its output is
replaced by the verifier's own greedy continuation with a rejected token every
Geometric(mean 6) positions.  The unscripted run is reported beside it.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--batch B] [--impl reference]

Prints ONE JSON line.  `--impl reference` times the CPU oracle instead.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2203_16487_b200 import replicas, workloads as W  # noqa: E402

K_BLOCK, BETA, TAU = 25, 3, 1.0
GEO_MEAN = 6.0


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return float(d["hbm_gbs"]), float(d["bf16_tflops"]), "measured"
    return 6650.0, 1590.0, "fallback"


def workload(batch: int):
    """Sentences of the step stream: config 2 (batch 1) or config 3 (padded batches)."""
    if batch == 1:
        wl = W.config2_translation()
        name = "config2_translation_b1"
    else:
        wl = W.config3_batched(128)
        name = f"config3_batched_b{batch}"
    return wl, name


def config_of(name: str, batch: int, world: int) -> dict:
    return {"workload": name, "batch": batch, "k": K_BLOCK, "beta": BETA, "tau": TAU,
            "acceptance": f"scripted: greedy continuation, rejection every Geometric(mean {GEO_MEAN:g}) positions",
            "l2": "each step streams 248 MB of bf16 weights (both models) > 126 MB L2; no explicit flush",
            "parallelism": f"replicas x{world}"}


def make_script(greedy: np.ndarray, n: int, rng: np.random.Generator, vocab: int, width: int) -> np.ndarray:
    """Greedy continuation with a token the verifier rejects every Geometric(mean 6) positions."""
    s = np.full(width, -1, np.int32)
    s[:n] = greedy[:n]
    p = int(rng.geometric(1.0 / GEO_MEAN)) - 1
    while p < width:
        bad = int(rng.integers(W.N_SPECIAL, vocab))
        if p < n and bad == s[p]:
            bad = W.N_SPECIAL + (bad + 1 - W.N_SPECIAL) % (vocab - W.N_SPECIAL)
        s[p] = bad
        p += int(rng.geometric(1.0 / GEO_MEAN))
    return s


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons during the timed region."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "200"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=lambda: [self.lines.append(l) for l in self.proc.stdout], daemon=True)
            self.t.start()
        except Exception:
            self.proc = None

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.25)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for l in self.lines:
            f = [x.strip() for x in l.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for nme, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(nme)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------------------ oracle arm
def oracle_models(wl):
    from oracle import specdec_oracle as O
    wv = W.make_weights(wl.verifier, wl.seed_verifier, True)
    wd = W.make_weights(wl.drafter, wl.seed_drafter, True)
    return O, O.model_from(wl.verifier, wv), O.model_from(wl.drafter, wd)


def oracle_step(O, mv, md, wl, idx: int, rng):
    """Untimed: the oracle's own greedy output -> script.  Timed: scripted SpecDec on one sentence."""
    src, mt = wl.src[idx], wl.max_tgt[idx]
    g = np.array(O.greedy_decode(mv, src, mt, W.BOS_ID, W.EOS_ID), np.int32)
    script = make_script(g, len(g), rng, wl.verifier.vocab, mt + K_BLOCK)
    t0 = time.perf_counter()
    out, st = O.specdec_generate(mv, md, src, mt, K_BLOCK, BETA, TAU, W.BOS_ID, W.EOS_ID, W.MASK_ID, script=script)
    return len(out), time.perf_counter() - t0, st


def cores_used() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 0) for p in threadpool_info() if p.get("user_api") == "blas"]
        if n:
            return int(max(n))
    except Exception:
        pass
    return os.cpu_count() or 1


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl, name = workload(1)
    O, mv, md = oracle_models(wl)
    rng = np.random.default_rng(7)
    for i in range(args.warmup):
        oracle_step(O, mv, md, wl, i % len(wl.src), rng)
    toks, secs = 0, 0.0
    for i in range(args.steps):
        n, t, _ = oracle_step(O, mv, md, wl, (args.warmup + i) % len(wl.src), rng)
        toks += n; secs += t
    v = toks / secs
    sample = f"{args.steps} sentences of {name}, batch 1, scripted acceptance (geometric mean {GEO_MEAN:g})"
    print(json.dumps({
        "impl": "reference", "metric": "generated tokens/s", "value": v, "unit": "tokens/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * secs / max(args.steps, 1),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": config_of(name, 1, 1),
        "cpu_baseline": {"value": v, "unit": "tokens/s", "cores": cores_used(), "kind": "oracle", "sample": sample},
        "e2e": {"value": v, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


# ------------------------------------------------------------------------------------------ CUDA arm
MIN_TIMED_MS = 2000.0          # the timed region repeats the K-step stream until it is at least this long


def tokens_leg(torch, binding, B: int, K_: int, W_: int, rank: int, world: int, local: int, opts, poll_lag, want_breakdown: bool):
    """Generated tokens/s of specdec_generate on the batch-B workload: device-resident inputs, host buffers (e2e),
    the unscripted drafter, greedy autoregressive decoding (k = 0) and the per-phase split."""
    dev = torch.device("cuda", local)
    wl, name = workload(B)
    wv = W.make_weights(wl.verifier, wl.seed_verifier, True)
    wd = W.make_weights(wl.drafter, wl.seed_drafter, True)
    max_src = max(len(s) for s in wl.src)
    max_tgt = max(wl.max_tgt)
    sd = binding.SpecDec(wl.verifier, wv, wl.drafter, wd, k_max=K_BLOCK, max_batch=B, max_src=max_src,
                         max_tgt=max_tgt, bf16=True, device=f"cuda:{local}")
    del wv, wd
    if poll_lag is not None:
        sd.set_option("poll_lag", poll_lag)
    for kv in opts:
        opt_name, _, val = kv.partition("=")
        sd.set_option(opt_name, int(val))

    # the step stream: rank r takes batches r, r + world, ... (replicas; no data-path collective)
    n_total = W_ + K_
    n_batches = max(len(wl.src) // B, 1)

    def batch_of(step):
        i = replicas.batch_index(step, rank, world, n_batches) * B
        srcs, mts = wl.src[i:i + B], wl.max_tgt[i:i + B]
        src, lens = W.pad_batch(srcs, max_src)
        return src, lens, np.asarray(mts, np.int32)

    # untimed set-up: greedy outputs of the verifier (strict rule, lossless) -> scripts
    rng = np.random.default_rng(7 + rank)
    steps_in = []
    for s in range(n_total):
        src, lens, mts = batch_of(s)
        sd.set_draft_script(None)
        out, n, _ = sd.generate(src, lens, mts, K_BLOCK, 1, 0.0)
        out, n = out.cpu().numpy(), n.cpu().numpy()
        script = np.stack([make_script(out[b], int(n[b]), rng, wl.verifier.vocab, max_tgt + K_BLOCK) for b in range(B)])
        dv = (torch.from_numpy(src).to(dev), torch.from_numpy(lens).to(dev), torch.from_numpy(mts).to(dev))
        hv = tuple(torch.from_numpy(a).pin_memory() for a in (src, lens, mts))
        steps_in.append((dv, hv, script, out, n))
    ho = torch.zeros((B, max_tgt), dtype=torch.int32).pin_memory()
    hn = torch.zeros(B, dtype=torch.int32).pin_memory()

    def barrier():
        import torch.distributed as dist
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    diverged = [0]

    def one_pass(first, count, host, scripted, k, check):
        toks, ms, stats = 0, 0.0, []
        for s in range(first, first + count):
            dv, hv, script, ref_out, ref_n = steps_in[s]
            sd.set_draft_script(script if scripted else None)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            if host:
                e0.record()
                st = sd.generate_host(hv[0], hv[1], hv[2], ho, hn, k, BETA, TAU, want_stats=True)
                e1.record()
                torch.cuda.synchronize()
                n, out = hn.numpy(), ho.numpy()
            else:
                e0.record()
                o, nn, st = sd.generate(dv[0], dv[1], dv[2], k, BETA, TAU)
                e1.record()
                torch.cuda.synchronize()
                n = nn.cpu().numpy()
                out = o.cpu().numpy() if check else None
            ms += e0.elapsed_time(e1)
            toks += int(n.sum())
            stats.append(st)
            if check and scripted:      # greedy drafts are always accepted: the result must be the greedy output
                for b in range(B):
                    if out[b, :n[b]].tolist() != ref_out[b, :ref_n[b]].tolist():
                        diverged[0] += 1
        return toks, ms, stats

    def timed(host=False, scripted=True, k=K_BLOCK, min_ms=None):
        """The K-step stream, repeated until the region is at least min_ms long; returns (tokens, ms, stats, repeats)."""
        toks, ms, stats, reps = 0, 0.0, [], 0
        min_ms = MIN_TIMED_MS if min_ms is None else min_ms
        while reps == 0 or ms < min_ms:
            t, m, st = one_pass(W_, K_, host, scripted, k, check=(reps == 0))
            toks += t; ms += m; stats += st; reps += 1
            if reps >= 400:
                break
        return toks, ms, stats, reps

    one_pass(0, W_, False, True, K_BLOCK, False)                      # warm-up (untimed)
    sampler = ClockSampler(local)
    barrier()
    sampler.start()
    l0 = sd.launch_count()
    toks, ms, stats, reps = timed()
    launches = sd.launch_count() - l0
    barrier()
    clocks = sampler.stop()
    e_toks, e_ms, _, e_reps = timed(host=True)                        # end to end, host buffers
    n_toks, n_ms, n_stats, _ = timed(scripted=False, min_ms=MIN_TIMED_MS / 4)     # unscripted drafter
    one_pass(0, min(W_, 1), False, False, 0, False)                   # the k = 0 graphs are captured here
    a_toks, a_ms, _, _ = timed(scripted=False, k=0, min_ms=MIN_TIMED_MS / 4)      # greedy autoregressive baseline
    ph = None
    if want_breakdown:
        # per-phase times: a pass of its own, because an event after every phase keeps the host from queueing whole
        # iterations ahead (the timed pass above records none)
        sd.set_option("stats_timing", 1)
        _, _, ph_stats = one_pass(W_, K_, False, True, K_BLOCK, False)
        sd.set_option("stats_timing", 0)
        ph = dict({k: sum(s[k] for s in ph_stats) / max(K_, 1) for k in ("ms_encode", "ms_draft", "ms_verify", "ms_commit", "ms_total")},
                  note="separate untimed pass with an event after every phase (option stats_timing): each iteration "
                       "then waits for the host, so ms_total here exceeds ms_per_step")
    sd.close()
    toks_all, ms_max = replicas.reduce_job(toks, ms, dev)
    e_toks_all, e_ms_max = replicas.reduce_job(e_toks, e_ms, dev)
    n_toks_all, n_ms_max = replicas.reduce_job(n_toks, n_ms, dev)
    a_toks_all, a_ms_max = replicas.reduce_job(a_toks, a_ms, dev)
    seq_it = sum(s["seq_iterations"] for s in stats)
    ar = a_toks_all / (a_ms_max * 1e-3)
    leg = {
        "workload": name, "value": toks_all / (ms_max * 1e-3), "unit": "tokens/s",
        "ms_per_step": ms_max / max(K_ * reps, 1), "timed_ms": ms_max, "repeats": reps,
        "e2e": {"value": e_toks_all / (e_ms_max * 1e-3), "unit": "tokens/s",
                "h2d_bytes_per_step": int(B * max_src * 4 + B * 8), "d2h_bytes_per_step": int(B * max_tgt * 4 + B * 4)},
        "gpu_launches": int(launches), "clocks": clocks,
        "tok_per_iteration": {"accepted": sum(s["accepted"] for s in stats) / max(seq_it, 1), "emitted": toks / max(seq_it, 1)},
        "iterations": sum(s["iterations"] for s in stats),
        "scripted_runs_differing_from_greedy": diverged[0],
        "unscripted": {"value": n_toks_all / (n_ms_max * 1e-3), "unit": "tokens/s",
                       "tok_per_iteration": sum(s["emitted"] for s in n_stats) / max(sum(s["seq_iterations"] for s in n_stats), 1)},
        "greedy_ar": {"value": ar, "unit": "tokens/s", "specdec_speedup": toks_all / (ms_max * 1e-3) / ar,
                      "note": "k = 0: the verifier alone, one token per step, same kernels; the paper reports SpecDec at "
                              "about 4.6x greedy (5.1x / 1.1x over beam-5, Table 1) on a P100 with trained models"},
    }
    if ph:
        leg["ms_breakdown"] = ph
    return leg


# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) from ncu captures of the verify microbenchmark, keyed by
# (batch, what): one whole verify step, or the vocabulary kernel alone.  ncu measures every kernel with cold caches, so at
# batch 128 the step figure counts activations that normally stay in L2 (an upper bound); cells never captured are absent.
NCU_TRAFFIC = {(1, "step"): 84391168, (1, "vocabulary"): 33608960, (128, "step"): 817641984, (128, "vocabulary"): 37020000}


def verify_step_roofline(torch, binding, B: int, local: int, opts, reps: int = 50):
    """The metric's second half: one verify step at (B, k = 25, committed prefix 64, source 64), L2 flushed between
    repetitions, against the HBM roofline (weights + K/V once) or the bf16 tensor roofline (batch 128); with the cost
    of each kernel class inside the step (every launch of the class issued twice: the step grows by the class's cost)."""
    from paper_2203_16487_b200 import microbench as MB
    hbm_peak, tc_peak, peak_kind = load_peaks()
    peaks_all = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json"))) if peak_kind == "measured" else {}
    k, j, S = K_BLOCK, 64, 64
    wl = W.config5_microbench(B, S)
    wv = W.make_weights(wl.verifier, wl.seed_verifier, True)
    wd = W.make_weights(wl.drafter, wl.seed_drafter, True)
    sd = binding.SpecDec(wl.verifier, wv, wl.drafter, wd, k_max=k, max_batch=B, max_src=S, max_tgt=j + k + 2, bf16=True,
                         device=f"cuda:{local}")
    del wv, wd
    for kv in opts:
        opt_name, _, val = kv.partition("=")
        sd.set_option(opt_name, int(val))
    flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device=f"cuda:{local}")
    l0 = sd.launch_count()
    us, us_min, mean_a = MB.measure(sd, wl, B, k, j, S, reps, 5, flush)
    n_calls = None
    params, bytes_, flops = MB.algorithmic_work(B, k, j, S, wl.verifier)
    # launches of one step: count them on one extra call
    c0 = sd.launch_count()
    d = torch.zeros((B, k), dtype=torch.int32, device=f"cuda:{local}")
    acc_t = torch.zeros(B, dtype=torch.int32, device=f"cuda:{local}"); bif_t = torch.zeros_like(acc_t)
    sd.verify_raw(d, BETA, TAU, acc_t, bif_t)
    torch.cuda.synchronize()
    launches_per_step = sd.launch_count() - c0
    by_kernel = []
    d_model, V = wl.verifier.d_model, wl.verifier.vocab
    rows = B * (k + 1)
    classes = [(1, "attention (self + cross)", 2 * wl.verifier.dec_layers, B * wl.verifier.dec_layers * (j + k + 1 + S) * 2 * d_model * 2),
               (2, "LayerNorm launches", None, None),
               (4, "layer GEMMs without residual (QKV, cross-Q, FFN1)", 3 * wl.verifier.dec_layers,
                wl.verifier.dec_layers * (3 * d_model * d_model + d_model * d_model + wl.verifier.d_ffn * d_model) * 2),
               (8, "vocabulary projection + row statistics", 1, V * d_model * 2 + rows * d_model * 2)]
    for bit, label, n_launch, cls_bytes in classes:
        sd.set_option("diag_repeat", bit)
        us_c, _, _ = MB.measure(sd, wl, B, k, j, S, max(reps // 2, 10), 3, flush)
        sd.set_option("diag_repeat", 0)
        cost = max(us_c - us, 0.0)
        e = {"class": label, "launches": n_launch, "us_in_step": cost, "share_of_step": cost / us}
        if cls_bytes:
            e["algorithmic_bytes"] = int(cls_bytes)
            e["hbm_frac"] = (cls_bytes / (cost * 1e-6) / 1e9 / hbm_peak) if cost > 0 else None
        if bit == 8:
            e["traffic"] = NCU_TRAFFIC.get((B, "vocabulary"))
        by_kernel.append(e)
    rest = us - sum(e["us_in_step"] for e in by_kernel)
    by_kernel.append({"class": "residual GEMMs (attention out x2, FFN2), embedding, accept scan, the rest", "launches": None,
                      "us_in_step": rest, "share_of_step": rest / us})
    link_us = sd.link_cost(64, 148)
    round_ns = sd.cluster_round(16, 2048, 64)
    sd.close()
    del flush
    hbm_bound = (bytes_ / (hbm_peak * 1e9)) >= (flops / (tc_peak * 1e12))
    if hbm_bound:
        achieved = bytes_ / (us * 1e-6) / 1e9
        roof = {"bound": "hbm", "achieved": achieved, "peak": hbm_peak, "unit": "GB/s", "frac": achieved / hbm_peak}
    else:
        achieved = flops / (us * 1e-6) / 1e12
        roof = {"bound": "tensor", "achieved": achieved, "peak": tc_peak, "unit": "TFLOP/s", "frac": achieved / tc_peak}
        sus = peaks_all.get("bf16_tflops_sustained")
        if sus:
            roof["frac_of_sustained_peak"] = achieved / float(sus)
    roof.update({
        "traffic": NCU_TRAFFIC.get((B, "step")),
        "traffic_note": "one whole step under ncu (every kernel measured with cold caches: activations that stay in L2 in a real step are counted)",
        "kernel": f"verify step (all {launches_per_step} launches): B={B}, k={k}, committed prefix {j}, source {S}, L2 flushed between repetitions",
        "peak_kind": f"of {peak_kind}", "us_per_step_median": us, "us_per_step_min": us_min, "repetitions": reps,
        "launches_per_step": int(launches_per_step), "algorithmic_bytes_per_launch": int(bytes_), "algorithmic_flops_per_launch": flops,
        "roofline_us": max(bytes_ / (hbm_peak * 1e9), flops / (tc_peak * 1e12)) * 1e6, "mean_accepted": mean_a, "by_kernel": by_kernel,
        # the step is a chain of dependent launches: what the chain alone costs, from the library's own probes
        "latency_floor": {"launches_per_step": int(launches_per_step), "us_per_kernel_boundary": link_us,
                          "us": launches_per_step * link_us, "step_over_floor": us / (launches_per_step * link_us),
                          "us_per_16cta_cluster_exchange_of_32KB": round_ns / 1e3,
                          "note": "kernel boundary = one link of a chain of dependent 148-CTA launches (programmatic dependent launch, "
                                  "replayed from a graph); the cluster exchange is what a fused cluster kernel would pay instead of a boundary"},
    })
    return roof


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2203_16487_b200 import binding

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    B = args.batch
    leg = tokens_leg(torch, binding, B, args.steps, args.warmup, rank, world, local, args.opt, args.poll_lag, True)
    line = {
        "metric": "generated tokens/s", "value": leg["value"], "unit": "tokens/s",
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": leg["ms_per_step"],
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": dict(config_of(leg["workload"], B, world), timed_region_ms=leg["timed_ms"],
                       repeats_of_the_step_stream=leg["repeats"]),
    }
    for key in ("e2e", "gpu_launches", "clocks", "tok_per_iteration", "iterations", "scripted_runs_differing_from_greedy",
                "ms_breakdown", "unscripted", "greedy_ar"):
        if key in leg:
            line[key] = leg[key]
    if rank == 0 and not args.no_roofline:
        # the verify step against its roofline (rank 0: a single-GPU measurement)
        line["roofline"] = verify_step_roofline(torch, binding, B, local, args.opt)
    if B == 1 and not args.no_batch128:
        # the metric's batch-128 half, in the same line: tokens/s on the padded-batch workload and the verify step
        # against the tensor roofline
        b128 = tokens_leg(torch, binding, 128, min(args.steps, 6), args.warmup, rank, world, local, args.opt, args.poll_lag, False)
        if rank == 0 and not args.no_roofline:
            b128["roofline"] = verify_step_roofline(torch, binding, 128, local, args.opt, reps=30)
        b128["config"] = config_of(b128.pop("workload"), 128, world)
        line["batch128"] = b128
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        wl1, name1 = workload(1)
        O, mv, md = oracle_models(wl1)
        rng = np.random.default_rng(7)
        n_s, ctoks, csecs = 0, 0, 0.0
        while n_s < 128 and csecs < 15.0:              # a bounded sample: 10-20 s of CPU work
            n, t, _ = oracle_step(O, mv, md, wl1, n_s, rng)
            ctoks += n; csecs += t; n_s += 1
        line["cpu_baseline"] = {"value": ctoks / csecs, "unit": "tokens/s", "cores": cores_used(), "kind": "oracle",
                                "sample": f"first {n_s} sentences of {name1}, batch 1, same scripted acceptance; {csecs:.1f} s"}
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def spawn_replicas(args) -> int:
    """`python bench.py --gpus N` without a launcher: start the N ranks here (one process per GPU, NCCL only for the
    final max / sum) and pass their single JSON line through."""
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=16)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--batch", type=int, default=1)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-batch128", action="store_true", help="skip the batch-128 leg of the default (batch 1) run")
    ap.add_argument("--no-roofline", action="store_true", help="skip the verify-step roofline legs (profiling runs)")
    ap.add_argument("--min-timed-ms", type=float, default=None, help="length of the timed region that the K-step stream is repeated to "
                    "reach (default 2000; 0 = the K steps once, for profiling runs)")
    ap.add_argument("--opt", action="append", default=[], help="experiments: name=value passed to specdec_set_option")
    ap.add_argument("--poll-lag", type=int, default=None, help="experiments: iterations the host runs ahead of the finish counter")
    args = ap.parse_args()
    if args.min_timed_ms is not None:
        global MIN_TIMED_MS
        MIN_TIMED_MS = args.min_timed_ms
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        run_reference(args)
    elif args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        raise SystemExit(spawn_replicas(args))
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
