#!/usr/bin/env python
"""Benchmark of the SpecDec draft -> verify -> commit path on B200.

One step = one call of specdec_generate (encode + every draft/verify/commit round
until the sequences finish) on one batch of the translation-shaped workload
(Transformer-base verifier 6+6, drafter 12+2, d=512, vocab 32768, k=25, beta=3,
tau=1.0; sources of 20..40 Zipf ids; batch 1 by default, --batch 128 for the
padded-batch shape with sources of 10..80 ids).  Random-init models almost never
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
    dev = torch.device("cuda", local)
    hbm_peak, tc_peak, peak_kind = load_peaks()

    B = args.batch
    wl, name = workload(B)
    wv = W.make_weights(wl.verifier, wl.seed_verifier, True)
    wd = W.make_weights(wl.drafter, wl.seed_drafter, True)
    max_src = max(len(s) for s in wl.src)
    max_tgt = max(wl.max_tgt)
    sd = binding.SpecDec(wl.verifier, wv, wl.drafter, wd, k_max=K_BLOCK, max_batch=B, max_src=max_src,
                         max_tgt=max_tgt, bf16=True, device=f"cuda:{local}")
    del wv, wd
    if args.poll_lag is not None:
        sd.set_option("poll_lag", args.poll_lag)
    for kv in args.opt:
        name, _, val = kv.partition("=")
        sd.set_option(name, int(val))

    # the step stream: rank r takes batches r, r + world, ... (replicas; no data-path collective)
    n_total = args.warmup + args.steps
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
        steps_in.append((src, lens, mts, script, out, n))

    def dev_inputs(s):
        src, lens, mts, script, _, _ = steps_in[s]
        return (torch.from_numpy(src).to(dev), torch.from_numpy(lens).to(dev), torch.from_numpy(mts).to(dev), script)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    diverged = [0]

    def timed_pass(first, count, host: bool, scripted: bool = True, k: int = K_BLOCK):
        """Runs steps [first, first+count); returns (tokens, ms, stats list)."""
        toks, ms, stats = 0, 0.0, []
        for s in range(first, first + count):
            src, lens, mts, script, ref_out, ref_n = steps_in[s]
            sd.set_draft_script(script if scripted else None)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            if host:
                hs, hl, hm = (torch.from_numpy(a).pin_memory() for a in (src, lens, mts))
                ho = torch.zeros((B, max_tgt), dtype=torch.int32).pin_memory()
                hn = torch.zeros(B, dtype=torch.int32).pin_memory()
                torch.cuda.synchronize()
                e0.record()
                st = sd.generate_host(hs, hl, hm, ho, hn, k, BETA, TAU, want_stats=True)
                e1.record()
                n = hn.numpy()
                out = ho.numpy()
            else:
                dsrc, dlen, dmt, _ = dev_inputs(s)
                torch.cuda.synchronize()
                e0.record()
                o, nn, st = sd.generate(dsrc, dlen, dmt, k, BETA, TAU)
                e1.record()
                out, n = o.cpu().numpy(), nn.cpu().numpy()
            torch.cuda.synchronize()
            ms += e0.elapsed_time(e1)
            toks += int(n.sum())
            stats.append(st)
            if scripted:       # greedy drafts are always accepted: the result should be the greedy output
                for b in range(B):
                    if out[b, :n[b]].tolist() != ref_out[b, :ref_n[b]].tolist():
                        diverged[0] += 1
        return toks, ms, stats

    W_, K_ = args.warmup, args.steps
    timed_pass(0, W_, host=False)                                   # warm-up (untimed)
    sampler = ClockSampler(local)
    barrier()
    sampler.start()
    l0 = sd.launch_count()
    toks, ms, stats = timed_pass(W_, K_, host=False)
    launches = sd.launch_count() - l0
    barrier()
    clocks = sampler.stop()
    e_toks, e_ms, _ = timed_pass(W_, K_, host=True)                 # end to end, host buffers
    n_toks, n_ms, n_stats = timed_pass(W_, K_, host=False, scripted=False)   # unscripted drafter
    timed_pass(0, min(W_, 1), host=False, scripted=False, k=0)               # one untimed step: the k = 0 graphs are captured here
    a_toks, a_ms, _ = timed_pass(W_, K_, host=False, scripted=False, k=0)    # greedy autoregressive baseline (verifier alone)
    # dominant kernel: the vocabulary projection with fused row statistics
    sd.set_option("profile", 1)
    timed_pass(W_, K_, host=False)
    vocab_ms, vocab_n = sd.profile_read()
    sd.set_option("profile", 0)
    # per-phase times: a pass of its own, because an event after every phase keeps the host from queueing whole
    # iterations ahead (the timed pass above records none)
    sd.set_option("stats_timing", 1)
    _, _, ph_stats = timed_pass(W_, K_, host=False)
    sd.set_option("stats_timing", 0)

    toks_all, ms_max = replicas.reduce_job(toks, ms, dev)
    e_toks_all, e_ms_max = replicas.reduce_job(e_toks, e_ms, dev)
    n_toks_all, n_ms_max = replicas.reduce_job(n_toks, n_ms, dev)
    a_toks_all, a_ms_max = replicas.reduce_job(a_toks, a_ms, dev)

    it = sum(s["iterations"] for s in stats)
    seq_it = sum(s["seq_iterations"] for s in stats)
    acc = sum(s["accepted"] for s in stats)
    d, V = wl.verifier.d_model, wl.verifier.vocab
    rows = B * (K_BLOCK + 1)
    # column halves per row that the kernel writes 16-byte partial statistics for: one 224-wide tile per SM up to
    # 128 rows, 128-wide tiles up to 512 rows, 256-wide above (the library's tile rule for this kernel)
    tile = 224 if rows <= 128 else (128 if rows <= 512 else 256)
    n_part = 2 * ((V + tile - 1) // tile)
    alg_bytes = V * d * 2 + rows * d * 2 + rows * n_part * 16 + rows * 8
    per_launch_ms = vocab_ms / max(vocab_n, 1)
    achieved = alg_bytes / (per_launch_ms * 1e-3) / 1e9 if per_launch_ms > 0 else 0.0
    flops = 2.0 * rows * d * V
    tf = flops / (per_launch_ms * 1e-3) / 1e12 if per_launch_ms > 0 else 0.0
    bound_hbm = (alg_bytes / (hbm_peak * 1e9)) >= (flops / (tc_peak * 1e12))
    roof = ({"bound": "hbm", "achieved": achieved, "peak": hbm_peak, "unit": "GB/s", "frac": achieved / hbm_peak}
            if bound_hbm else
            {"bound": "tensor", "achieved": tf, "peak": tc_peak, "unit": "TFLOP/s", "frac": tf / tc_peak})
    # DRAM bytes of one launch from the ncu capture summarised in profiles/vocab_stats_kernel_b1_ncu.md
    # (dram__bytes_read.sum + dram__bytes_write.sum at 26 rows); none was taken at other row counts
    traffic = 33608960 if B == 1 else None
    roof.update({"traffic": traffic, "kernel": "k_gemm_tc<EPI_STATS> (vocabulary projection + row statistics, verify step)",
                 "peak_kind": f"of {peak_kind}", "launches_timed": int(vocab_n), "us_per_launch": per_launch_ms * 1e3,
                 "algorithmic_bytes_per_launch": alg_bytes})

    line = {
        "metric": "generated tokens/s", "value": toks_all / (ms_max * 1e-3), "unit": "tokens/s",
        "n_gpus": world, "steps": K_, "warmup": W_, "ms_per_step": ms_max / max(K_, 1),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": config_of(name, B, world),
        "e2e": {"value": e_toks_all / (e_ms_max * 1e-3), "unit": "tokens/s",
                "h2d_bytes_per_step": int(B * max_src * 4 + B * 8), "d2h_bytes_per_step": int(B * max_tgt * 4 + B * 4)},
        "gpu_launches": int(launches),
        "clocks": clocks,
        "roofline": roof,
        "tok_per_iteration": {"accepted": acc / max(seq_it, 1), "emitted": toks / max(seq_it, 1)},
        "iterations": it,
        "scripted_runs_differing_from_greedy": diverged[0],
        "ms_breakdown": dict({k: sum(s[k] for s in ph_stats) / max(K_, 1) for k in ("ms_encode", "ms_draft", "ms_verify", "ms_commit", "ms_total")},
                             note="separate untimed pass with an event after every phase (option stats_timing): each iteration "
                                  "then waits for the host, so ms_total here exceeds ms_per_step"),
        "unscripted": {"value": n_toks_all / (n_ms_max * 1e-3), "unit": "tokens/s",
                       "tok_per_iteration": sum(s["emitted"] for s in n_stats) / max(sum(s["seq_iterations"] for s in n_stats), 1)},
    }

    ar = a_toks_all / (a_ms_max * 1e-3)
    line["greedy_ar"] = {"value": ar, "unit": "tokens/s", "specdec_speedup": line["value"] / ar,
                         "note": "k = 0: the verifier alone, one token per step, same kernels; the paper reports SpecDec at "
                                 "about 4.6x greedy (5.1x / 1.1x over beam-5, Table 1) on a P100 with trained models"}
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
    sd.close()
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=16)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--batch", type=int, default=1)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--opt", action="append", default=[], help="experiments: name=value passed to specdec_set_option")
    ap.add_argument("--poll-lag", type=int, default=None, help="experiments: iterations the host runs ahead of the finish counter")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
