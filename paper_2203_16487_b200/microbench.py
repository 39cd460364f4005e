"""Verify-step microbenchmark (Transformer-base verifier decoder, bf16): times specdec_verify alone.

  python -m paper_2203_16487_b200.microbench --batch 1 --k 25 --prefix 64 [--reps 50] [--no-flush] [--draft]

A session is encoded on sources of 64 Zipf ids, a committed prefix of `prefix`
tokens is built through verify + commit(keep, next), and the verify step is
then repeated on a fixed draft block (the verifier's own greedy continuation
with one substitution at a Geometric(mean 6) position).  Each repetition is
timed with CUDA events on the launching stream; unless --no-flush is given a
256 MiB buffer is rewritten between repetitions so the weights come from HBM.
Prints one JSON line with the median time, the algorithmic bytes / flops of the
step and the achieved fraction of the measured HBM and bf16 peaks.
--draft times specdec_draft instead.
"""
from __future__ import annotations

import argparse
import json
import os

import numpy as np
import torch

from . import binding, workloads as W


def algorithmic_work(B: int, k: int, j: int, S: int, dims: W.ModelDims):
    """Bytes that must move and flops that must run for one verify step."""
    d, F, V, L = dims.d_model, dims.d_ffn, dims.vocab, dims.dec_layers
    per_layer = 3 * d * d + 3 * d + d * d + d + d * d + d + d * d + d + 2 * F * d + F + d + 6 * d   # self qkv/o, cross q/o, ffn, 3 LN
    params = L * per_layer + V * d + 2 * d
    M = B * (k + 1)
    kv_read = B * L * (j + S) * 2 * d * 2
    kv_new = B * L * (k + 1) * 2 * d * 2 * 2
    bytes_ = params * 2 + kv_read + kv_new + M * d * 2 + B * 8
    flops = 2.0 * M * (L * (4 * d * d + 2 * d * d + 2 * F * d) + V * d) + 4.0 * B * L * (k + 1) * d * ((j + k + 1) + S)
    return params, bytes_, flops


def measure(sd, wl, B, k, j, S, reps, warmup, flush, draft=False):
    """Builds a committed prefix of j tokens, a draft block with scripted rejections, and times the step."""
    src, lens = W.pad_batch(wl.src)
    sd.encode(src, lens, None)
    prefix, rej = W.config5_prefix_and_rejections(B, j)
    prefix = np.stack(prefix) if j > 0 else np.zeros((B, 0), np.int32)
    kb = min(k, 25)
    done = 0
    while done < j:            # verify a block of prefix tokens, keep c of them plus the next one
        c = min(kb, j - done - 1)
        block = np.zeros((B, kb), np.int32)
        block[:, :c] = prefix[:, done:done + c]
        sd.verify(block, 1, 0.0)
        sd.commit(np.full(B, c, np.int32), prefix[:, done + c])
        done += c + 1
    out, n, _ = sd.output()
    assert int(n.min()) == j and int(n.max()) == j
    # draft block: the verifier's greedy continuation from that prefix, one substitution per sequence
    drafts = np.zeros((B, k), np.int32)
    for i in range(k + 1):
        acc, bif = sd.verify(drafts, 1, 0.0)
        a, t = acc.cpu().numpy(), bif.cpu().numpy()
        if int(a.min()) >= k:
            break
        for b in range(B):
            if a[b] < k:
                drafts[b, a[b]] = t[b]
    for b in range(B):
        if rej[b] <= k:
            drafts[b, rej[b] - 1] = (drafts[b, rej[b] - 1] + 17) % wl.verifier.vocab
    d_drafts = torch.from_numpy(drafts).cuda()
    acc_t = torch.zeros(B, dtype=torch.int32, device="cuda")
    bif_t = torch.zeros(B, dtype=torch.int32, device="cuda")
    sd.verify_raw(d_drafts, 3, 1.0, acc_t, bif_t)
    mean_a = float(acc_t.float().mean())
    times = []
    for r in range(warmup + reps):
        if flush is not None:
            flush.fill_(r & 0xff)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        if draft:
            sd.draft(k)
        else:
            sd.verify_raw(d_drafts, 3, 1.0, acc_t, bif_t)
        e1.record()
        torch.cuda.synchronize()
        if r >= warmup:
            times.append(e0.elapsed_time(e1) * 1e3)
    return float(np.median(times)), float(np.min(times)), mean_a


def measure_ttft(sd, wl, k, reps, warmup, flush):
    """Time to the first committed tokens: specdec_encode (both encoders, cross K/V of every decoder layer), then one
    draft -> verify -> commit iteration.  Returns median microseconds of (encode, encode + first iteration)."""
    src, lens = W.pad_batch(wl.src)
    d_src = torch.from_numpy(src).cuda(); d_len = torch.from_numpy(lens).cuda()
    enc, tot = [], []
    for r in range(warmup + reps):
        if flush is not None:
            flush.fill_(r & 0xff)
        e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
        e0.record()
        sd.encode(d_src, d_len, None)
        e1.record()
        d = sd.draft(k)
        sd.verify(d, 3, 1.0)
        sd.commit(None, None)
        e2.record()
        torch.cuda.synchronize()
        if r >= warmup:
            enc.append(e0.elapsed_time(e1) * 1e3); tot.append(e0.elapsed_time(e2) * 1e3)
    return float(np.median(enc)), float(np.median(tot))


def peaks():
    p = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return d["hbm_gbs"], d["bf16_tflops"], "measured"
    return 6650.0, 1590.0, "fallback"


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--batch", type=int, default=1)
    ap.add_argument("--k", type=int, default=25)
    ap.add_argument("--prefix", type=int, default=64)
    ap.add_argument("--src-len", type=int, default=64)
    ap.add_argument("--reps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--no-flush", action="store_true")
    ap.add_argument("--draft", action="store_true")
    ap.add_argument("--gemm", type=int, default=1)
    ap.add_argument("--graphs", type=int, default=1)
    ap.add_argument("--tc-bn", type=int, default=0, help="force the N tile of the tensor-core GEMM (experiments)")
    ap.add_argument("--model", choices=["base", "bart"], default="base",
                    help="Transformer-base pair (default) or the BART-base-shaped pair (GELU, learned positions)")
    ap.add_argument("--opt", action="append", default=[], help="library option name=value (repeatable; experiments)")
    ap.add_argument("--grid", action="store_true", help="the whole k x prefix x batch grid of the verify microbench")
    ap.add_argument("--ttft", action="store_true", help="time to the first tokens on summarisation-shaped inputs (batch 8, "
                    "sources of 300-512 ids) or, with --translation, on one translation-shaped sentence")
    ap.add_argument("--translation", action="store_true")
    ap.add_argument("--mma-rate", action="store_true", help="clocks per tcgen05.mma with operands resident in shared memory, "
                    "and the cost of a kernel boundary (library diagnostics)")
    args = ap.parse_args()
    if args.mma_rate:
        wl = W.config1_tiny()
        dims = W.ModelDims(128, 2, 512, 32768, 1, 1, 64)       # (an 8 MB embedding table: the source of the background stream)
        wv, wd = W.make_weights(dims, 1, True), W.make_weights(dims, 2, True)
        sd = binding.SpecDec(dims, wv, dims, wd, k_max=8, max_batch=32, max_src=16, max_tgt=16, bf16=True)
        rows = []
        loaded = []       # the same MMAs with what a main loop adds: a commit per k-block, a producer's writes into shared memory
        for bn, two in ((128, False), (256, False), (256, True)):
            for bg in (0, 1, 2, 3, 4, 6):
                issue, done, bpc = sd.mma_rate_bg(bn, two, 8192, bg, 1)
                loaded.append({"M": 256 if two else 128, "N": bn, "two_sm": two, "commit_per_k_block": True, "bulk_copies_in_flight": bg,
                               "completion_clocks": done, "landed_bytes_per_clock": bpc, "landed_GBs_per_sm": bpc * 1.965})
        for bn, two in ((64, False), (128, False), (256, False), (128, True), (256, True)):
            issue, done = sd.mma_rate(bn, two, 8192)
            m = 256 if two else 128
            ideal = m * bn * 16 * 2 / (2250e12 / 148 / 1.965e9) / (2 if two else 1)     # clocks per MMA at the nominal dense bf16 rate of the SMs involved
            rows.append({"M": m, "N": bn, "two_sm": two, "issue_clocks": issue, "completion_clocks": done, "nominal_clocks": ideal,
                         "fraction_of_nominal": ideal / done})
        rounds = {f"{cs} CTAs, {b} B per peer": sd.cluster_round(cs, b, 64) for cs in (8, 16) for b in (0, 2048, 4096)}
        print(json.dumps({"step": "mma_rate", "rows": rows, "with_commits_and_background_stream": loaded, "link_cost_us": {g: sd.link_cost(64, g) for g in (8, 148, 592)},
                          "cluster_round_ns": rounds}))
        sd.close()
        return
    if args.ttft:
        wl = W.config2_translation(1) if args.translation else W.config4_summarization()
        wv = W.make_weights(wl.verifier, wl.seed_verifier, True)
        wd = W.make_weights(wl.drafter, wl.seed_drafter, True)
        sd = binding.SpecDec(wl.verifier, wv, wl.drafter, wd, k_max=25, max_batch=len(wl.src), max_src=max(len(s) for s in wl.src),
                             max_tgt=max(wl.max_tgt), bf16=True)
        for o in args.opt:
            sd.set_option(o.split("=")[0], int(o.split("=")[1]))
        flush = None if args.no_flush else torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device="cuda")
        enc, tot = measure_ttft(sd, wl, 25, args.reps, args.warmup, flush)
        print(json.dumps({"step": "ttft", "workload": wl.name, "batch": len(wl.src), "source_lens": [len(s) for s in wl.src],
                          "us_encode_median": enc, "us_to_first_tokens_median": tot, "l2_flush": flush is not None,
                          "link_cost_us": {g: sd.link_cost(64, g) for g in (8, 148, 592)}}))
        sd.close()
        return
    S = args.src_len
    hbm, tc, kind = peaks()
    flush = None if args.no_flush else torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device="cuda")
    batches = [1, 8, 64, 128] if args.grid else [args.batch]
    ks = [5, 10, 25, 50] if args.grid else [args.k]
    prefixes = [0, 64, 256] if args.grid else [args.prefix]
    if args.grid:
        print(f"| B | k | prefix | us/step | MB | GFLOP | HBM GB/s | % of {kind} HBM | TFLOP/s | % of {kind} bf16 | mean accepted |")
        print("|---|---|---|---|---|---|---|---|---|---|---|")
    for B in batches:
        wl = W.config5_microbench(B, S)
        bart = args.model == "bart"
        if bart:
            wl.verifier, wl.drafter = W.BART_V, W.BART_D
            wl.src = [W.zipf_ids(np.random.default_rng(105 + b), S, W.BART_V.vocab) for b in range(B)]
        wv = W.make_weights(wl.verifier, wl.seed_verifier, True, learned_pos=bart)
        wd = W.make_weights(wl.drafter, wl.seed_drafter, True, learned_pos=bart)
        sd = binding.SpecDec(wl.verifier, wv, wl.drafter, wd, k_max=max(ks), max_batch=B, max_src=S,
                             max_tgt=max(prefixes) + max(ks) + 2, bf16=True, activation="gelu" if bart else "relu")
        del wv, wd
        sd.set_option("gemm", args.gemm)
        sd.set_option("graphs", args.graphs)
        sd.set_option("tc_bn", args.tc_bn)
        for o in args.opt:
            sd.set_option(o.split("=")[0], int(o.split("=")[1]))
        for j in prefixes:
            for k in ks:
                us, us_min, mean_a = measure(sd, wl, B, k, j, S, args.reps, args.warmup, flush, args.draft)
                params, bytes_, flops = algorithmic_work(B, k, j, S, wl.verifier)
                if args.grid:
                    print(f"| {B} | {k} | {j} | {us:.1f} | {bytes_ / 1e6:.1f} | {flops / 1e9:.2f} | {bytes_ / us / 1e3:.0f} | "
                          f"{100 * bytes_ / us / 1e3 / hbm:.1f} | {flops / us / 1e6:.1f} | {100 * flops / us / 1e6 / tc:.1f} | {mean_a:.2f} |",
                          flush=True)
                else:
                    print(json.dumps({
                        "step": "draft" if args.draft else "verify", "batch": B, "k": k, "prefix": j, "src_len": S,
                        "us_median": us, "us_min": us_min, "l2_flush": flush is not None, "mean_accepted": mean_a,
                        "algorithmic_MB": bytes_ / 1e6, "algorithmic_GFLOP": flops / 1e9,
                        "hbm_GBs": bytes_ / us / 1e3, "hbm_frac": bytes_ / us / 1e3 / hbm,
                        "tensor_TFLOPs": flops / us / 1e6, "tensor_frac": flops / us / 1e6 / tc, "peaks": kind,
                    }))
        sd.close()


if __name__ == "__main__":
    main()
