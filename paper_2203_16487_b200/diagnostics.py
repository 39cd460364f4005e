"""Timing diagnostics that the performance notes under profiles/ are made with.

  python -m paper_2203_16487_b200.diagnostics --cluster-trace   # per-phase time inside the cluster decoder kernel
  python -m paper_2203_16487_b200.diagnostics --vocab-trace     # time line of one CTA of the vocabulary GEMM
  python -m paper_2203_16487_b200.diagnostics --boundary-probe  # cost of a dependency between two small kernels, two ways to wait
  python -m paper_2203_16487_b200.diagnostics --ingest-probe    # bytes per second one / eight / all SMs can pull from HBM

The traces use the library's "cl_trace" option: the kernels record the global nanosecond timer at a few
points (first CTA only) into a small device buffer that specdec_debug_cluster_trace copies back.
"""
from __future__ import annotations

import argparse
import os
import subprocess

import numpy as np
import torch

from . import binding, workloads as W


def _handle(k=25, batch=1):
    wl = W.config5_microbench(batch, 64)
    wv = W.make_weights(wl.verifier, wl.seed_verifier, True)
    wd = W.make_weights(wl.drafter, wl.seed_drafter, True)
    sd = binding.SpecDec(wl.verifier, wv, wl.drafter, wd, k_max=k, max_batch=batch, max_src=64, max_tgt=100, bf16=True)
    src, lens = W.pad_batch(wl.src)
    return sd, src, lens


def cluster_trace(reps=20):
    sd, src, lens = _handle()
    sd.set_option("cluster", 1); sd.set_option("cl_trace", 1); sd.set_option("graphs", 0)
    sd.encode(src, lens, None)
    drafts = np.arange(100, 125, dtype=np.int32)[None]
    for _ in range(reps):
        sd.verify(drafts, 3, 1.0)
    torch.cuda.synchronize()
    tt = np.array(sd.cluster_trace(256), dtype=np.int64)
    t, ck = tt[:61], tt[128:189]
    print(f"SM clock during the kernel: {(ck[60] - ck[0]) / ((t[60] - t[0]) / 1e3):.0f} MHz")
    names = sum([[f"L{l} LN1", f"L{l} QKV GEMM", f"L{l} self-attention", f"L{l} barrier", f"L{l} out-proj (+barrier)",
                  f"L{l} LNc+Q+cross-attn (+barrier)", f"L{l} cross out-proj (+barrier)", f"L{l} LN2+FFN1 (+barrier)",
                  f"L{l} load hidden rows", f"L{l} FFN2 (+barrier)"] for l in range(6)], [])
    for n, x in zip(names, np.diff(t)):
        print(f"{n:34s} {x / 1e3:7.2f} us")
    print(f"whole kernel (after the wait on its predecessor): {(t[60] - t[0]) / 1e3:.1f} us")
    sd.close()


def vocab_trace(reps=20, opts=(), batch=1):
    sd, src, lens = _handle(batch=batch)
    sd.set_option("cl_trace", 1); sd.set_option("graphs", 0)
    for name, value in opts:
        sd.set_option(name, value)
    sd.encode(src, lens, None)
    drafts = np.tile(np.arange(100, 125, dtype=np.int32)[None], (batch, 1))
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    for it in range(reps):
        flush.fill_(it & 0xff)
        sd.verify(drafts, 3, 1.0)
    torch.cuda.synchronize()
    t = np.array(sd.cluster_trace(256), dtype=np.int64)[200:214]
    tt = np.array(sd.cluster_trace(256), dtype=np.int64)
    print("k-block landings (us since entry):", [round((x - t[0]) / 1e3, 2) for x in tt[240:256]])
    t = np.concatenate([t[:1], t[12:14], t[1:12]])
    names = ["kernel entry", "mbarriers initialised", "TMEM allocated", "barriers + TMEM ready", "first TMA issued", "all TMA issued", "first stage landed",
             "tile 0 MMAs committed", "last tile MMAs committed", "epilogue tile 0 start", "epilogue tile 0 end",
             "epilogue tile 1 start", "epilogue tile 1 end", "exit"]
    for n, x in zip(names, t):
        print(f"{n:28s} {(x - t[0]) / 1e3:7.2f} us")
    sd.close()


def ingest_probe():
    here = os.path.dirname(os.path.abspath(__file__))
    exe = "/tmp/specdec_ingest_probe"
    subprocess.check_call(["nvcc", "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-o", exe,
                           os.path.join(here, "csrc", "ingest_probe.cu")])
    subprocess.check_call([exe])


def boundary_probe():
    here = os.path.dirname(os.path.abspath(__file__))
    exe = "/tmp/specdec_boundary_probe"
    subprocess.check_call(["nvcc", "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-o", exe,
                           os.path.join(here, "csrc", "boundary_probe.cu")])
    subprocess.check_call([exe])


if __name__ == "__main__":
    ap = argparse.ArgumentParser()
    ap.add_argument("--cluster-trace", action="store_true")
    ap.add_argument("--vocab-trace", action="store_true")
    ap.add_argument("--ingest-probe", action="store_true")
    ap.add_argument("--boundary-probe", action="store_true")
    ap.add_argument("--batch", type=int, default=1, help="vocab trace: sequences in the verify step")
    ap.add_argument("--opt", action="append", default=[], help="library option name=value (repeatable), vocab trace only")
    a = ap.parse_args()
    if a.cluster_trace:
        cluster_trace()
    if a.vocab_trace:
        vocab_trace(batch=a.batch, opts=[(o.split("=")[0], int(o.split("=")[1])) for o in a.opt])
    if a.ingest_probe:
        ingest_probe()
    if a.boundary_probe:
        boundary_probe()
