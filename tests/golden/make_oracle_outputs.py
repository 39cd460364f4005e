"""Writes tests/golden/oracle_outputs.json: token sequences that ONLY the CPU oracle produced, for the full-size
parity tests whose oracle work is too slow to repeat inside a test (Transformer-base shapes, whole sentences,
every (beta, tau) cell of the batched workload).

  python tests/golden/make_oracle_outputs.py          (a few minutes on 8 cores)

It imports the oracle and the seeded input generator only; nothing here touches the CUDA path.  Contents:
  config2.natural[i]      O.specdec_generate on sentence i of the translation-shaped workload (the real drafter)
  config2.greedy[i]       O.greedy_decode on the same sentence (the scripted-acceptance test builds its script from it)
  config3.cells[i][cell]  sequence i of the batched workload under (beta, tau) = cell, for the nine cells
The nine cells of one sequence are advanced together: cells whose committed prefixes coincide share one drafter pass
and one verifier pass (the rule is then applied per cell to the same rows), which is what the functions compute
anyway -- only repeated work is skipped.
"""
from __future__ import annotations

import json
import os
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from oracle import specdec_oracle as O                      # noqa: E402
from paper_2203_16487_b200 import workloads as W           # noqa: E402

K = 25
CELLS = [(b, t) for b in (1, 3, 5) for t in (0.0, 1.0, 3.0)]
CONFIG2_SENTENCES = list(range(8))
CONFIG3_B32 = [0, 3, 7, 12, 18, 23, 27, 31]                 # all nine cells
CONFIG3_B128_EXTRA = [40, 77, 101, 127]                     # (3, 1.0) only (with the eight above: 12 sequences of the batch of 128)


def copy_cache(c: O.DecoderCache, n: int) -> O.DecoderCache:
    return O.DecoderCache([a[:n].copy() for a in c.k], [a[:n].copy() for a in c.v], c.ck, c.cv)


def cells_together(mv, md, src, max_tgt, cells):
    """O.specdec_generate for several (beta, tau) on one source, sharing passes between cells with equal prefixes."""
    mem_v, mem_d = O.encode(mv, src), O.encode(md, src)
    groups = [(tuple(), O.new_cache(mv, mem_v), list(cells))]
    out = {}
    while groups:
        prefix, cache, members = groups.pop()
        if len(prefix) >= max_tgt and len(prefix) > 0 or max_tgt <= 0:
            for c in members:
                out[c] = list(prefix)
            continue
        committed = list(prefix)
        d = O.draft(md, mem_d, committed, K, W.BOS_ID, W.MASK_ID)
        rows = O.verify_rows(mv, mem_v, committed, d, W.BOS_ID, cache)
        nxt = {}
        for c in members:
            a, bif = O.verify(rows, d, c[0], c[1])
            o = list(committed)
            done = O.commit(o, d, a, bif, max_tgt, W.EOS_ID)
            if done:
                out[c] = o
            else:
                nxt.setdefault(tuple(o), []).append(c)
        for p, ms in nxt.items():
            groups.append((p, copy_cache(cache, len(p)), ms))
    return out


def main():
    t0 = time.time()
    res = {"k": K, "config2": {"natural": {}, "greedy": {}}, "config3": {"cells": {}}}
    wl2 = W.config2_translation()
    wv = W.make_weights(wl2.verifier, wl2.seed_verifier, True)
    wd = W.make_weights(wl2.drafter, wl2.seed_drafter, True)
    mv, md = O.model_from(wl2.verifier, wv, mode="bf16"), O.model_from(wl2.drafter, wd, mode="bf16")
    for i in CONFIG2_SENTENCES:
        src, mt = wl2.src[i], wl2.max_tgt[i]
        nat, _ = O.specdec_generate(mv, md, src, mt, K, 3, 1.0, W.BOS_ID, W.EOS_ID, W.MASK_ID)
        res["config2"]["natural"][str(i)] = [int(t) for t in nat]
        res["config2"]["greedy"][str(i)] = [int(t) for t in O.greedy_decode(mv, src, mt, W.BOS_ID, W.EOS_ID)]
        print(f"config2 sentence {i}: {len(nat)} tokens, {time.time() - t0:.0f} s", flush=True)
    wl3 = W.config3_batched(128)
    for i in CONFIG3_B32 + CONFIG3_B128_EXTRA:
        cells = CELLS if i in CONFIG3_B32 else [(3, 1.0)]
        got = cells_together(mv, md, wl3.src[i], wl3.max_tgt[i], cells)
        res["config3"]["cells"][str(i)] = {f"{b},{t:g}": [int(x) for x in got[(b, t)]] for b, t in cells}
        print(f"config3 sequence {i}: {len(wl3.src[i])} source ids, {len(got[cells[0]])} tokens, {time.time() - t0:.0f} s", flush=True)
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "oracle_outputs.json")
    with open(path, "w") as f:
        json.dump(res, f, separators=(",", ":"))
    print("wrote", path, f"{time.time() - t0:.0f} s")


if __name__ == "__main__":
    main()
