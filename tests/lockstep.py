"""Lock-step comparison of the CUDA path with the CPU oracle (test infrastructure).

Every iteration both sides start from the same committed prefix: the CUDA
drafter's output is compared with the oracle's, then both verify the ORACLE's
drafts, the decisions (accepted length, bifurcation token) are compared, and the
oracle's decision is committed on both sides (specdec_commit with explicit
keep / next).  A disagreement never propagates, so every position of every
sequence is checked.  A disagreement is "allowed" only when the oracle's margin
for the decision that differed is below `margin` (1e-3 in the bf16 configs, 0
in fp32), and it is counted.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional

import numpy as np
import torch

from oracle import specdec_oracle as O
from paper_2203_16487_b200 import workloads as W


@dataclass
class Report:
    iterations: int = 0
    draft_positions: int = 0
    draft_near_ties: int = 0
    draft_failures: int = 0
    verify_rows: int = 0
    verify_near_ties: int = 0
    verify_failures: int = 0
    max_logit_err: float = 0.0
    max_stat_err: float = 0.0
    outputs: List[List[int]] = field(default_factory=list)
    notes: List[str] = field(default_factory=list)

    @property
    def ok(self):
        return self.draft_failures == 0 and self.verify_failures == 0


def run(sd, mv: O.Model, md: O.Model, srcs, max_tgt, k, beta, tau, margin: float,
        eos: int = W.EOS_ID, max_iters: Optional[int] = None, check_logits_every: int = 0,
        logit_tol: float = 1e-4, draft_fn=None, pad_to: Optional[int] = None,
        drafter_reading: str = "bidirectional") -> Report:
    rep = Report()
    B = len(srcs)
    sd.set_option("row_lse", 1)
    sd.set_option("drafter_prefix_causal", 1 if drafter_reading == "prefix_causal" else 0)
    src, lens = W.pad_batch(srcs, pad_to)
    sd.encode(src, lens, np.asarray(max_tgt, np.int32))
    mem_v = [O.encode(mv, s) for s in srcs]
    mem_d = [O.encode(md, s) for s in srcs]
    cache = [O.new_cache(mv, m) for m in mem_v]
    out: List[List[int]] = [[] for _ in range(B)]
    done = [mt <= 0 for mt in max_tgt]
    it = 0
    while not all(done) and (max_iters is None or it < max_iters):
        # ---- draft
        g_draft = sd.draft(k).cpu().numpy()
        o_draft = np.zeros((B, k), np.int32)
        for b in range(B):
            if done[b]:
                continue
            if draft_fn is not None:
                o_draft[b] = draft_fn(b, list(out[b]), k)
                continue
            j = len(out[b])
            logits = O.decoder_rows(md, [W.BOS_ID] + out[b] + [W.MASK_ID] * k, mem_d[b], causal=False,
                                    n_causal=(j + 1 if drafter_reading == "prefix_causal" else None))[j + 1:]
            o_draft[b] = logits.argmax(axis=1)
            for i in range(k):
                rep.draft_positions += 1
                if g_draft[b, i] != o_draft[b, i]:
                    gap = float(logits[i, o_draft[b, i]] - logits[i, g_draft[b, i]]) if 0 <= g_draft[b, i] < logits.shape[1] else np.inf
                    if gap < margin:
                        rep.draft_near_ties += 1
                    else:
                        rep.draft_failures += 1
                        rep.notes.append(f"draft it={it} b={b} i={i} gpu={g_draft[b, i]} oracle={o_draft[b, i]} gap={gap:.3e}")
        # ---- verify the oracle's drafts on both sides
        acc, bif = sd.verify(o_draft, beta, tau)
        acc, bif = acc.cpu().numpy(), bif.cpu().numpy()
        stats = sd.debug_row_stats(k).cpu().numpy()
        want_logits = check_logits_every and it % check_logits_every == 0
        g_logits = sd.debug_logits(0, B * (k + 1)).cpu().numpy().reshape(B, k + 1, -1) if want_logits else None
        keep = np.zeros(B, np.int32)
        nxt = np.zeros(B, np.int32)
        for b in range(B):
            if done[b]:
                continue
            d = o_draft[b].tolist()
            rows = O.verify_rows(mv, mem_v[b], out[b], d, W.BOS_ID, cache[b])
            a, t = O.verify(rows, d, beta, tau)
            keep[b], nxt[b] = a, t
            if g_logits is not None:
                rep.max_logit_err = max(rep.max_logit_err, float(np.abs(g_logits[b] - rows).max()))
            # row statistics the CUDA epilogue derives without storing logits
            for c in range(k + 1):
                rep.verify_rows += 1
                rep.max_stat_err = max(rep.max_stat_err, abs(float(stats[b, c, 0]) - float(rows[c].max())))
                lse = float(np.log(np.exp(rows[c].astype(np.float64) - rows[c].max()).sum()) + rows[c].max())
                rep.max_stat_err = max(rep.max_stat_err, abs(float(stats[b, c, 2]) - lse))
                if c < k:
                    rep.max_stat_err = max(rep.max_stat_err, abs(float(stats[b, c, 4]) - float(rows[c][d[c]])))
            if (acc[b], bif[b]) != (a, t):
                # which decision differed first?
                first = min(int(acc[b]), a)
                m_rank, m_tau, gap = O.decision_margins(rows[first], d[first] if first < k else None, beta, tau)
                if acc[b] != a:
                    near = min(m_rank, m_tau) < margin
                    what = f"accept row {first}: margins rank={m_rank:.3e} tau={m_tau:.3e}"
                else:
                    near = gap < margin
                    what = f"bifurcation row {first}: top1-top2={gap:.3e}"
                if near:
                    rep.verify_near_ties += 1
                else:
                    rep.verify_failures += 1
                    rep.notes.append(f"verify it={it} b={b} gpu=({acc[b]},{bif[b]}) oracle=({a},{t}) {what}")
        # ---- commit the oracle's decision on both sides
        sd.commit(keep, nxt)
        for b in range(B):
            if done[b]:
                continue
            done[b] = O.commit(out[b], o_draft[b].tolist(), int(keep[b]), int(nxt[b]), max_tgt[b], eos)
            cache[b].truncate(len(out[b]))
        it += 1
    rep.iterations = it
    g_out, g_n, g_fin = sd.output()
    g_out, g_n, g_fin = g_out.cpu().numpy(), g_n.cpu().numpy(), g_fin.cpu().numpy()
    for b in range(B):
        got = g_out[b, :g_n[b]].tolist()
        if got != out[b] or bool(g_fin[b]) != bool(done[b]):
            rep.verify_failures += 1
            rep.notes.append(f"state b={b}: gpu len {g_n[b]} fin {g_fin[b]} vs oracle len {len(out[b])} fin {done[b]}")
    rep.outputs = out
    return rep
