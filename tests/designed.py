"""Hand-checkable model pair used by both the oracle pins and the GPU parity tests.

All attention output projections and the second FFN matrices (with their
biases) are zero, so every sublayer adds nothing and the decoder output is
LN_f(sqrt(d) E[token] + P[position]) E^T: a function of (token, position)
only.  The embedding rows of chosen tokens are then set so that

  * the verifier's top-1 after consuming target token T[t] at position t is T[t+1];
  * the drafter's top-1 at a [MASK] placed at position p is D[p].

With T and D laid out as in the paper's worked example (Appendix "Case Study":
k = 10, three iterations, an [EOS] drafted too early, a final accepted [EOS])
the expected accepted lengths and emitted counts are known without running
any model.
"""
from __future__ import annotations

import numpy as np

from paper_2203_16487_b200 import workloads as W

ALPHA = 0.05


def _ln(x):
    mu = x.mean()
    return (x - mu) / np.sqrt(((x - mu) ** 2).mean() + 1e-5)


def _zero_sublayers(w, dims):
    for name in list(w):
        if name.endswith(".o.w") or name.endswith(".o.b") or name.endswith(".w2") or name.endswith(".b2"):
            w[name] = np.zeros_like(w[name])
    for name in list(w):
        if name.endswith("ln_f.g"):
            w[name] = np.ones_like(w[name])
        if name.endswith("ln_f.b"):
            w[name] = np.zeros_like(w[name])


def case_study_pair(seed: int = 77, near_top_at: int = 0):
    """Returns (dims_v, w_v, dims_d, w_d, T, D, src).

    T[1..15]: the verifier's greedy output (T[15] = EOS).  D[p]: the drafter's
    token at position p.  D = T except D[3] (a wrong token), D[13] = EOS (too
    early) and D[p > 15] (filler).  If near_top_at = p > 0, D[p] is instead a
    token U whose verifier logit at row p-1 is 0.9x the top-1's: accepted by
    (beta=3, tau=1), rejected by strict matching.
    """
    rng = np.random.default_rng(seed)
    dv, dd = W.TINY_V, W.TINY_D
    wv = W.make_weights(dv, seed + 1, False)
    wd = W.make_weights(dd, seed + 2, False)
    _zero_sublayers(wv, dv)
    _zero_sublayers(wd, dd)
    d = dv.d_model
    wv["pos_dec"] = rng.standard_normal((dv.max_pos, d)).astype(np.float32)
    wd["pos_dec"] = rng.standard_normal((dd.max_pos, d)).astype(np.float32)

    ids = rng.permutation(np.arange(10, 900))[:64].astype(int)
    L = 15
    T = [W.BOS_ID] + [int(t) for t in ids[:L - 1]] + [W.EOS_ID]          # T[0] = BOS, T[15] = EOS
    wrong = [int(t) for t in ids[20:60]]
    sq = np.float32(np.sqrt(d))

    # verifier: E[T[t+1]] = alpha * LN(sqrt(d) E[T[t]] + P[t]), built left to right
    E = wv["embed"]
    U = int(ids[62])
    for t in range(L):
        x = sq * E[T[t]] + wv["pos_dec"][t]
        E[T[t + 1]] = (ALPHA * _ln(x)).astype(np.float32)
        if near_top_at and t == near_top_at - 1:
            E[U] = (0.9 * ALPHA * _ln(x)).astype(np.float32)

    # drafter: the row at a mask position p sees sqrt(d) E_D[MASK] + P_D[p]
    D = {p: T[p] for p in range(1, L + 1)}
    D[3] = wrong[0]
    D[13] = W.EOS_ID
    if near_top_at:
        D[near_top_at] = U
    for p in range(L + 1, 40):
        D[p] = wrong[p - L]
    ED = wd["embed"]
    acc = {}
    for p, tok in D.items():
        x = sq * ED[W.MASK_ID] + wd["pos_dec"][p]
        acc[tok] = acc.get(tok, 0) + ALPHA * _ln(x)
    for tok, v in acc.items():
        ED[tok] = v.astype(np.float32)

    src = W.zipf_ids(rng, 12, dv.vocab)
    return dv, wv, dd, wd, T, D, src
