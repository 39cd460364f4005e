"""CPU oracle for the SpecDec draft -> verify -> commit path.  TEST INFRASTRUCTURE ONLY.

A plain, slow, readable numpy implementation of what the CUDA path must
compute, written from the paper: the autoregressive encoder-decoder verifier,
the non-autoregressive Spec-Drafter pass over k [MASK] queries (Section 3.1.3,
the inference equation), vanilla draft-then-verify (Section 2, Eq. 1-3), the
Spec-Verification rule (Section 3.2, Eq. 7-9) and the decode loop (Section 2,
last sentence; Appendix "Case Study").

It is independent of the CUDA path: it imports nothing from the package, shares
no helper, table or constant with it, and only tests, the smoke check and the
benchmark's CPU-baseline leg may import it.  The product never routes through it.

Precision: the paper ran in fp32 (its memory tables are fp32), so the oracle
computes in np.float32 by default; pass dtype=np.float64 to measure its own
rounding noise.  `mode="bf16"` additionally rounds values to bf16 at the points
where the CUDA path feeds bf16 operands to its tensor-core contractions
(normalised activations, Q/K/V, un-normalised attention probabilities,
attention output, feed-forward activation output, encoder memory); accumulation
stays in `dtype`.

The paper gives only layer counts and 512/2048 widths (Section 4.1).  The rest
of the architecture is a stated reading: pre-LN blocks, ReLU, eps 1e-5,
sqrt(d)-scaled shared embeddings plus a position table, biases everywhere, tied
output projection without bias, argmax ties to the lowest id.  `act="gelu"`
switches the feed-forward activation to the exact (erf) GELU for the BART-base
shaped pair of the summarisation experiment (Section 5.2; BART's dimensions are
public knowledge, not the paper's: 768 wide, 12 heads, 3072 inner, 50265 ids,
learned position tables, which here are simply the pos_enc / pos_dec weights).

Pinned (tests/test_oracle_pins.py): greedy equivalence at beta=1, tau=0;
brute-force log-prob form of Eq. 7-8 on tiny vocabularies; monotonicity in
beta and tau; block-parallel == sequential rows; cached == from scratch; the
worked example's iteration structure; the parameter count implied by the
paper's memory table; a closed-form model with zeroed sublayers; the whole
encoder / decoder stack against torch.nn's pre-LN Transformer layers in fp64
(ReLU and GELU); every weight shown to influence the output; the points at
which mode="bf16" rounds (a recorder in place of bf16_round); decision_margins
on hand-worked rows; the prefix-causal drafter reading against torch.nn layers
given the same mask, against the plain causal decoder on its prefix rows, cached
against from scratch.
Parity unpinned: nothing about translation quality (needs trained weights).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np
from scipy.special import erf as _erf      # library routine: the error function of the exact GELU

LN_EPS = 1e-5


# ----------------------------------------------------------------------------
# small numeric helpers
# ----------------------------------------------------------------------------
def bf16_round(a: np.ndarray) -> np.ndarray:
    """Nearest-even rounding to bf16, returned in the input's float dtype."""
    dt = a.dtype
    f = np.ascontiguousarray(a, dtype=np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).reshape(a.shape).astype(dt)


def argmax_lowest(v: np.ndarray) -> int:
    """Index of the maximum; the lowest index among equal maxima."""
    return int(np.argmax(v))  # numpy returns the first occurrence


@dataclass
class Model:
    """Weights of one encoder-decoder Transformer plus its dimensions."""
    d_model: int
    n_heads: int
    d_ffn: int
    vocab: int
    enc_layers: int
    dec_layers: int
    w: Dict[str, np.ndarray]
    dtype: type = np.float32
    mode: str = "pure"            # "pure" | "bf16"
    act: str = "relu"             # feed-forward activation: "relu" (Transformer-base, Section 4.1) | "gelu" (BART-base, Section 5.2)

    def __post_init__(self):
        self.w = {k: np.asarray(v, dtype=self.dtype) for k, v in self.w.items()}

    def r(self, a: np.ndarray) -> np.ndarray:
        return bf16_round(a) if self.mode == "bf16" else a


def model_from(dims, weights, dtype=np.float32, mode="pure", act="relu") -> Model:
    return Model(dims.d_model, dims.n_heads, dims.d_ffn, dims.vocab,
                 dims.enc_layers, dims.dec_layers, weights, dtype, mode, act)


# ----------------------------------------------------------------------------
# Transformer blocks (pre-LN)
# ----------------------------------------------------------------------------
def layer_norm(x: np.ndarray, g: np.ndarray, b: np.ndarray) -> np.ndarray:
    mu = x.mean(axis=-1, keepdims=True)
    var = ((x - mu) ** 2).mean(axis=-1, keepdims=True)          # biased variance
    return (x - mu) / np.sqrt(var + x.dtype.type(LN_EPS)) * g + b


def linear(m: Model, x: np.ndarray, name: str) -> np.ndarray:
    return x @ m.w[name + ".w"].T + m.w[name + ".b"]


def attention(m: Model, q: np.ndarray, k: np.ndarray, v: np.ndarray,
              allowed: np.ndarray) -> np.ndarray:
    """softmax(q k^T / sqrt(d_h) + mask) v per head.

    q [Tq,d], k/v [Tk,d], allowed [Tq,Tk] bool.  In bf16 mode q, k, v arrive
    already rounded; the un-normalised probabilities exp(s - max) are rounded
    before the weighted sum while the normaliser uses the unrounded ones.
    """
    H, dh = m.n_heads, m.d_model // m.n_heads
    scale = q.dtype.type(1.0 / np.sqrt(dh))
    out = np.zeros_like(q)
    for h in range(H):
        sl = slice(h * dh, (h + 1) * dh)
        s = (q[:, sl] @ k[:, sl].T) * scale
        s = np.where(allowed, s, -np.inf)
        e = np.exp(s - s.max(axis=-1, keepdims=True))
        denom = e.sum(axis=-1, keepdims=True)
        out[:, sl] = (m.r(e) @ v[:, sl]) / denom
    return out


def embed(m: Model, tokens: Sequence[int], positions: Sequence[int], table: str) -> np.ndarray:
    tok = np.asarray(tokens, dtype=np.int64)
    pos = np.asarray(positions, dtype=np.int64)
    return m.w["embed"][tok] * m.dtype(np.sqrt(m.d_model)) + m.w[table][pos]


def gelu(x: np.ndarray) -> np.ndarray:
    """x * Phi(x) with the exact normal CDF (the erf form), in the dtype of x."""
    return (x * (x.dtype.type(0.5) * (x.dtype.type(1) + _erf(x * x.dtype.type(1.0 / np.sqrt(2.0)))))).astype(x.dtype)


def ffn(m: Model, y: np.ndarray, p: str) -> np.ndarray:
    pre = y @ m.w[p + ".w1"].T + m.w[p + ".b1"]
    hdn = gelu(pre) if m.act == "gelu" else np.maximum(pre, 0)
    return m.r(hdn) @ m.w[p + ".w2"].T + m.w[p + ".b2"]


def encode(m: Model, src: Sequence[int]) -> np.ndarray:
    """Encoder stack over one unpadded source -> memory [S,d] (final LN applied)."""
    S = len(src)
    x = embed(m, src, range(S), "pos_enc")
    allowed = np.ones((S, S), dtype=bool)
    for l in range(m.enc_layers):
        p = f"enc.{l}"
        y = m.r(layer_norm(x, m.w[p + ".ln1.g"], m.w[p + ".ln1.b"]))
        q, k, v = (m.r(linear(m, y, f"{p}.self.{n}")) for n in "qkv")
        x = x + linear(m, m.r(attention(m, q, k, v, allowed)), p + ".self.o")
        y = m.r(layer_norm(x, m.w[p + ".ln2.g"], m.w[p + ".ln2.b"]))
        x = x + ffn(m, y, p + ".ffn")
    return m.r(layer_norm(x, m.w["enc.ln_f.g"], m.w["enc.ln_f.b"]))


@dataclass
class DecoderCache:
    """Self-attention K/V of already processed positions, per layer; cross K/V of the memory."""
    k: List[np.ndarray]
    v: List[np.ndarray]
    ck: List[np.ndarray]
    cv: List[np.ndarray]

    @property
    def length(self) -> int:
        return self.k[0].shape[0]

    def truncate(self, n: int) -> None:
        self.k = [a[:n] for a in self.k]
        self.v = [a[:n] for a in self.v]


def new_cache(m: Model, mem: np.ndarray) -> DecoderCache:
    ck, cv = [], []
    for l in range(m.dec_layers):
        ck.append(m.r(linear(m, mem, f"dec.{l}.cross.k")))
        cv.append(m.r(linear(m, mem, f"dec.{l}.cross.v")))
    z = [np.zeros((0, m.d_model), dtype=m.dtype) for _ in range(m.dec_layers)]
    return DecoderCache(list(z), list(z), ck, cv)


def decoder_rows(m: Model, tokens: Sequence[int], mem: np.ndarray, causal: bool,
                 cache: Optional[DecoderCache] = None, n_causal: Optional[int] = None) -> np.ndarray:
    """Decoder stack -> logits [len(tokens), V] = LN_f(h) E^T (tied, no bias).

    Without a cache the tokens occupy positions 0..T-1 and everything is
    computed from scratch (the plain definition).  With a cache the tokens
    occupy positions cache.length.. and attend to the cached positions too; the
    cache is extended in place with the new rows.

    Self-attention mask: causal (position p sees 0..p), none (causal=False), or
    -- n_causal given -- "prefix-causal": positions below n_causal are causal,
    the positions from n_causal on see every position of the pass (the drafter's
    second reading: committed tokens never look at the [MASK] block, so their
    rows can be cached like an autoregressive decoder's).  Cached passes need a
    mask under which cached rows never depend on later ones: causal or
    prefix-causal with the cache inside the causal part.
    """
    T = len(tokens)
    start = 0 if cache is None else cache.length
    if cache is None:
        cache = new_cache(m, mem)
    else:
        assert causal or (n_causal is not None and start <= n_causal), "a non-causal pass cannot reuse cached rows"
    x = embed(m, tokens, range(start, start + T), "pos_dec")
    qpos = np.arange(start, start + T)[:, None]
    kpos = np.arange(0, start + T)[None, :]
    if n_causal is not None:
        allowed = (kpos <= qpos) | (qpos >= n_causal)
    else:
        allowed = (kpos <= qpos) if causal else np.ones((T, start + T), dtype=bool)
    cross_ok = np.ones((T, mem.shape[0]), dtype=bool)
    for l in range(m.dec_layers):
        p = f"dec.{l}"
        y = m.r(layer_norm(x, m.w[p + ".ln1.g"], m.w[p + ".ln1.b"]))
        q, k, v = (m.r(linear(m, y, f"{p}.self.{n}")) for n in "qkv")
        cache.k[l] = np.concatenate([cache.k[l], k], axis=0)
        cache.v[l] = np.concatenate([cache.v[l], v], axis=0)
        a = attention(m, q, cache.k[l], cache.v[l], allowed)
        x = x + linear(m, m.r(a), p + ".self.o")
        y = m.r(layer_norm(x, m.w[p + ".ln_cross.g"], m.w[p + ".ln_cross.b"]))
        q = m.r(linear(m, y, p + ".cross.q"))
        a = attention(m, q, cache.ck[l], cache.cv[l], cross_ok)
        x = x + linear(m, m.r(a), p + ".cross.o")
        y = m.r(layer_norm(x, m.w[p + ".ln2.g"], m.w[p + ".ln2.b"]))
        x = x + ffn(m, y, p + ".ffn")
    y = m.r(layer_norm(x, m.w["dec.ln_f.g"], m.w["dec.ln_f.b"]))
    return y @ m.w["embed"].T


# ----------------------------------------------------------------------------
# Greedy autoregressive decoding with the verifier (the thing SpecDec accelerates)
# ----------------------------------------------------------------------------
def greedy_decode(m: Model, src: Sequence[int], max_tgt: int, bos: int, eos: int,
                  use_cache: bool = True) -> List[int]:
    mem = encode(m, src)
    out: List[int] = []
    cache = new_cache(m, mem) if use_cache else None
    while len(out) < max_tgt:
        if use_cache:
            row = decoder_rows(m, [out[-1] if out else bos], mem, True, cache)[-1]
        else:
            row = decoder_rows(m, [bos] + out, mem, True)[-1]
        tok = argmax_lowest(row)
        out.append(tok)
        if tok == eos:
            break
    return out


# ----------------------------------------------------------------------------
# Spec-Drafter inference (Section 3.1.3, inference equation)
# ----------------------------------------------------------------------------
def draft(md: Model, mem_d: np.ndarray, committed: Sequence[int], k: int,
          bos: int, mask: int, reading: str = "bidirectional",
          cache: Optional[DecoderCache] = None) -> List[int]:
    """k drafted tokens: argmax at the k [MASK] rows of one decoder pass.

    Input is [BOS, y_1..y_j, MASK x k] at positions 0..j+k; the row at a mask
    position predicts the token at that position (non-shifted).

    reading = "bidirectional" (default): no self-attention mask at all, every row
    sees every row ("mask-predict manner", Section 3.1).  reading =
    "prefix_causal": the committed tokens attend causally among themselves and
    the [MASK] rows see everything; the drafter decoder can then keep a K/V cache
    of the committed positions across iterations (Section 3.1.2's latency
    principle: the decoder is forwarded every iteration, so its work should not
    grow with the prefix).  With `cache` (positions 0..c-1 of [BOS, y...], c <=
    j+1) only the rows from c on are computed; the cache is left holding
    positions 0..j.
    """
    j = len(committed)
    tokens = [bos] + list(committed) + [mask] * k
    if reading == "bidirectional":
        assert cache is None
        logits = decoder_rows(md, tokens, mem_d, causal=False)
        return [argmax_lowest(logits[j + 1 + i]) for i in range(k)]
    assert reading == "prefix_causal"
    c = 0 if cache is None else cache.length
    assert c <= j + 1
    logits = decoder_rows(md, tokens[c:], mem_d, causal=False, cache=cache, n_causal=j + 1)
    if cache is not None:
        cache.truncate(j + 1)                   # the [MASK] rows are not part of the prefix
    return [argmax_lowest(logits[j + 1 - c + i]) for i in range(k)]


# ----------------------------------------------------------------------------
# Verification (Section 2 Eq. 1-3; Section 3.2 Eq. 7-9)
# ----------------------------------------------------------------------------
def verify_rows(mv: Model, mem_v: np.ndarray, committed: Sequence[int], drafts: Sequence[int],
                bos: int, cache: Optional[DecoderCache] = None) -> np.ndarray:
    """The k+1 verifier rows: row r is the distribution of y_{j+r+1} given the
    committed tokens, the first r drafts and the source.

    With a cache holding positions 0..j-1 only the block [y_j, drafts] is run.
    """
    j, k = len(committed), len(drafts)
    inputs = [bos] + list(committed) + list(drafts)
    if cache is None:
        return decoder_rows(mv, inputs, mem_v, True)[j:j + k + 1]
    assert cache.length == j
    return decoder_rows(mv, inputs[j:], mem_v, True, cache)


def accept_length(rows: np.ndarray, drafts: Sequence[int], beta: int, tau: float) -> int:
    """Number of leading drafts accepted under Eq. 7 and Eq. 8.

    Draft i (1-based) is checked on row i-1.  Eq. 7: its log-prob is at least
    the beta-th ranked log-prob, i.e. fewer than beta entries are strictly
    larger.  Eq. 8: top-1 log-prob minus its log-prob is at most tau.  The
    log-softmax normaliser is common to both sides of each inequality, so both
    are evaluated on the logits.  beta=1, tau=0 is the strict top-1 match of
    Eq. 2 (up to exact ties).
    """
    a = 0
    tau_t = rows.dtype.type(tau)
    for i, tok in enumerate(drafts):
        l = rows[i]
        ld = l[tok]
        n_greater = int(np.count_nonzero(l > ld))
        if n_greater <= beta - 1 and (l.max() - ld) <= tau_t:
            a += 1
        else:
            break
    return a


def verify(rows: np.ndarray, drafts: Sequence[int], beta: int, tau: float) -> Tuple[int, int]:
    """(accepted length a, bifurcation token): the token is the verifier's top-1 on
    row a -- the replacement of the first rejected draft, or the bonus token
    after a fully accepted block (Eq. 3 with c = a + 1)."""
    a = accept_length(rows, drafts, beta, tau)
    return a, argmax_lowest(rows[a])


def commit(out: List[int], drafts: Sequence[int], a: int, bif: int,
           max_tgt: int, eos: int) -> bool:
    """Append (drafts[:a], bif); cut after the first EOS and at max_tgt.  True = finished."""
    for tok in list(drafts[:a]) + [bif]:
        if len(out) >= max_tgt:
            return True
        out.append(int(tok))
        if tok == eos:
            return True
    return len(out) >= max_tgt


@dataclass
class GenStats:
    iterations: int = 0
    drafted: int = 0
    accepted: int = 0
    emitted: int = 0
    trace: List[Tuple[List[int], int, int]] = field(default_factory=list)  # (drafts, a, bif)


def specdec_generate(mv: Model, md: Model, src: Sequence[int], max_tgt: int, k: int,
                     beta: int, tau: float, bos: int, eos: int, mask: int,
                     use_cache: bool = True, draft_fn=None,
                     keep_trace: bool = False, script: Optional[Sequence[int]] = None,
                     drafter_reading: str = "bidirectional") -> Tuple[List[int], GenStats]:
    """Draft -> verify -> commit until EOS or max_tgt, one sequence.

    draft_fn(committed, k) may replace the drafter (scripted drafts in tests).
    drafter_reading: see draft(); "prefix_causal" keeps a drafter K/V cache when use_cache is set.
    script (benchmark hook, no counterpart in the paper): after the drafter has run,
    the draft for target index t is replaced by script[t] wherever script[t] >= 0.
    """
    mem_v = encode(mv, src)
    mem_d = encode(md, src) if draft_fn is None else None
    cache = new_cache(mv, mem_v) if use_cache else None
    dcache = new_cache(md, mem_d) if (use_cache and draft_fn is None and drafter_reading == "prefix_causal") else None
    out: List[int] = []
    st = GenStats()
    done = max_tgt <= 0
    while not done:
        d = draft(md, mem_d, out, k, bos, mask, drafter_reading, dcache) if draft_fn is None else list(draft_fn(list(out), k))
        if script is not None:
            j = len(out)
            d = [int(script[j + i]) if j + i < len(script) and script[j + i] >= 0 else d[i] for i in range(k)]
        rows = verify_rows(mv, mem_v, out, d, bos, cache)
        a, bif = verify(rows, d, beta, tau)
        n_before = len(out)
        done = commit(out, d, a, bif, max_tgt, eos)
        if cache is not None:
            cache.truncate(len(out))          # rollback: keep positions 0..j'-1 only
        st.iterations += 1
        st.drafted += k
        st.accepted += a
        st.emitted += len(out) - n_before
        if keep_trace:
            st.trace.append((list(d), a, bif))
    return out, st


# ----------------------------------------------------------------------------
# decision margins, for classifying near-ties when two implementations disagree
# ----------------------------------------------------------------------------
def decision_margins(row: np.ndarray, draft_tok: Optional[int], beta: int, tau: float):
    """(rank margin, tau margin, top1-top2 gap) of one verifier row.

    rank margin: distance of the draft's logit to the value it must not cross
    for the Eq. 7 outcome to flip; tau margin: |(max - l_d) - tau|; gap: how far
    the argmax is from changing.  inf where a quantity does not apply.
    """
    srt = np.sort(row.astype(np.float64))[::-1]
    gap = float(srt[0] - srt[1]) if srt.size > 1 else float("inf")
    if draft_tok is None:
        return float("inf"), float("inf"), gap
    ld = float(row[draft_tok])
    n_greater = int(np.count_nonzero(row > row[draft_tok]))
    if n_greater <= beta - 1:           # accepted by rank: flips if it drops below the next outsider
        others = np.delete(row.astype(np.float64), draft_tok)
        so = np.sort(others)[::-1]
        thr = so[beta - 1] if so.size >= beta else -np.inf
    else:                                # rejected by rank: flips if it reaches the beta-th value
        thr = srt[beta - 1]
    m_rank = abs(ld - float(thr))
    m_tau = abs((float(srt[0]) - ld) - float(tau))
    return m_rank, m_tau, gap
