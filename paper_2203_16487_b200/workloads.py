"""Seeded synthetic inputs for the SpecDec draft/verify path.

This module only *generates inputs*: model dimensions, random-init weights,
sinusoidal position tables, Zipf-distributed source token ids, length mixes and
the five workload recipes.  It holds none of the method's arithmetic (no layer
norm, attention, projection or acceptance rule) so that both the CUDA path and
the CPU oracle can be fed from it without sharing any code of the method.

The paper measures on WMT14/WMT16 translation test sets and CNN-DM
summarisation (Section 4.1); neither the data nor trained weights are available
offline, so every workload here is a seeded stand-in that keeps only the
*shapes*: sentence-level sources of tens of BPE ids over a joint 32K
vocabulary, paragraph-level sources of hundreds of ids, Transformer-base
verifier (6+6 layers, 512/2048; Section 4.1) and a 12+2 drafter.
"""
from __future__ import annotations

from dataclasses import dataclass, field, asdict
from typing import Dict, List, Optional

import numpy as np

PAD_ID, BOS_ID, EOS_ID, MASK_ID = 0, 1, 2, 3
N_SPECIAL = 4


@dataclass(frozen=True)
class ModelDims:
    d_model: int
    n_heads: int
    d_ffn: int
    vocab: int
    enc_layers: int
    dec_layers: int
    max_pos: int

    @property
    def d_head(self) -> int:
        return self.d_model // self.n_heads


@dataclass
class Workload:
    """One configuration: two models, sources and decoding hyper-parameters."""
    name: str
    verifier: ModelDims
    drafter: ModelDims
    k: int
    beta: int
    tau: float
    bf16: bool
    seed_verifier: int
    seed_drafter: int
    seed_data: int
    src: List[np.ndarray] = field(default_factory=list)      # each int32 [S_i]
    max_tgt: List[int] = field(default_factory=list)


# ----------------------------------------------------------------------------
# bf16 rounding of *inputs* (weights are rounded once, both sides use the result)
# ----------------------------------------------------------------------------
def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """Round fp32 values to the nearest bf16 (ties to even), returned as fp32."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    u = (u + np.uint32(0x7FFF) + lsb) & np.uint32(0xFFFF0000)      # finite inputs only: no carry out of bit 31
    return u.view(np.float32).reshape(a.shape)


def sinusoid_table(n_pos: int, d: int) -> np.ndarray:
    """Fixed sinusoidal position table [n_pos, d] evaluated in float64.

    First half sine, second half cosine over geometrically spaced wavelengths;
    passed to both sides as an ordinary weight buffer, so learned tables would
    work just as well.
    """
    half = d // 2
    freq = np.exp(-np.log(10000.0) * np.arange(half, dtype=np.float64) / max(half - 1, 1))
    ang = np.arange(n_pos, dtype=np.float64)[:, None] * freq[None, :]
    tab = np.zeros((n_pos, d), dtype=np.float64)
    tab[:, :half] = np.sin(ang)
    tab[:, half:2 * half] = np.cos(ang)
    return tab.astype(np.float32)


def make_weights(dims: ModelDims, seed: int, bf16: bool,
                 embed_std: float = 0.02, learned_pos: bool = False) -> Dict[str, np.ndarray]:
    """Random-init weights N(0, 0.02^2); LN gain 1 + N(0, 0.02^2).

    Names (row-major [out, in], y = x W^T + b):
      embed [V,d] (shared by encoder input, decoder input and output projection)
      pos_enc, pos_dec [max_pos,d]
      enc.{l}.ln1.{g,b}  enc.{l}.self.{q,k,v,o}.{w,b}  enc.{l}.ln2.{g,b}
      enc.{l}.ffn.{w1,b1,w2,b2}  enc.ln_f.{g,b}
      dec.{l}. ... same plus  ln_cross.{g,b}  cross.{q,k,v,o}.{w,b} ;  dec.ln_f.{g,b}
    With bf16=True every matrix (ndim >= 2, position tables excepted) is rounded
    once to bf16-representable values.  learned_pos=True draws the position tables
    N(0, 0.02^2) instead of evaluating sinusoids (BART-style learned positions).
    """
    rng = np.random.default_rng(seed)
    d, f, v = dims.d_model, dims.d_ffn, dims.vocab
    w: Dict[str, np.ndarray] = {}

    def mat(name, shape, std=0.02):
        a = rng.standard_normal(shape, dtype=np.float32) * np.float32(std)
        w[name] = round_to_bf16(a) if (bf16 and a.ndim >= 2) else a

    def ln(name):
        w[name + ".g"] = (1.0 + rng.standard_normal(d) * 0.02).astype(np.float32)
        w[name + ".b"] = (rng.standard_normal(d) * 0.02).astype(np.float32)

    def attn(prefix):
        for p in ("q", "k", "v", "o"):
            mat(f"{prefix}.{p}.w", (d, d))
            mat(f"{prefix}.{p}.b", (d,))

    def ffn(prefix):
        mat(prefix + ".w1", (f, d)); mat(prefix + ".b1", (f,))
        mat(prefix + ".w2", (d, f)); mat(prefix + ".b2", (d,))

    mat("embed", (v, d), embed_std)
    if learned_pos:
        w["pos_enc"] = rng.standard_normal((dims.max_pos, d), dtype=np.float32) * np.float32(0.02)
        w["pos_dec"] = rng.standard_normal((dims.max_pos, d), dtype=np.float32) * np.float32(0.02)
    else:
        w["pos_enc"] = sinusoid_table(dims.max_pos, d)
        w["pos_dec"] = sinusoid_table(dims.max_pos, d)
    for l in range(dims.enc_layers):
        ln(f"enc.{l}.ln1"); attn(f"enc.{l}.self"); ln(f"enc.{l}.ln2"); ffn(f"enc.{l}.ffn")
    ln("enc.ln_f")
    for l in range(dims.dec_layers):
        ln(f"dec.{l}.ln1"); attn(f"dec.{l}.self")
        ln(f"dec.{l}.ln_cross"); attn(f"dec.{l}.cross")
        ln(f"dec.{l}.ln2"); ffn(f"dec.{l}.ffn")
    ln("dec.ln_f")
    return w


def count_params(w: Dict[str, np.ndarray], include_pos: bool = False) -> int:
    return int(sum(a.size for n, a in w.items() if include_pos or not n.startswith("pos_")))


# ----------------------------------------------------------------------------
# token ids and lengths
# ----------------------------------------------------------------------------
def zipf_ids(rng: np.random.Generator, n: int, vocab: int, s: float = 1.1) -> np.ndarray:
    """n ids with rank r = 1..V-4 drawn with p(r) ~ r^-s, id = 3 + r (never a special id)."""
    ranks = np.arange(1, vocab - N_SPECIAL + 1, dtype=np.float64)
    p = ranks ** (-s)
    p /= p.sum()
    r = rng.choice(ranks.size, size=n, p=p) + 1
    return (r + (N_SPECIAL - 1)).astype(np.int32)


def make_sources(rng, n_src, lo, hi, vocab) -> List[np.ndarray]:
    lens = rng.integers(lo, hi + 1, size=n_src)
    return [zipf_ids(rng, int(L), vocab) for L in lens]


def pad_batch(seqs: List[np.ndarray], pad_to: Optional[int] = None):
    """Right-pad with PAD_ID: returns (ids [B,S_max] int32, lens [B] int32)."""
    lens = np.array([len(s) for s in seqs], dtype=np.int32)
    smax = int(pad_to if pad_to is not None else lens.max())
    out = np.full((len(seqs), smax), PAD_ID, dtype=np.int32)
    for i, s in enumerate(seqs):
        out[i, :len(s)] = s
    return out, lens


# ----------------------------------------------------------------------------
# the five workload recipes
# ----------------------------------------------------------------------------
TINY_V = ModelDims(64, 4, 256, 1000, 2, 2, 64)
TINY_D = ModelDims(64, 4, 256, 1000, 2, 1, 64)
BASE_V = ModelDims(512, 8, 2048, 32768, 6, 6, 1024)
BASE_D = ModelDims(512, 8, 2048, 32768, 12, 2, 1024)
# BART-base shapes (public model card, not the paper): 768 wide, 12 heads, 3072 inner, 50265 ids, GELU, learned
# positions; the drafter starts from the BART-base encoder (Section 5.2), so 6 encoder layers + 2 decoder layers.
BART_V = ModelDims(768, 12, 3072, 50265, 6, 6, 1026)
BART_D = ModelDims(768, 12, 3072, 50265, 6, 2, 1026)


def config1_tiny(beta: int = 3, tau: float = 1.0) -> Workload:
    """Tiny fp32 models, 4 sources of 16 ids, batch 1, max target 32, k=8."""
    wl = Workload("config1_tiny_fp32", TINY_V, TINY_D, 8, beta, tau, False, 11, 12, 101)
    rng = np.random.default_rng(wl.seed_data)
    wl.src = [zipf_ids(rng, 16, TINY_V.vocab) for _ in range(4)]
    wl.max_tgt = [32] * 4
    return wl


def config2_translation(n_src: int = 256) -> Workload:
    """Translation-shaped, batch 1: sources U[20,40], max target floor(1.2 S)+10, k=25."""
    wl = Workload("config2_translation_b1", BASE_V, BASE_D, 25, 3, 1.0, True, 1001, 1002, 102)
    rng = np.random.default_rng(wl.seed_data)
    wl.src = make_sources(rng, 256, 20, 40, BASE_V.vocab)[:n_src]
    wl.max_tgt = [int(1.2 * len(s)) + 10 for s in wl.src]
    return wl


def config3_batched(batch: int = 128, beta: int = 3, tau: float = 1.0) -> Workload:
    """Same models, padded batch of 32 or 128, sources U[10,80]."""
    wl = Workload(f"config3_batched_b{batch}", BASE_V, BASE_D, 25, beta, tau, True, 1001, 1002, 103)
    rng = np.random.default_rng(wl.seed_data)
    wl.src = make_sources(rng, 128, 10, 80, BASE_V.vocab)[:batch]
    wl.max_tgt = [int(1.2 * len(s)) + 10 for s in wl.src]
    return wl


def config4_summarization(batch: int = 8) -> Workload:
    """Summarisation-shaped: sources U[300,512], max target 128, batch 8."""
    wl = Workload("config4_summarization_b8", BASE_V, BASE_D, 25, 3, 1.0, True, 1001, 1002, 104)
    rng = np.random.default_rng(wl.seed_data)
    wl.src = make_sources(rng, 8, 300, 512, BASE_V.vocab)[:batch]
    wl.max_tgt = [128] * len(wl.src)
    return wl


def config_bart_summarization(batch: int = 4, lo: int = 300, hi: int = 512) -> Workload:
    """BART-base-shaped pair on paragraph-length sources (the summarisation setting of Section 5.2); weights via
    make_weights(..., learned_pos=True), handle / oracle with the GELU activation."""
    rng = np.random.default_rng(106)
    src = make_sources(rng, batch, lo, hi, BART_V.vocab)
    return Workload("config_bart_summarization", BART_V, BART_D, 25, 3, 1.0, True, 3001, 3002, 106, src,
                    [128] * batch)


def config5_microbench(batch: int, src_len: int = 64) -> Workload:
    """Verify-step microbench: verifier decoder only, encoder memory length 64."""
    wl = Workload(f"config5_verify_b{batch}", BASE_V, BASE_D, 50, 3, 1.0, True, 1001, 1002, 105)
    rng = np.random.default_rng(wl.seed_data)
    wl.src = [zipf_ids(rng, src_len, BASE_V.vocab) for _ in range(128)][:batch]
    wl.max_tgt = [320] * len(wl.src)
    return wl


def config5_prefix_and_rejections(batch: int, j: int, seed: int = 105):
    """Committed prefixes (j Zipf ids per sequence) and first-rejection positions.

    r ~ Geometric(p = 1/6) (mean 6), the 1-based draft index that the harness
    replaces with a token the verifier rejects; expected accepted length is
    min(r - 1, k).
    """
    rng = np.random.default_rng(seed + 7 * j + 1)
    prefix = [zipf_ids(rng, j, BASE_V.vocab) for _ in range(128)][:batch]
    rej = rng.geometric(1.0 / 6.0, size=128).astype(np.int32)[:batch]
    return prefix, rej


def sharp_tiny_models(seed: int = 31):
    """Tiny models whose embedding table is N(0, 0.06^2): top-1 to top-2 logit gaps are about 1,
    so tau in {0.5, 1, 3} and beta change what is accepted."""
    wv = make_weights(TINY_V, seed, False, embed_std=0.06)
    wd = make_weights(TINY_D, seed + 1, False, embed_std=0.06)
    return wv, wd


def describe(wl: Workload) -> dict:
    d = {k: v for k, v in asdict(wl).items() if k not in ("src", "max_tgt")}
    d["n_src"] = len(wl.src)
    return d
