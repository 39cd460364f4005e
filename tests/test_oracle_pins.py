"""Pins for the CPU oracle: checks against what the paper and the mathematics fix.

None of these retype the oracle's own formulas: they use library routines
(torch.nn Transformer layers), closed-form constructions, brute force in
log-probability space, invariants, and the iteration structure of the paper's
worked example (tests/golden/case_study_structure.txt).
"""
import itertools
import math
import os

import numpy as np
import pytest
import torch

from oracle import specdec_oracle as O
from paper_2203_16487_b200 import workloads as W
from tests import designed

BOS, EOS, MASK = W.BOS_ID, W.EOS_ID, W.MASK_ID
GOLD = os.path.join(os.path.dirname(__file__), "golden")


@pytest.fixture(scope="module")
def tiny():
    wl = W.config1_tiny()
    mv = O.model_from(wl.verifier, W.make_weights(wl.verifier, wl.seed_verifier, False))
    md = O.model_from(wl.drafter, W.make_weights(wl.drafter, wl.seed_drafter, False))
    return wl, mv, md


# ---------------------------------------------------------------- model definition
def test_parameter_count_matches_memory_table():
    """Appendix memory table: the AR model's weights take 232.4 MB in fp32.  A 6+6,
    512/2048 Transformer with one shared 32768x512 table, biases and LN, no
    position parameters has 60,917,760 parameters = 232.38 MiB."""
    w = W.make_weights(W.ModelDims(512, 8, 2048, 32768, 6, 6, 8), 0, False)
    n = W.count_params(w)
    assert n == 60_917_760
    assert abs(n * 4 / 2 ** 20 - 232.4) < 0.05
    wd = W.make_weights(W.ModelDims(512, 8, 2048, 32768, 12, 2, 8), 0, False)
    assert W.count_params(wd) == 63_015_936


def _torch_stack(m: O.Model, act="relu"):
    """The same weights loaded into torch.nn pre-LN Transformer layers (fp64)."""
    d, H, F = m.d_model, m.n_heads, m.d_ffn
    t = lambda a: torch.tensor(np.asarray(a, dtype=np.float64))

    def load_attn(mod, p):
        mod.in_proj_weight.data = torch.cat([t(m.w[f"{p}.{n}.w"]) for n in "qkv"])
        mod.in_proj_bias.data = torch.cat([t(m.w[f"{p}.{n}.b"]) for n in "qkv"])
        mod.out_proj.weight.data = t(m.w[p + ".o.w"])
        mod.out_proj.bias.data = t(m.w[p + ".o.b"])

    def load_common(layer, p, norm2):
        layer.linear1.weight.data = t(m.w[p + ".ffn.w1"]); layer.linear1.bias.data = t(m.w[p + ".ffn.b1"])
        layer.linear2.weight.data = t(m.w[p + ".ffn.w2"]); layer.linear2.bias.data = t(m.w[p + ".ffn.b2"])
        layer.norm1.weight.data = t(m.w[p + ".ln1.g"]); layer.norm1.bias.data = t(m.w[p + ".ln1.b"])
        norm2.weight.data = t(m.w[p + ".ln2.g"]); norm2.bias.data = t(m.w[p + ".ln2.b"])

    enc, dec = [], []
    for l in range(m.enc_layers):
        L = torch.nn.TransformerEncoderLayer(d, H, F, 0.0, activation=act, norm_first=True, batch_first=True).double()
        load_attn(L.self_attn, f"enc.{l}.self"); load_common(L, f"enc.{l}", L.norm2)
        enc.append(L.eval())
    for l in range(m.dec_layers):
        L = torch.nn.TransformerDecoderLayer(d, H, F, 0.0, activation=act, norm_first=True, batch_first=True).double()
        load_attn(L.self_attn, f"dec.{l}.self"); load_attn(L.multihead_attn, f"dec.{l}.cross")
        load_common(L, f"dec.{l}", L.norm3)
        L.norm2.weight.data = t(m.w[f"dec.{l}.ln_cross.g"]); L.norm2.bias.data = t(m.w[f"dec.{l}.ln_cross.b"])
        dec.append(L.eval())
    return enc, dec


@pytest.mark.parametrize("causal,act", [(True, "relu"), (False, "relu"), (True, "gelu"), (False, "gelu")])
def test_stack_equals_torch_library_layers(tiny, causal, act):
    """Encoder memory and decoder logits equal torch.nn's pre-LN Transformer layers
    fed the same weights (library routine as the independent definition), for both
    feed-forward activations (torch's "gelu" is the exact erf form)."""
    wl, mv, _ = tiny
    m = O.model_from(wl.verifier, mv.w, dtype=np.float64, act=act)
    enc, dec = _torch_stack(m, act)
    t = lambda a: torch.tensor(np.asarray(a, dtype=np.float64))
    src = wl.src[0]
    tokens = [BOS, 17, 230, 5, 999, MASK, MASK]
    with torch.no_grad():
        x = t(m.w["embed"])[torch.tensor(src, dtype=torch.long)] * math.sqrt(m.d_model) + t(m.w["pos_enc"])[:len(src)]
        x = x[None]
        for L in enc:
            x = L(x)
        mem = torch.nn.functional.layer_norm(x, (m.d_model,), t(m.w["enc.ln_f.g"]), t(m.w["enc.ln_f.b"]), 1e-5)
        y = t(m.w["embed"])[torch.tensor(tokens)] * math.sqrt(m.d_model) + t(m.w["pos_dec"])[:len(tokens)]
        y = y[None]
        T = len(tokens)
        mask = torch.triu(torch.full((T, T), float("-inf"), dtype=torch.float64), 1) if causal else None
        for L in dec:
            y = L(y, mem, tgt_mask=mask)
        y = torch.nn.functional.layer_norm(y, (m.d_model,), t(m.w["dec.ln_f.g"]), t(m.w["dec.ln_f.b"]), 1e-5)
        logits_ref = (y[0] @ t(m.w["embed"]).T).numpy()
    mem_o = O.encode(m, src)
    np.testing.assert_allclose(mem_o, mem[0].numpy(), rtol=0, atol=1e-10)
    logits = O.decoder_rows(m, tokens, mem_o, causal)
    np.testing.assert_allclose(logits, logits_ref, rtol=0, atol=1e-10)
    # and the fp32 oracle agrees with its fp64 self to rounding noise
    m32 = O.model_from(wl.verifier, mv.w, act=act)
    l32 = O.decoder_rows(m32, tokens, O.encode(m32, src), causal)
    assert np.abs(l32 - logits_ref).max() < 2e-5


def test_gelu_closed_form_values():
    """x * Phi(x): Phi(1) = 0.841344746068543 (standard normal table), odd part x / 2, limits 0 and x."""
    x = np.array([0.0, 1.0, -1.0, 2.0, 30.0, -30.0], dtype=np.float64)
    g = O.gelu(x)
    assert g[0] == 0.0
    assert abs(g[1] - 0.841344746068543) < 1e-15 and abs(g[2] + (1.0 - 0.841344746068543)) < 1e-15
    assert abs(g[3] - 2.0 * 0.977249868051821) < 1e-14
    assert g[4] == 30.0 and g[5] == 0.0
    np.testing.assert_allclose(O.gelu(x) - O.gelu(-x), x, rtol=0, atol=1e-14)       # gelu(x) - gelu(-x) = x
    assert O.gelu(x.astype(np.float32)).dtype == np.float32


def test_every_weight_is_used(tiny):
    """Perturbing any single weight tensor changes the verifier logits (no dropped term)."""
    wl, mv, _ = tiny
    src, tokens = wl.src[1], [BOS, 40, 41, 42]
    base = O.decoder_rows(mv, tokens, O.encode(mv, src), True)
    rng = np.random.default_rng(0)
    for name in mv.w:
        if name.endswith(".k.b"):
            continue      # a key bias shifts every score of a query equally: softmax cancels it
        w2 = dict(mv.w)
        w2[name] = mv.w[name] + rng.standard_normal(mv.w[name].shape).astype(np.float32) * 0.05
        m2 = O.model_from(wl.verifier, w2)
        out = O.decoder_rows(m2, tokens, O.encode(m2, src), True)
        assert np.abs(out - base).max() > 1e-7, name


def test_bf16_round_matches_torch():
    rng = np.random.default_rng(3)
    a = np.concatenate([rng.standard_normal(5000).astype(np.float32) * 3,
                        np.array([1.00390625, 1.01171875, -1.00390625, 0.0, 65504.0], np.float32)])
    ref = torch.tensor(a).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(O.bf16_round(a), ref)
    assert np.array_equal(W.round_to_bf16(a), ref)


# ---------------------------------------------------------------- acceptance rule (Eq. 7-8)
def _bruteforce_accept(rows, drafts, beta, tau):
    """Eq. 7-8 applied literally in log-probability space (float64): sort, take the
    beta-th ranked log-prob, compare; stop at the first failure."""
    a = 0
    for i, tok in enumerate(drafts):
        l = rows[i].astype(np.float64)
        logp = l - (np.log(np.sum(np.exp(l - l.max()))) + l.max())
        ranked = sorted(logp.tolist(), reverse=True)
        c1 = logp[tok] >= ranked[beta - 1]
        c2 = (ranked[0] - logp[tok]) <= tau
        if c1 and c2:
            a += 1
        else:
            break
    return a


def test_accept_rule_bruteforce_tiny_vocab():
    rng = np.random.default_rng(5)
    n = 0
    for V in (2, 3, 5, 8, 16):
        for trial in range(120):
            k = int(rng.integers(1, 6))
            # logits on a 1/4 grid: exactly representable, so ties are engineered and the
            # log-prob form is compared where its own rounding cannot decide (margin >= 0.25)
            rows = rng.integers(-8, 9, size=(k + 1, V)).astype(np.float32) / 4
            drafts = rng.integers(0, V, size=k).tolist()
            for beta in range(1, V + 1):
                for tau in (0.0, 0.3, 0.6, 1.1, 2.6, 100.0):
                    assert O.accept_length(rows, drafts, beta, tau) == _bruteforce_accept(rows, drafts, beta, tau)
                    n += 1
    assert n > 10000


def test_accept_hand_cases():
    """Worked by hand.  Row 0 = [2, 1, 0, -1]; row 1 = [0, 0, 3, 2.5]."""
    rows = np.array([[2, 1, 0, -1], [0, 0, 3, 2.5], [5, 0, 0, 0]], np.float32)
    assert O.verify(rows, [0, 2], 1, 0.0) == (2, 0)       # both top-1 -> bonus token from row 2
    assert O.verify(rows, [1, 2], 1, 0.0) == (0, 0)       # rank 2 rejected by strict rule
    assert O.verify(rows, [1, 2], 2, 1.0) == (2, 0)       # rank 2, gap 1.0 <= tau (inclusive)
    assert O.verify(rows, [1, 2], 2, 0.99) == (0, 0)      # gap 1.0 > 0.99
    assert O.verify(rows, [1, 3], 2, 1.0) == (2, 0)       # row 1: rank 2, gap 0.5
    # row 1 sorted: 3, 2.5, 0, 0; token 0 has 2 strictly greater -> ties the 3rd value -> inside top-3
    assert O.accept_length(rows, [1, 0], 3, 10.0) == 2
    assert O.accept_length(rows, [1, 0], 2, 10.0) == 1    # 2 strictly greater > beta-1 = 1


def test_accept_monotone_and_limits():
    rng = np.random.default_rng(9)
    V, k = 50, 12
    for trial in range(60):
        rows = (rng.standard_normal((k + 1, V)) * 3).astype(np.float32)
        top = rows.argmax(axis=1)
        drafts = [int(top[i]) if rng.random() < 0.6 else int(rng.integers(0, V)) for i in range(k)]
        betas, taus = [1, 2, 3, 5, 10, V], [0.0, 0.5, 1.0, 3.0, 10.0, np.inf]
        grid = np.array([[O.accept_length(rows, drafts, b, t) for t in taus] for b in betas])
        assert ((grid >= 0) & (grid <= k)).all()
        assert (np.diff(grid, axis=0) >= 0).all() and (np.diff(grid, axis=1) >= 0).all()
        assert grid[-1, -1] == k                                  # beta = V and tau = inf accept everything
        # tau = inf is the pure top-beta rule; beta = V is the pure gap rule
        for bi, b in enumerate(betas):
            pure = 0
            for i, tok in enumerate(drafts):
                if sorted(rows[i].tolist(), reverse=True).index(rows[i][tok]) < b:
                    pure += 1
                else:
                    break
            assert grid[bi, -1] == pure


# ---------------------------------------------------------------- decoding
def test_block_parallel_equals_sequential_and_cache(tiny):
    """Row r of the (k+1)-row pass = the single-row output after feeding the same
    inputs one at a time; cached = from scratch (Section 2, 'verified in parallel')."""
    wl, mv, _ = tiny
    src = wl.src[2]
    mem = O.encode(mv, src)
    committed, drafts = [5, 77, 300], [9, 8, 7, 600, 2, 31]
    scratch = O.verify_rows(mv, mem, committed, drafts, BOS)
    cache = O.new_cache(mv, mem)
    O.decoder_rows(mv, [BOS] + committed[:-1], mem, True, cache)
    cached = O.verify_rows(mv, mem, committed, drafts, BOS, cache)
    assert np.abs(scratch - cached).max() < 2e-5
    cache2 = O.new_cache(mv, mem)
    seq = [O.decoder_rows(mv, [t], mem, True, cache2)[0] for t in [BOS] + committed + drafts]
    assert np.abs(np.stack(seq[len(committed):]) - scratch).max() < 2e-5


@pytest.mark.parametrize("kind", ["drafter", "random", "all_eos", "greedy", "greedy_then_wrong"])
def test_strict_verification_equals_greedy(tiny, kind):
    """beta=1, tau=0 reproduces greedy AR decoding token for token, whatever is drafted (Section 3.2)."""
    wl, mv, md = tiny
    rng = np.random.default_rng(1)
    for s, src in enumerate(wl.src[:3]):
        g = O.greedy_decode(mv, src, 32, BOS, EOS)
        assert g == O.greedy_decode(mv, src, 32, BOS, EOS, use_cache=False)
        fn = None
        if kind == "random":
            fn = lambda c, k: rng.integers(0, wl.verifier.vocab, size=k).tolist()
        elif kind == "all_eos":
            fn = lambda c, k: [EOS] * k
        elif kind == "greedy":
            fn = lambda c, k: (g[len(c):len(c) + k] + [7] * k)[:k]
        elif kind == "greedy_then_wrong":
            fn = lambda c, k: (g[len(c):len(c) + 3] + [11] * k)[:k]
        out, st = O.specdec_generate(mv, md, src, 32, wl.k, 1, 0.0, BOS, EOS, MASK, draft_fn=fn,
                                     use_cache=(s != 1))
        assert out == g
        assert st.emitted == len(out) and st.iterations <= len(out)      # >= 1 token per iteration
        if kind == "greedy":
            assert st.iterations == math.ceil(len(g) / (wl.k + 1))       # a = k every full block


def test_eos_truncation_and_invariants(tiny):
    wl, mv, md = tiny
    src = wl.src[0]
    g = O.greedy_decode(mv, src, 32, BOS, eos=-1)
    eos = g[5]                                        # a token the greedy decode is known to emit
    first = g.index(eos)
    g2 = O.greedy_decode(mv, src, 32, BOS, eos)
    assert g2 == g[:first + 1]
    fn = lambda c, k: (g[len(c):len(c) + k] + [7] * k)[:k]            # drafts run past the EOS
    out, st = O.specdec_generate(mv, md, src, 32, wl.k, 1, 0.0, BOS, eos, MASK, draft_fn=fn)
    assert out == g2 and out.count(eos) == 1 and out[-1] == eos
    out, st = O.specdec_generate(mv, md, src, 7, wl.k, 3, 1.0, BOS, -1, MASK)
    assert len(out) == 7


def test_relaxed_rule_trends(tiny):
    """Per-step accepted length never decreases with beta or tau on the same context (Table 4 trend)."""
    wl, mv, md = tiny
    src = wl.src[3]
    mem = O.encode(mv, src)
    g = O.greedy_decode(mv, src, 20, BOS, -1)
    rng = np.random.default_rng(2)
    for j in (0, 3, 9):
        drafts = g[j:j + 8]
        rows = O.verify_rows(mv, mem, g[:j], drafts, BOS)
        # replace two drafts by the verifier's 2nd / 4th ranked token
        order = np.argsort(-rows, axis=1, kind="stable")
        drafts[2], drafts[5] = int(order[2][1]), int(order[5][3])
        rows = O.verify_rows(mv, mem, g[:j], drafts, BOS)
        prev = -1
        for beta, tau in [(1, 0.0), (2, 0.5), (2, 5.0), (4, 5.0), (1000, np.inf)]:
            a = O.accept_length(rows, drafts, beta, tau)
            assert a >= prev
            prev = a
        assert O.accept_length(rows, drafts, 1, 0.0) == 2
        assert O.accept_length(rows, drafts, 1000, np.inf) == 8


# ---------------------------------------------------------------- worked example + closed form
def _read_case():
    it, meta = [], {}
    for line in open(os.path.join(GOLD, "case_study_structure.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        p = line.split()
        if p[0].isdigit():
            it.append(tuple(int(x) for x in p))
        else:
            meta[p[0]] = float(p[1])
    return meta, it


@pytest.mark.parametrize("rule", ["paper", "strict"])
def test_case_study_structure_on_closed_form_model(rule):
    """A model pair whose outputs are known in closed form is laid out like the paper's
    worked example; the oracle must reproduce that example's iteration structure."""
    meta, iters = _read_case()
    k = int(meta["k"])
    beta, tau = (int(meta["beta"]), meta["tau"]) if rule == "paper" else (1, 0.0)
    dv, wv, dd, wd, T, D, src = designed.case_study_pair()
    mv, md = O.model_from(dv, wv), O.model_from(dd, wd)
    # closed form: logits depend on (token, position) only, so greedy = T and drafts = D
    assert O.greedy_decode(mv, src, 40, BOS, EOS) == T[1:]
    mem_d = O.encode(md, src)
    assert O.draft(md, mem_d, T[1:4], k, BOS, MASK) == [D[p] for p in range(4, 4 + k)]
    out, st = O.specdec_generate(mv, md, src, 40, k, beta, tau, BOS, EOS, MASK, keep_trace=True)
    assert out == T[1:] and len(out) == int(meta["result_len_with_eos"])
    assert st.iterations == len(iters)
    n = 0
    for (it, n_rows, a_exp, emit_exp, fin), (drafts, a, bif) in zip(iters, st.trace):
        assert len(drafts) + 1 == n_rows
        assert a == a_exp
        emitted = drafts[:a] + [bif]
        if EOS in emitted:                          # everything after the end token is dropped
            emitted = emitted[:emitted.index(EOS) + 1]
        assert len(emitted) == emit_exp
        assert (EOS in emitted) == bool(fin)
        assert out[n:n + emit_exp] == emitted
        n += emit_exp
    assert n == len(out)
    # iteration 2: the drafted EOS at the last position is replaced by the verifier's token
    assert st.trace[1][0][k - 1] == EOS and st.trace[1][2] == T[13]


def test_relaxed_rule_accepts_near_top_token():
    """A draft whose verifier logit is 0.9x the top-1's (gap 0.32, rank 2) is kept by
    (beta=3, tau=1) and replaced under strict matching."""
    dv, wv, dd, wd, T, D, src = designed.case_study_pair(near_top_at=5)
    mv, md = O.model_from(dv, wv), O.model_from(dd, wd)
    mem = O.encode(mv, src)
    rows = O.verify_rows(mv, mem, T[1:4], [D[p] for p in range(4, 14)], BOS)
    top, u = rows[1][T[5]], rows[1][D[5]]
    assert abs(top - 0.05 * 64) < 0.05 and abs(u - 0.9 * top) < 1e-3      # closed-form logits
    strict, _ = O.specdec_generate(mv, md, src, 40, 10, 1, 0.0, BOS, EOS, MASK)
    relaxed, _ = O.specdec_generate(mv, md, src, 40, 10, 3, 1.0, BOS, EOS, MASK)
    tight, _ = O.specdec_generate(mv, md, src, 40, 10, 3, 0.3, BOS, EOS, MASK)
    assert strict == T[1:] and tight == T[1:]
    assert relaxed[4] == D[5] and relaxed[:4] == T[1:5]


def test_batch_of_independent_sequences_and_modes(tiny):
    """bf16-operand mode stays close to pure fp32 (it only rounds operands)."""
    wl, mv, md = tiny
    wq = {n: (W.round_to_bf16(a) if a.ndim >= 2 and not n.startswith("pos_") else a) for n, a in mv.w.items()}
    mp, mb = O.model_from(wl.verifier, wq), O.model_from(wl.verifier, wq, mode="bf16")
    src = wl.src[0]
    lp = O.decoder_rows(mp, [BOS, 4, 5, 6], O.encode(mp, src), True)
    lb = O.decoder_rows(mb, [BOS, 4, 5, 6], O.encode(mb, src), True)
    assert 0 < np.abs(lp - lb).max() < 2e-2
