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


# ---------------------------------------------------------------- near-tie classification helper
def test_decision_margins_hand_cases():
    """decision_margins on rows written by hand; every expected triple below was worked out on paper.

    Row values (index = token id):  [5.0, 4.0, 3.0, 2.0, 1.0, 0.0]
    """
    row = np.array([5.0, 4.0, 3.0, 2.0, 1.0, 0.0], np.float32)
    inf = float("inf")
    # beta = 2: the draft must have fewer than 2 entries above it.
    # draft = token 1 (4.0): one entry above -> accepted by rank; it flips when it drops to the best outsider, 3.0:
    # rank margin 1.0.  tau = 1.25: (5 - 4) - 1.25 = -0.25 -> tau margin 0.25.  top-1 minus top-2 = 1.0.
    assert O.decision_margins(row, 1, 2, 1.25) == pytest.approx((1.0, 0.25, 1.0))
    # draft = token 2 (3.0): two entries above -> rejected by rank; it flips when it reaches the 2nd value, 4.0:
    # rank margin 1.0.  tau = 1.75: (5 - 3) - 1.75 = +0.25 -> 0.25.
    assert O.decision_margins(row, 2, 2, 1.75) == pytest.approx((1.0, 0.25, 1.0))
    # a draft 0.25 above the (beta+1)-th value: beta = 3, values [5, 4, 3.25(draft), 3, ...]
    r2 = np.array([5.0, 4.0, 3.0, 3.25, 1.0], np.float32)
    assert O.decision_margins(r2, 3, 3, 10.0) == pytest.approx((0.25, 10.0 - 1.75, 1.0))
    # a draft 0.25 below the beta-th value: beta = 2, values [5, 4, 3.75(draft)]
    r3 = np.array([5.0, 3.75, 4.0], np.float32)
    assert O.decision_margins(r3, 1, 2, 0.0) == pytest.approx((0.25, 1.25, 1.0))
    # the draft is the top-1 itself with beta = 1: it flips when it falls to the runner-up
    assert O.decision_margins(row, 0, 1, 0.0) == pytest.approx((1.0, 0.0, 1.0))
    # two-way tie at the top: the argmax gap is 0; a tied draft is accepted under beta = 1 (no entry strictly above)
    # and sits exactly on the outsider's value (margin 0)
    r4 = np.array([2.0, 7.0, 7.0, 1.0], np.float32)
    assert O.decision_margins(r4, 2, 1, 0.0) == pytest.approx((0.0, 0.0, 0.0))
    # beta as large as the vocabulary: nothing can push the draft out by rank
    assert O.decision_margins(row, 5, 6, 2.0)[0] == inf
    # the bonus row has no draft: only the argmax gap applies
    assert O.decision_margins(row, None, 3, 1.0) == (inf, inf, 1.0)
    # consistency with the rule itself: moving the draft's logit across the rank margin flips accept_length
    for tok, beta in [(1, 2), (2, 2), (3, 3), (4, 1)]:
        m_rank, _, _ = O.decision_margins(row, tok, beta, 1e9)
        before = O.accept_length(row[None], [tok], beta, 1e9)
        for sign in (+1, -1):
            moved = row.copy(); moved[tok] += sign * (m_rank + 0.01)
            after = O.accept_length(moved[None], [tok], beta, 1e9)
            if (sign > 0) == (before == 0):        # towards the threshold: must flip
                assert after != before, (tok, beta, sign)
        short = row.copy(); short[tok] += (0.5 * m_rank if before == 0 else -0.5 * m_rank)
        assert O.accept_length(short[None], [tok], beta, 1e9) == before


# ---------------------------------------------------------------- where mode="bf16" rounds
def test_bf16_mode_rounds_exactly_the_contraction_operands(monkeypatch):
    """The bf16 mode may round only values that the CUDA path feeds to a tensor-core contraction as a bf16 operand:
    normalised activations, Q / K / V (cached and new), the un-normalised probabilities exp(s - max), the attention
    output, the feed-forward activation output, the encoder memory and the cross-attention K / V.  Logits and the
    residual stream are never rounded (Section 3.2: the rule is evaluated on the verifier's scores as computed).

    The rounding routine is replaced by a recorder; what it is handed is recognised by shape and by properties that
    follow from the definition of each quantity (unit LayerNorm gains: zero mean, unit variance rows; probabilities:
    row maximum exactly 1, all in (0, 1]; ReLU output: non-negative with zeros)."""
    import inspect
    d, H, F, V, L = 32, 2, 96, 50, 2
    dims = W.ModelDims(d, H, F, V, 1, L, 32)
    w = W.make_weights(dims, 5, False)
    for n in w:
        if ".ln" in n or "ln_f" in n:
            w[n] = np.ones_like(w[n]) if n.endswith(".g") else np.zeros_like(w[n])
    calls = []
    real = O.bf16_round

    def recorder(a):
        fn = next(f.function for f in inspect.stack()[2:] if f.function != "<genexpr>")     # the oracle function that rounds
        calls.append((fn, np.array(a, copy=True)))
        return real(a)

    monkeypatch.setattr(O, "bf16_round", recorder)
    m = O.model_from(dims, w, mode="bf16")
    S, j, T = 7, 3, 5
    src = list(range(4, 4 + S))

    def is_ln(a):
        return a.shape[-1] == d and np.allclose(a.mean(-1), 0, atol=1e-5) and np.allclose(a.var(-1), 1, atol=1e-3)

    def is_prob(a, keys):
        return a.shape[-1] == keys and np.all(a.max(-1) == 1.0) and np.all(a >= 0) and np.all(a <= 1)

    # ---- encoder: per layer LN, q, k, v, H probability tiles, attention output, LN, activation; then the memory
    mem = O.encode(m, src)
    kinds = [(f, a.shape) for f, a in calls]
    per_enc = [("encode", (S, d))] * 4 + [("attention", (S, S))] * H + [("encode", (S, d))] * 2 + [("ffn", (S, F))]
    assert kinds == per_enc * dims.enc_layers + [("encode", (S, d))]
    assert is_ln(calls[0][1]) and is_ln(calls[4 + H + 1][1]) and is_ln(calls[-1][1])
    assert all(is_prob(a, S) for f, a in calls if f == "attention")
    act = [a for f, a in calls if f == "ffn"][0]
    assert act.min() == 0.0 and (act == 0).mean() > 0.2
    assert np.array_equal(mem, real(calls[-1][1]))                       # the memory is the rounded final LayerNorm
    # ---- cross K / V once per decoder layer
    calls.clear()
    cache = O.new_cache(m, mem)
    assert [(f, a.shape) for f, a in calls] == [("new_cache", (S, d))] * (2 * L)
    # ---- a cached causal block of T rows after j cached positions
    O.decoder_rows(m, [1] + list(range(4, 4 + j - 1)), mem, True, cache)
    calls.clear()
    logits = O.decoder_rows(m, list(range(9, 9 + T)), mem, True, cache)
    kinds = [(f, a.shape) for f, a in calls]
    per_dec = ([("decoder_rows", (T, d))] * 4 + [("attention", (T, j + T))] * H + [("decoder_rows", (T, d))] * 3
               + [("attention", (T, S))] * H + [("decoder_rows", (T, d))] * 2 + [("ffn", (T, F))])
    assert kinds == per_dec * L + [("decoder_rows", (T, d))]
    n_per = len(per_dec)
    for l in range(L):
        blk = calls[l * n_per:(l + 1) * n_per]
        assert is_ln(blk[0][1]) and is_ln(blk[4 + H + 1][1]) and is_ln(blk[4 + H + 3 + H + 1][1])
        assert all(is_prob(a, j + T) for f, a in blk[4:4 + H])
        # causal: row i sees j + i + 1 keys, the rest carry probability exactly 0
        assert all(np.count_nonzero(a[i]) == j + i + 1 for f, a in blk[4:4 + H] for i in range(T))
        assert all(is_prob(a, S) for f, a in blk[4 + H + 3:4 + H + 3 + H])
        assert blk[-1][1].min() == 0.0
        # q, k, v handed over are linear images of the rounded LayerNorm output
        y = real(blk[0][1])
        for idx, nm in zip((1, 2, 3), "qkv"):
            assert np.allclose(blk[idx][1], y @ m.w[f"dec.{l}.self.{nm}.w"].T + m.w[f"dec.{l}.self.{nm}.b"], atol=1e-5)
        # the cache holds the rounded K / V of the block
        assert np.array_equal(cache.k[l][j:], real(blk[2][1])) and np.array_equal(cache.v[l][j:], real(blk[3][1]))
    assert is_ln(calls[-1][1])
    # logits never pass through the rounding: nothing V wide was recorded, and the result is the exact product
    assert all(a.shape[-1] != V for f, a in calls)
    assert np.array_equal(logits, real(calls[-1][1]) @ m.w["embed"].T)
    assert not np.array_equal(logits, real(logits))
    # with rounding switched off the same code path is the pure model: all rounding goes through this one routine
    monkeypatch.setattr(O, "bf16_round", lambda a: a)
    mp = O.model_from(dims, w, mode="pure")
    memp = O.encode(mp, src)
    assert np.array_equal(O.encode(m, src), memp)
    assert np.array_equal(O.decoder_rows(m, [1, 4, 5], memp, True), O.decoder_rows(mp, [1, 4, 5], memp, True))


# ---------------------------------------------------------------- the drafter's prefix-causal reading
def test_prefix_causal_mask_equals_torch_layers_and_causal_prefix(tiny):
    """decoder_rows(..., n_causal = p): positions below p attend causally, positions from p on see everything.
    (1) fp64 equality with torch.nn decoder layers given that boolean mask; (2) the rows below p equal the plain
    causal decoder on the prefix alone (they never see the [MASK] block, whatever follows them); (3) a one-layer
    decoder gives the same [MASK] rows under both readings (first-layer keys and values are functions of token and
    position only)."""
    wl, mv, md = tiny
    m = O.model_from(wl.drafter, md.w, dtype=np.float64)
    _, dec = _torch_stack(m)
    t = lambda a: torch.tensor(np.asarray(a, dtype=np.float64))
    src = wl.src[2]
    prefix, k = [BOS, 17, 230, 5, 999], 6
    tokens = prefix + [MASK] * k
    T, p = len(tokens), len(prefix)
    mem = O.encode(m, src)
    blocked = torch.zeros((T, T), dtype=torch.bool)
    for q in range(p):
        blocked[q, q + 1:] = True                       # True = not allowed, torch's convention
    with torch.no_grad():
        y = (t(m.w["embed"])[torch.tensor(tokens)] * math.sqrt(m.d_model) + t(m.w["pos_dec"])[:T])[None]
        for L in dec:
            y = L(y, t(mem)[None], tgt_mask=blocked)
        y = torch.nn.functional.layer_norm(y, (m.d_model,), t(m.w["dec.ln_f.g"]), t(m.w["dec.ln_f.b"]), 1e-5)
        ref = (y[0] @ t(m.w["embed"]).T).numpy()
    got = O.decoder_rows(m, tokens, mem, causal=False, n_causal=p)
    np.testing.assert_allclose(got, ref, rtol=0, atol=1e-10)
    np.testing.assert_allclose(got[:p], O.decoder_rows(m, prefix, mem, causal=True), rtol=0, atol=1e-12)
    np.testing.assert_allclose(got[:p], O.decoder_rows(m, prefix + [MASK] * 2, mem, causal=False, n_causal=p)[:p], rtol=0, atol=1e-12)
    full = O.decoder_rows(m, tokens, mem, causal=False)
    assert np.abs(full[p:] - got[p:]).max() > 1e-6 or m.dec_layers == 1     # the readings differ beyond one layer ...
    one = O.model_from(W.ModelDims(m.d_model, m.n_heads, m.d_ffn, m.vocab, m.enc_layers, 1, 64), m.w, dtype=np.float64)
    a = O.decoder_rows(one, tokens, mem, causal=False)
    b = O.decoder_rows(one, tokens, mem, causal=False, n_causal=p)
    np.testing.assert_allclose(a[p:], b[p:], rtol=0, atol=1e-12)            # ... and coincide on the [MASK] rows of one layer
    assert np.abs(a[:p] - b[:p]).max() > 1e-6


def test_prefix_causal_drafter_cache_equals_from_scratch(tiny):
    """draft(reading="prefix_causal") with a K/V cache carried across iterations gives the drafts of the uncached
    pass, for prefixes that grow by 1..k+1 tokens per iteration; the whole loop gives the same output either way, and
    at beta = 1, tau = 0 it is still greedy decoding (the drafter's reading cannot change a lossless rule's output)."""
    wl, mv, md = tiny
    src = wl.src[1]
    mem_d = O.encode(md, src)
    cache = O.new_cache(md, mem_d)
    committed = []
    rng = np.random.default_rng(5)
    for step in range(5):
        d_cached = O.draft(md, mem_d, committed, wl.k, BOS, MASK, "prefix_causal", cache)
        d_plain = O.draft(md, mem_d, committed, wl.k, BOS, MASK, "prefix_causal")
        assert d_cached == d_plain and cache.length == len(committed) + 1
        committed = committed + [int(t) for t in rng.integers(4, 1000, size=int(rng.integers(1, wl.k + 2)))]
    a, sa = O.specdec_generate(mv, md, src, 32, wl.k, 3, 1.0, BOS, EOS, MASK, drafter_reading="prefix_causal")
    b, sb = O.specdec_generate(mv, md, src, 32, wl.k, 3, 1.0, BOS, EOS, MASK, drafter_reading="prefix_causal", use_cache=False)
    assert a == b and sa.accepted == sb.accepted and sa.iterations == sb.iterations
    g, _ = O.specdec_generate(mv, md, src, 32, wl.k, 1, 0.0, BOS, EOS, MASK, drafter_reading="prefix_causal")
    assert g == O.greedy_decode(mv, src, 32, BOS, EOS)
