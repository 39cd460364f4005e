"""GPU parity at the full sizes of the workload recipes (configs 3, 4, 5), on sampled outputs.

The oracle cannot follow 128 sequences for a hundred iterations inside a test, so at full size the
CUDA path runs the whole batch and a few sampled sequences are compared with the oracle's batch-1
result; lock-step checks cover every decision on a few sequences.  Tolerances as in
test_gpu_parity.py (bf16 handles: decisions bit-exact outside 1e-3 margins).
"""
import json
import os

import numpy as np
import pytest
import torch

from oracle import specdec_oracle as O
from paper_2203_16487_b200 import workloads as W
from tests import lockstep

pytestmark = pytest.mark.gpu
BOS, EOS, MASK = W.BOS_ID, W.EOS_ID, W.MASK_ID


@pytest.fixture(scope="module")
def base():
    from paper_2203_16487_b200 import binding
    wv = W.make_weights(W.BASE_V, 1001, True)
    wd = W.make_weights(W.BASE_D, 1002, True)
    mv, md = O.model_from(W.BASE_V, wv, mode="bf16"), O.model_from(W.BASE_D, wd, mode="bf16")
    return binding, wv, wd, mv, md


def _prefix_match(a, b):
    n = 0
    for x, y in zip(a, b):
        if x != y:
            break
        n += 1
    return n


GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "oracle_outputs.json")))


def _check_against_oracle_tokens(binding, wv, wd, mv, md, dims_v, dims_d, src, max_tgt, beta, tau, got, ref, counts):
    """got == ref, or the first differing decision is a near-tie by the oracle's own margins (< 1e-3): then the
    sequence is re-run in lock-step (every decision compared, the oracle's committed on both sides) and must be clean."""
    counts["sequences"] += 1
    if got == ref:
        return
    sd1 = binding.SpecDec(dims_v, wv, dims_d, wd, k_max=25, max_batch=1, max_src=len(src), max_tgt=max_tgt, bf16=True)
    rep = lockstep.run(sd1, mv, md, [src], [max_tgt], 25, beta, tau, margin=1e-3)
    sd1.close()
    counts["near_tie_sequences"] += 1
    counts["near_ties"] += rep.draft_near_ties + rep.verify_near_ties
    assert rep.ok and rep.draft_near_ties + rep.verify_near_ties > 0, (beta, tau, _prefix_match(got, ref), rep.notes[:3])


def test_config3_batch32_all_nine_cells(base):
    """Config 3, batch 32: every (beta, tau) in {1,3,5} x {0,1,3}; eight sequences per cell compared over their whole
    length with the oracle's batch-1 output (tests/golden/oracle_outputs.json, written by the oracle alone)."""
    binding, wv, wd, mv, md = base
    wl = W.config3_batched(32)
    smax, tmax = max(len(s) for s in wl.src), max(wl.max_tgt)
    sd = binding.SpecDec(W.BASE_V, wv, W.BASE_D, wd, k_max=25, max_batch=32, max_src=smax, max_tgt=tmax, bf16=True)
    src, lens = W.pad_batch(wl.src)
    counts = {"sequences": 0, "near_tie_sequences": 0, "near_ties": 0}
    idx = sorted(int(i) for i, c in GOLD["config3"]["cells"].items() if len(c) == 9)
    assert len(idx) >= 8
    for beta in (1, 3, 5):
        for tau in (0.0, 1.0, 3.0):
            out, n, st = sd.generate(src, lens, wl.max_tgt, 25, beta, tau)
            out, n = out.cpu().numpy(), n.cpu().numpy()
            assert st["emitted"] == int(n.sum()) and (n <= np.array(wl.max_tgt)).all() and (n >= 1).all()
            assert st["iterations"] <= tmax and st["seq_iterations"] <= st["emitted"]      # >= 1 token per sequence-iteration
            for b in idx:
                ref = GOLD["config3"]["cells"][str(b)][f"{beta},{tau:g}"]
                _check_against_oracle_tokens(binding, wv, wd, mv, md, W.BASE_V, W.BASE_D, wl.src[b], wl.max_tgt[b], beta, tau,
                                             out[b, :n[b]].tolist(), ref, counts)
    print("config 3, batch 32:", counts)
    assert counts["sequences"] == 9 * len(idx)
    sd.close()


@pytest.mark.parametrize("pair", [0, 1])
def test_config3_batch128_sampled_sequences(base, pair):
    """Config 3, batch 128 at (beta, tau) = (3, 1): twelve sequences over their whole length against the oracle, and
    batch invariance on the device.  pair = 1: the wide GEMMs over many rows (QKV, FFN1, vocabulary, encoder K/V) run as
    two-SM tiles, and every LayerNorm is applied inside the residual GEMM before it (clusters of four CTAs per row tile)."""
    binding, wv, wd, mv, md = base
    wl = W.config3_batched(128)
    smax, tmax = max(len(s) for s in wl.src), max(wl.max_tgt)
    sd = binding.SpecDec(W.BASE_V, wv, W.BASE_D, wd, k_max=25, max_batch=128, max_src=smax, max_tgt=tmax, bf16=True)
    sd.set_option("pair", pair)
    sd.set_option("ln_fuse", pair)
    sd.set_option("attn_rs", 2 if pair else 1)             # 2: attention scores stay in registers wherever the keys allow
    src, lens = W.pad_batch(wl.src)
    out, n, st = sd.generate(src, lens, wl.max_tgt, 25, 3, 1.0)
    out, n = out.cpu().numpy(), n.cpu().numpy()
    assert st["emitted"] == int(n.sum()) and (n <= np.array(wl.max_tgt)).all() and (n >= 1).all()
    counts = {"sequences": 0, "near_tie_sequences": 0, "near_ties": 0}
    idx = sorted(int(i) for i in GOLD["config3"]["cells"])
    assert len(idx) >= 12
    for b in idx:
        ref = GOLD["config3"]["cells"][str(b)]["3,1"]
        _check_against_oracle_tokens(binding, wv, wd, mv, md, W.BASE_V, W.BASE_D, wl.src[b], wl.max_tgt[b], 3, 1.0,
                                     out[b, :n[b]].tolist(), ref, counts)
    print("config 3, batch 128:", counts)
    # batch invariance on the device: the same sequences decoded alone
    order = np.argsort([len(s) for s in wl.src])
    for b in (int(order[1]), int(order[-2])):
        o1, n1, _ = sd.generate(wl.src[b][None], [len(wl.src[b])], [wl.max_tgt[b]], 25, 3, 1.0)
        assert o1[0, :int(n1[0])].cpu().tolist() == out[b, :n[b]].tolist()
    sd.close()


def test_config2_whole_sentences_free_running_and_scripted(base):
    """Config 2 (batch 1): specdec_generate on eight whole sentences against the oracle's free-running output, and the
    scripted-acceptance run that bench.py times (drafts replaced by the greedy continuation with a rejected token every
    Geometric(mean 6) positions) against the oracle's specdec_generate with the same script."""
    binding, wv, wd, mv, md = base
    wl = W.config2_translation()
    idx = sorted(int(i) for i in GOLD["config2"]["natural"])
    assert len(idx) >= 8
    smax, tmax = max(len(wl.src[i]) for i in idx), max(wl.max_tgt[i] for i in idx)
    sd = binding.SpecDec(W.BASE_V, wv, W.BASE_D, wd, k_max=25, max_batch=1, max_src=smax, max_tgt=tmax, bf16=True)
    counts = {"sequences": 0, "near_tie_sequences": 0, "near_ties": 0}
    rng = np.random.default_rng(7)
    accepted = 0
    for i in idx:
        s, mt = wl.src[i], wl.max_tgt[i]
        sd.set_draft_script(None)
        out, n, st = sd.generate(s[None], [len(s)], [mt], 25, 3, 1.0)
        _check_against_oracle_tokens(binding, wv, wd, mv, md, W.BASE_V, W.BASE_D, s, mt, 3, 1.0,
                                     out[0, :int(n[0])].cpu().tolist(), GOLD["config2"]["natural"][str(i)], counts)
        # scripted acceptance: the greedy continuation (the oracle's) with rejected tokens sprinkled in
        greedy = np.array(GOLD["config2"]["greedy"][str(i)], np.int32)
        script = np.full(tmax + 25, -1, np.int32)
        script[:len(greedy)] = greedy
        p = int(rng.geometric(1.0 / 6.0)) - 1
        while p < len(script):
            bad = int(rng.integers(W.N_SPECIAL, W.BASE_V.vocab))
            if p < len(greedy) and bad == greedy[p]:
                bad = W.N_SPECIAL + (bad + 1 - W.N_SPECIAL) % (W.BASE_V.vocab - W.N_SPECIAL)
            script[p] = bad
            p += int(rng.geometric(1.0 / 6.0))
        ref, ost = O.specdec_generate(mv, md, s, mt, 25, 3, 1.0, BOS, EOS, MASK, script=script)
        sd.set_draft_script(script[None])
        out, n, st = sd.generate(s[None], [len(s)], [mt], 25, 3, 1.0)
        got = out[0, :int(n[0])].cpu().tolist()
        assert got == ref, (i, _prefix_match(got, ref))
        assert (st["accepted"], st["seq_iterations"], st["emitted"]) == (ost.accepted, ost.iterations, len(ref))
        assert ref == greedy.tolist()                          # greedy drafts are accepted, rejected ones replaced by the top-1
        accepted += ost.accepted
    print("config 2:", counts, "scripted accepted drafts:", accepted)
    assert accepted > 4 * len(idx)                             # the script really exercises acceptance (a > 0)
    sd.close()


def test_config4_long_sources(base):
    binding, wv, wd, mv, md = base
    wl = W.config4_summarization()
    smax = max(len(s) for s in wl.src)
    sd = binding.SpecDec(W.BASE_V, wv, W.BASE_D, wd, k_max=25, max_batch=8, max_src=smax, max_tgt=128, bf16=True)
    # every decision of two long-source sequences for a few iterations (cross-attention over 300-512 keys)
    rep = lockstep.run(sd, mv, md, wl.src[:2], [128, 128], 25, 3, 1.0, margin=1e-3, check_logits_every=2, max_iters=3)
    print(rep.iterations, rep.draft_near_ties, rep.verify_near_ties, rep.max_logit_err, rep.max_stat_err, rep.notes[:3])
    assert rep.ok, rep.notes
    assert rep.max_logit_err < 2e-2
    # the whole batch of 8, full length; one sampled sequence against the oracle
    src, lens = W.pad_batch(wl.src)
    out, n, st = sd.generate(src, lens, wl.max_tgt, 25, 3, 1.0)
    n = n.cpu().numpy()
    assert st["emitted"] == int(n.sum()) and (n >= 1).all() and (n <= 128).all()
    out = out.cpu().numpy()
    for b in range(8):                                          # a sequence shorter than its budget ended on [EOS]
        assert n[b] == 128 or out[b, n[b] - 1] == EOS
    ref, _ = O.specdec_generate(mv, md, wl.src[3], 12, 25, 3, 1.0, BOS, EOS, MASK)
    assert out[3, :12].tolist() == ref
    sd.close()


@pytest.mark.parametrize("B,k,prefix", [(2, 5, 64), (2, 50, 64), (2, 25, 256), (2, 10, 0), (8, 25, 256), (8, 50, 64),
                                        (128, 25, 256), (128, 50, 64)])
def test_config5_verify_step_with_scripted_rejections(base, B, k, prefix):
    """Drafts = the oracle verifier's greedy continuation with one substitution at position r ~ Geometric(mean 6):
    the accepted length must be min(r - 1, k) and the bifurcation token the oracle's top-1 there.  Default options at
    every batch; at batch 8 / 128 four sampled sequences carry oracle drafts (the others verify placeholder drafts)."""
    binding, wv, wd, mv, md = base
    S = 64
    wl = W.config5_microbench(B, S)
    prefixes, rej = W.config5_prefix_and_rejections(B, prefix)
    sd = binding.SpecDec(W.BASE_V, wv, W.BASE_D, wd, k_max=50, max_batch=B, max_src=S, max_tgt=prefix + 52, bf16=True)
    src, lens = W.pad_batch(wl.src)
    sd.encode(src, lens, None)
    done = 0
    pre = np.stack(prefixes) if prefix else np.zeros((B, 0), np.int32)
    kb = 25
    while done < prefix:                                  # build the prefix through verify + commit(keep, next)
        c = min(kb, prefix - done - 1)
        block = np.zeros((B, kb), np.int32); block[:, :c] = pre[:, done:done + c]
        sd.verify(block, 1, 0.0)
        sd.commit(np.full(B, c, np.int32), pre[:, done + c])
        done += c + 1
    sample = list(range(B)) if B <= 4 else [0, B // 3, (2 * B) // 3, B - 1]
    drafts = np.full((B, k), 5, np.int32)                 # placeholder drafts for the sequences that are not sampled
    expect = {}
    for b in sample:
        mem = O.encode(mv, wl.src[b])
        cache = O.new_cache(mv, mem)
        committed = pre[b].tolist()
        if committed:
            O.decoder_rows(mv, [BOS] + committed[:-1], mem, True, cache)
        g = []
        for _ in range(k):                                # oracle greedy continuation, one token at a time
            row = O.decoder_rows(mv, [(committed + g)[-1] if committed + g else BOS], mem, True, cache)[-1]
            g.append(int(np.argmax(row)))
        d = list(g)
        r = int(rej[b])
        cache.truncate(len(committed))
        if r <= k:
            rows = O.verify_rows(mv, mem, committed, g, BOS, cache)
            cache.truncate(len(committed))
            d[r - 1] = int(np.argmin(rows[r - 1]))       # the lowest-logit token: rejected under every beta < V
        drafts[b] = d
        rows = O.verify_rows(mv, mem, committed, d, BOS, cache)
        a, t = O.verify(rows, d, 3, 1.0)
        assert a == min(r - 1, k)
        expect[b] = (a, t)
    acc, bif = sd.verify(drafts, 3, 1.0)
    acc, bif = acc.cpu().tolist(), bif.cpu().tolist()
    assert {b: (acc[b], bif[b]) for b in sample} == expect
    assert all(0 <= a <= k for a in acc)
    sd.close()


def test_shape_variants_12_2_verifier_and_narrow_heads():
    """The paper also accelerates a 12+2 Transformer-base verifier (Table 1, lower half); and a bf16 model whose
    heads are 32 wide exercises the tensor-core GEMM together with the warp-per-row attention."""
    from paper_2203_16487_b200 import binding
    v122 = W.ModelDims(512, 8, 2048, 32768, 12, 2, 1024)
    wv, wd = W.make_weights(v122, 2001, True), W.make_weights(W.BASE_D, 1002, True)
    mv, md = O.model_from(v122, wv, mode="bf16"), O.model_from(W.BASE_D, wd, mode="bf16")
    wl = W.config2_translation(2)
    sd = binding.SpecDec(v122, wv, W.BASE_D, wd, k_max=10, max_batch=2, max_src=40, max_tgt=48, bf16=True)
    rep = lockstep.run(sd, mv, md, wl.src, [20, 20], 10, 3, 1.0, margin=1e-3, check_logits_every=3, max_iters=5)
    assert rep.ok, rep.notes
    assert rep.max_logit_err < 2e-2
    sd.close()
    nv = W.ModelDims(128, 4, 256, 3000, 2, 2, 128)            # heads of 32
    nd = W.ModelDims(128, 4, 256, 3000, 2, 1, 128)
    wv, wd = W.make_weights(nv, 61, True), W.make_weights(nd, 62, True)
    mv, md = O.model_from(nv, wv, mode="bf16"), O.model_from(nd, wd, mode="bf16")
    rng = np.random.default_rng(3)
    srcs = [W.zipf_ids(rng, n, 3000) for n in (9, 30, 17)]
    sd = binding.SpecDec(nv, wv, nd, wd, k_max=6, max_batch=3, max_src=32, max_tgt=20, bf16=True)
    # a vocabulary of 3000 is 24 tiles of 128 = 48 half-tile statistics per row but only 47 tiles of 64: the table of
    # partial row statistics once was a slot per row too small for it; the red-zone check after every call sees that
    sd.set_option("debug_checks", 1)
    rep = lockstep.run(sd, mv, md, srcs, [20, 11, 16], 6, 2, 0.5, margin=1e-3, check_logits_every=2)
    assert rep.ok, rep.notes
    assert rep.max_logit_err < 2e-2
    out, n, _ = sd.generate(*W.pad_batch(srcs), [20, 11, 16], 6, 1, 0.0)
    for b, s in enumerate(srcs):                                # strict rule = greedy decoding (up to bf16 near-ties)
        ref = O.greedy_decode(mv, s, [20, 11, 16][b], BOS, EOS)
        got = out[b, :int(n[b])].cpu().tolist()
        assert got == ref, (b, _prefix_match(got, ref))
    sd.close()


def test_bart_base_shaped_pair_gelu_learned_positions():
    """The summarisation experiment's model family (Section 5.2): BART-base shapes (768 wide, 12 heads, 3072 inner,
    50265 ids: an odd vocabulary with a ragged last column tile), exact GELU, learned position tables, a drafter
    with the 6-layer encoder.  Lock-step against the oracle, then a batched generate with one sampled sequence."""
    from paper_2203_16487_b200 import binding
    wl = W.config_bart_summarization(3, 40, 150)
    wv = W.make_weights(wl.verifier, wl.seed_verifier, True, learned_pos=True)
    wd = W.make_weights(wl.drafter, wl.seed_drafter, True, learned_pos=True)
    mv = O.model_from(wl.verifier, wv, mode="bf16", act="gelu")
    md = O.model_from(wl.drafter, wd, mode="bf16", act="gelu")
    smax = max(len(s) for s in wl.src)
    sd = binding.SpecDec(wl.verifier, wv, wl.drafter, wd, k_max=25, max_batch=3, max_src=smax, max_tgt=40, bf16=True,
                         activation="gelu")
    rep = lockstep.run(sd, mv, md, wl.src[:2], [40, 40], 25, 3, 1.0, margin=1e-3, check_logits_every=2, max_iters=3)
    print(rep.iterations, rep.draft_near_ties, rep.verify_near_ties, rep.max_logit_err, rep.max_stat_err, rep.notes[:3])
    assert rep.ok, rep.notes
    assert rep.max_logit_err < 2e-2
    src, lens = W.pad_batch(wl.src)
    out, n, st = sd.generate(src, lens, [40, 30, 20], 25, 3, 1.0)
    assert st["emitted"] == int(n.sum()) and n.cpu().tolist() == [40, 30, 20]
    ref, _ = O.specdec_generate(mv, md, wl.src[2], 10, 25, 3, 1.0, BOS, EOS, MASK)
    assert out[2, :10].cpu().tolist() == ref
    sd.close()


@pytest.mark.parametrize("d,f,enc,dec", [(256, 1024, 12, 2), (512, 2048, 6, 6)])
def test_drafter_ablation_shapes(d, f, enc, dec):
    """The drafter-ablation table's other drafters (Section 4.1): model / FFN width 256 / 1024 ("w/o Principle I") and a
    balanced 6 + 6 drafter ("w/o Principle II"), each paired with the Transformer-base verifier: lock-step against the
    oracle on two sentences (drafts, accepted lengths, bifurcation tokens, logits)."""
    from paper_2203_16487_b200 import binding
    dd = W.ModelDims(d, 8 if d == 512 else 4, f, 32768, enc, dec, 1024)
    wv, wd = W.make_weights(W.BASE_V, 1001, True), W.make_weights(dd, 4002, True)
    mv, md = O.model_from(W.BASE_V, wv, mode="bf16"), O.model_from(dd, wd, mode="bf16")
    wl = W.config2_translation(2)
    sd = binding.SpecDec(W.BASE_V, wv, dd, wd, k_max=25, max_batch=2, max_src=40, max_tgt=48, bf16=True)
    rep = lockstep.run(sd, mv, md, wl.src, [16, 16], 25, 3, 1.0, margin=1e-3, check_logits_every=2, max_iters=4)
    print(rep.iterations, rep.draft_positions, rep.draft_near_ties, rep.verify_near_ties, rep.max_logit_err, rep.notes[:3])
    assert rep.ok, rep.notes
    assert rep.max_logit_err < 2e-2
    sd.close()
