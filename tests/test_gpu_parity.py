"""GPU parity tests: the CUDA path, called through the C ABI, against the CPU oracle.

Tolerances.  fp32 handles: logits within 1e-4 absolute (fp32 accumulation order
only), tokens and accepted lengths bit-exact.  bf16 handles: logits within 2e-2
absolute / 1e-2 relative of the pure-fp32 oracle, and of the oracle run with
bf16 operand rounding (two bf16 pipelines that differ only in fp32 summation
order still drift apart by rounding flips that cascade through the layers, so
the same bound applies); accepted lengths and tokens bit-exact except where the
oracle's margin for the differing decision is below 1e-3, which is counted and
printed.
"""
import math

import numpy as np
import pytest
import torch

from oracle import specdec_oracle as O
from paper_2203_16487_b200 import workloads as W
from tests import designed, lockstep

pytestmark = pytest.mark.gpu
BOS, EOS, MASK = W.BOS_ID, W.EOS_ID, W.MASK_ID


def _binding():
    from paper_2203_16487_b200 import binding
    return binding


def _handle(dv, wv, dd, wd, bf16, **kw):
    b = _binding()
    args = dict(k_max=8, max_batch=4, max_src=16, max_tgt=32, bf16=bf16)
    args.update(kw)
    return b.SpecDec(dv, wv, dd, wd, **args)


@pytest.fixture(scope="module")
def tiny():
    wl = W.config1_tiny()
    wv = W.make_weights(wl.verifier, wl.seed_verifier, False)
    wd = W.make_weights(wl.drafter, wl.seed_drafter, False)
    return wl, wv, wd, O.model_from(wl.verifier, wv), O.model_from(wl.drafter, wd)


# ---------------------------------------------------------------- the rule alone
@pytest.mark.parametrize("V,k,B", [(1000, 8, 7), (32768, 25, 5), (37, 3, 33)])
def test_accept_scan_matches_oracle(V, k, B):
    b = _binding()
    rng = np.random.default_rng(V + k)
    logits = (rng.standard_normal((B, k + 1, V)) * 3).astype(np.float32)
    logits[0, 0, :5] = logits[0, 0].max() + 1.0            # exact ties at the top
    top = logits.argmax(axis=2)
    drafts = np.where(rng.random((B, k)) < 0.7, top[:, :k], rng.integers(0, V, (B, k))).astype(np.int32)
    order = np.argsort(-logits[1, 1])
    drafts[1, 0], drafts[1, 1] = top[1, 0], order[2]        # a 3rd-ranked draft
    drafts[0, 0] = 3                                        # a draft inside the tie
    lg = torch.from_numpy(logits).cuda()
    for beta in (1, 3, 5, V):
        for tau in (0.0, 0.5, 1.0, 3.0, 1e9):
            acc, bif = b.accept_scan(lg, torch.from_numpy(drafts), beta, tau)
            acc, bif = acc.cpu().numpy(), bif.cpu().numpy()
            for s in range(B):
                assert (acc[s], bif[s]) == O.verify(logits[s], drafts[s].tolist(), beta, tau), (beta, tau, s)


# ---------------------------------------------------------------- config 1: tiny fp32
@pytest.mark.parametrize("beta,tau,graphs", [(3, 1.0, 1), (1, 0.0, 1), (3, 1.0, 0)])
def test_config1_generate_bit_exact(tiny, beta, tau, graphs):
    wl, wv, wd, mv, md = tiny
    sd = _handle(wl.verifier, wv, wl.drafter, wd, False)
    sd.set_option("graphs", graphs)
    for s in wl.src:                                         # batch 1, one source at a time
        out, n, st = sd.generate(s[None], [len(s)], [32], wl.k, beta, tau)
        got = out[0, :int(n[0])].cpu().tolist()
        ref, ost = O.specdec_generate(mv, md, s, 32, wl.k, beta, tau, BOS, EOS, MASK)
        assert got == ref
        assert st["emitted"] == len(ref) and st["accepted"] == ost.accepted and st["seq_iterations"] == ost.iterations
        if (beta, tau) == (1, 0.0):
            assert got == O.greedy_decode(mv, s, 32, BOS, EOS)
    # the padded batch gives the same sequences as batch 1
    src, lens = W.pad_batch(wl.src)
    out, n, _ = sd.generate(src, lens, wl.max_tgt, wl.k, beta, tau)
    for b, s in enumerate(wl.src):
        ref, _ = O.specdec_generate(mv, md, s, 32, wl.k, beta, tau, BOS, EOS, MASK)
        assert out[b, :int(n[b])].cpu().tolist() == ref
    assert sd.launch_count() > 100
    sd.close()


@pytest.mark.parametrize("opts", [
    {"gate": 0, "poll_flag": 0},                    # plain graphs, the counter copied back after every iteration
    {"gate": 0, "poll_flag": 0, "poll_lag": 2},     # ... read two iterations late: two wasted iterations at the end
    {"gate": 0, "poll_flag": 1, "poll_lag": 1},     # the commit kernel's posted word, one iteration late
    {"gate": 2, "poll_flag": 1},                    # every iteration behind a device-side IF node, host two ahead
    {"gate": 2, "poll_flag": 0, "poll_lag": 3},
    {"stats_timing": 1},                            # an event after every phase: separate draft / verify graphs
    {"graphs": 0},
])
def test_generate_loop_variants_bit_exact(tiny, opts):
    """Every way the host can drive the draft -> verify -> commit loop gives the oracle's sequences and counters
    (Algorithm 1 is the same; only who waits for whom changes)."""
    wl, wv, wd, mv, md = tiny
    sd = _handle(wl.verifier, wv, wl.drafter, wd, False)
    for name, val in opts.items():
        sd.set_option(name, val)
    src, lens = W.pad_batch(wl.src)
    refs = [O.specdec_generate(mv, md, s, 32, wl.k, 3, 1.0, BOS, EOS, MASK) for s in wl.src]
    for rep in range(2):                                     # the second call replays the graphs the first one built
        out, n, st = sd.generate(src, lens, wl.max_tgt, wl.k, 3, 1.0)
        for b, (ref, _) in enumerate(refs):
            assert out[b, :int(n[b])].cpu().tolist() == ref
        assert st["emitted"] == sum(len(r) for r, _ in refs)
        assert st["accepted"] == sum(o.accepted for _, o in refs)
        assert st["seq_iterations"] == sum(o.iterations for _, o in refs)
        longest = max(o.iterations for _, o in refs)
        wasted = opts.get("poll_lag", 0) if opts.get("gate", 1) == 0 else 0      # behind the gate they do not run
        assert st["iterations"] == min(longest + wasted, 32)            # the loop never runs past max_tgt iterations
        assert st["ms_total"] > 0 and st["ms_encode"] > 0
        assert (st["ms_verify"] > 0) == bool(opts.get("stats_timing", 0))
    # one sentence at a time after the batch: the posted commit count carries over between calls
    for s, (ref, _) in zip(wl.src, refs):
        out, n, _ = sd.generate(s[None], [len(s)], [32], wl.k, 3, 1.0)
        assert out[0, :int(n[0])].cpu().tolist() == ref
    sd.close()


def test_degenerate_shapes_bit_exact(tiny):
    """One-token sources, k = 1 and k = k_max, target budgets of 0, 1 and 2 tokens in one batch, a rule that accepts
    everything (beta = V, huge tau) and the strict one: each sequence must equal the oracle's batch-1 run."""
    wl, wv, wd, mv, md = tiny
    V = wl.verifier.vocab
    srcs = [np.array([7], np.int32), np.array([901], np.int32), wl.src[0][:2], wl.src[1]]
    budgets = [0, 1, 2, 5]
    sd = _handle(wl.verifier, wv, wl.drafter, wd, False)
    src, lens = W.pad_batch(srcs)
    for k in (1, 8):
        for beta, tau in ((V, 1e30), (1, 0.0), (2, 0.25)):
            out, n, st = sd.generate(src, lens, budgets, k, beta, tau)
            assert n.cpu().tolist()[0] == 0
            for b, s in enumerate(srcs):
                ref, _ = O.specdec_generate(mv, md, s, budgets[b], k, beta, tau, BOS, EOS, MASK)
                assert out[b, :int(n[b])].cpu().tolist() == ref, (k, beta, tau, b)
            assert st["emitted"] == int(n.sum())
    sd.close()


def test_k0_is_greedy_autoregressive_decoding(tiny):
    """k = 0 runs the verifier alone, one row per step: the greedy baseline of the paper's comparisons."""
    wl, wv, wd, mv, md = tiny
    sd = _handle(wl.verifier, wv, wl.drafter, wd, False)
    src, lens = W.pad_batch(wl.src)
    out, n, st = sd.generate(src, lens, wl.max_tgt, 0, 1, 0.0)
    for b, s in enumerate(wl.src):
        assert out[b, :int(n[b])].cpu().tolist() == O.greedy_decode(mv, s, 32, BOS, EOS)
    assert st["drafted"] == 0 and st["accepted"] == 0 and st["emitted"] == int(n.sum()) == st["seq_iterations"]
    sd.close()


def test_tiny_lockstep_logits_and_stats(tiny):
    wl, wv, wd, mv, md = tiny
    sd = _handle(wl.verifier, wv, wl.drafter, wd, False)
    rep = lockstep.run(sd, mv, md, wl.src, wl.max_tgt, wl.k, 3, 1.0, margin=0.0, check_logits_every=1)
    print(rep)
    assert rep.ok, rep.notes
    assert rep.max_logit_err < 1e-4 and rep.max_stat_err < 1e-4
    assert rep.draft_near_ties == 0 and rep.verify_near_ties == 0
    # drafter logits of the first pass
    src, lens = W.pad_batch(wl.src[:2])
    sd.encode(src, lens, [32, 32])
    sd.draft(wl.k)
    g = sd.debug_logits(1, 2 * wl.k).cpu().numpy().reshape(2, wl.k, -1)
    for b in range(2):
        ref = O.decoder_rows(md, [BOS] + [MASK] * wl.k, O.encode(md, wl.src[b]), False)[1:]
        assert np.abs(g[b] - ref).max() < 1e-4
    sd.close()


def test_sharp_models_tau_binds():
    """Embedding tables N(0, 0.06^2): top-1/top-2 gaps are about 1, so tau and beta change the accepted length."""
    wv, wd = W.sharp_tiny_models()
    mv, md = O.model_from(W.TINY_V, wv), O.model_from(W.TINY_D, wd)
    rng = np.random.default_rng(4)
    srcs = [W.zipf_ids(rng, n, 1000) for n in (16, 9, 13)]
    sd = _handle(W.TINY_V, wv, W.TINY_D, wd, False)
    g = [O.greedy_decode(mv, s, 24, BOS, -1) for s in srcs]

    def near_greedy(b, committed, k):
        # greedy continuation with every third draft replaced by the verifier's 2nd choice
        rows = O.verify_rows(mv, O.encode(mv, srcs[b]), committed, (g[b][len(committed):] + [5] * k)[:k], BOS)
        d = (g[b][len(committed):] + [5] * k)[:k]
        for i in range(2, k, 3):
            d[i] = int(np.argsort(-rows[i], kind="stable")[1])
        return d

    seen = set()
    for beta, tau in [(1, 0.0), (2, 0.5), (3, 1.0), (3, 3.0), (5, 0.1)]:
        rep = lockstep.run(sd, mv, md, srcs, [24] * 3, 8, beta, tau, margin=0.0, eos=-1, draft_fn=near_greedy)
        assert rep.ok, rep.notes
        seen.add(rep.iterations)
    assert len(seen) > 1          # the rule's parameters did change the trajectory
    sd.close()


def test_case_study_on_gpu():
    dv, wv, dd, wd, T, D, src = designed.case_study_pair()
    sd = _handle(dv, wv, dd, wd, False, k_max=10, max_tgt=40)
    for beta, tau in [(3, 1.0), (1, 0.0)]:
        out, n, st = sd.generate(src[None], [len(src)], [40], 10, beta, tau)
        assert out[0, :int(n[0])].cpu().tolist() == T[1:]
        assert st["seq_iterations"] == 3 and st["accepted"] == 2 + 9 + 2 and st["emitted"] == 15
    dv, wv, dd, wd, T, D, src = designed.case_study_pair(near_top_at=5)
    sd2 = _handle(dv, wv, dd, wd, False, k_max=10, max_tgt=40)
    out, n, _ = sd2.generate(src[None], [len(src)], [40], 10, 3, 1.0)
    assert out[0, 4].item() == D[5]
    out, n, _ = sd2.generate(src[None], [len(src)], [40], 10, 1, 0.0)
    assert out[0, :int(n[0])].cpu().tolist() == T[1:]
    sd.close(); sd2.close()


def test_eos_max_tgt_and_explicit_commit(tiny):
    wl, wv, wd, mv, md = tiny
    s = wl.src[0]
    g = O.greedy_decode(mv, s, 32, BOS, -1)
    eos = g[5]
    b = _binding()
    sd = b.SpecDec(wl.verifier, wv, wl.drafter, wd, k_max=8, max_batch=4, max_src=16, max_tgt=32, bf16=False, eos_id=eos)
    out, n, _ = sd.generate(s[None], [len(s)], [32], 8, 1, 0.0)
    assert out[0, :int(n[0])].cpu().tolist() == g[:g.index(eos) + 1]
    sd.close()
    sd = _handle(wl.verifier, wv, wl.drafter, wd, False)
    # max_tgt 0 / 1 / 7 and ragged sources in one batch
    srcs = [wl.src[0], wl.src[1][:5], wl.src[2][:11]]
    src, lens = W.pad_batch(srcs)
    out, n, _ = sd.generate(src, lens, [0, 1, 7], 8, 3, 1.0)
    assert n.cpu().tolist() == [0, 1, 7]
    for i, mt in enumerate([0, 1, 7]):
        ref, _ = O.specdec_generate(mv, md, srcs[i], mt, 8, 3, 1.0, BOS, EOS, MASK)
        assert out[i, :mt].cpu().tolist() == ref
    # explicit commit builds a prefix: keep = k drafts + next token
    sd.encode(s[None], [len(s)], [32])
    sd.verify(np.array([g[:8]], np.int32), 1, 0.0)
    sd.commit([8], [g[8]])
    o, n, fin = sd.output()
    assert o[0, :9].cpu().tolist() == g[:9] and int(n[0]) == 9 and int(fin[0]) == 0
    acc, bif = sd.verify(np.array([g[9:17]], np.int32), 1, 0.0)
    assert int(acc[0]) == 8 and int(bif[0]) == g[17]
    sd.commit([0], [g[9]])                                  # rollback: keep nothing, continue with one token
    acc, bif = sd.verify(np.array([g[10:18]], np.int32), 1, 0.0)
    assert int(acc[0]) == 8 and int(bif[0]) == g[18]
    sd.close()


def test_error_paths(tiny):
    wl, wv, wd, mv, md = tiny
    b = _binding()
    sd = _handle(wl.verifier, wv, wl.drafter, wd, False)
    with pytest.raises(b.SpecDecError) as e:
        sd.draft(4)
    assert e.value.code == -4
    src, lens = W.pad_batch(wl.src)
    with pytest.raises(b.SpecDecError) as e:
        sd.generate(np.concatenate([src, src]), np.concatenate([lens, lens]), None, 8, 3, 1.0)
    assert e.value.code == -3
    with pytest.raises(b.SpecDecError) as e:
        sd.generate(src, lens, None, 9, 3, 1.0)
    assert e.value.code == -3
    with pytest.raises(b.SpecDecError) as e:
        sd.generate(src, lens, None, 8, 0, 1.0)
    assert e.value.code == -1
    sd.encode(src, lens)
    with pytest.raises(b.SpecDecError):
        sd.commit()
    bad = dict(wv); del bad["dec.1.ffn.w2"]
    with pytest.raises(b.SpecDecError) as e:
        _handle(wl.verifier, bad, wl.drafter, wd, False)
    assert e.value.code == -2
    sd.close()


def test_generate_host_buffers(tiny):
    wl, wv, wd, mv, md = tiny
    sd = _handle(wl.verifier, wv, wl.drafter, wd, False)
    src, lens = W.pad_batch(wl.src)
    hs = torch.from_numpy(src).pin_memory(); hl = torch.from_numpy(lens).pin_memory()
    hm = torch.tensor(wl.max_tgt, dtype=torch.int32).pin_memory()
    ho = torch.zeros((4, 32), dtype=torch.int32).pin_memory(); hn = torch.zeros(4, dtype=torch.int32).pin_memory()
    sd.generate_host(hs, hl, hm, ho, hn, 8, 3, 1.0)
    for b, s in enumerate(wl.src):
        ref, _ = O.specdec_generate(mv, md, s, 32, 8, 3, 1.0, BOS, EOS, MASK)
        assert ho[b, :int(hn[b])].tolist() == ref
    sd.close()


# ---------------------------------------------------------------- bf16 operands
MID_V = W.ModelDims(128, 2, 512, 2000, 2, 2, 128)
MID_D = W.ModelDims(128, 2, 512, 2000, 3, 2, 128)


@pytest.mark.parametrize("gemm,attn", [(0, 0), (1, 0), (0, 1), (1, 1)])
def test_bf16_mid_lockstep(gemm, attn):
    wv, wd = W.make_weights(MID_V, 21, True), W.make_weights(MID_D, 22, True)
    mv, md = O.model_from(MID_V, wv, mode="bf16"), O.model_from(MID_D, wd, mode="bf16")
    rng = np.random.default_rng(6)
    srcs = [W.zipf_ids(rng, n, 2000) for n in (20, 7, 33, 12, 25)]
    sd = _handle(MID_V, wv, MID_D, wd, True, k_max=12, max_batch=8, max_src=40, max_tgt=40)
    try:
        sd.set_option("gemm", gemm)
        sd.set_option("attn", attn)
    except Exception as e:
        pytest.skip(f"tensor-core GEMM not available: {e}")
    rep = lockstep.run(sd, mv, md, srcs, [30, 18, 40, 5, 33], 12, 3, 1.0, margin=1e-3, check_logits_every=2,
                       pad_to=40)
    print(rep.iterations, rep.draft_near_ties, rep.verify_near_ties, rep.max_logit_err, rep.max_stat_err)
    assert rep.ok, rep.notes
    assert rep.max_logit_err < 2e-2 and rep.max_stat_err < 2e-2
    assert rep.draft_near_ties <= 0.05 * rep.draft_positions
    sd.close()


@pytest.mark.parametrize("nseq,skinny", [(2, 1), (4, 1), (2, 0), (4, 2)])
def test_bf16_mid_small_batches_weight_streaming_gemm(nseq, skinny):
    """Passes of at most 32 rows run the weight-streaming GEMM with fused LayerNorm (26 rows: two 16-row
    tiles); 52 rows run one 128-row tile of the tensor-core GEMM with 64-wide column tiles."""
    wv, wd = W.make_weights(MID_V, 21, True), W.make_weights(MID_D, 22, True)
    mv, md = O.model_from(MID_V, wv, mode="bf16"), O.model_from(MID_D, wd, mode="bf16")
    rng = np.random.default_rng(8)
    srcs = [W.zipf_ids(rng, n, 2000) for n in (20, 7, 33, 12)][:nseq]
    sd = _handle(MID_V, wv, MID_D, wd, True, k_max=12, max_batch=4, max_src=40, max_tgt=24)
    sd.set_option("skinny", min(skinny, 1))
    sd.set_option("ln_fuse", 1 if skinny == 2 else 0)      # 2: also fuse each LayerNorm into the residual GEMM before it
    sd.set_option("attn_rs", 2 if skinny == 2 else 1)      # ... and keep attention scores in registers wherever possible
    rep = lockstep.run(sd, mv, md, srcs, [24, 18, 9, 20][:nseq], 12, 3, 1.0, margin=1e-3, check_logits_every=2)
    print(rep.iterations, rep.draft_near_ties, rep.verify_near_ties, rep.max_logit_err, rep.max_stat_err)
    assert rep.ok, rep.notes
    assert rep.max_logit_err < 2e-2 and rep.max_stat_err < 2e-2
    sd.close()


@pytest.mark.parametrize("long_keys,mode", [(False, 2), (True, 2), (True, 3)])
def test_bf16_streaming_attention(long_keys, mode):
    """The streaming tile attention (key blocks of 64 through a two-stage ring, running maximum) against the
    oracle's one-pass softmax: forced on for the short case (a single, partly filled block), and over sources of
    up to 200 tokens and targets past 64 (several blocks, ragged last block, causal mask crossing a block edge)."""
    dv = W.ModelDims(128, 2, 512, 2000, 2, 2, 256)
    dd = W.ModelDims(128, 2, 512, 2000, 3, 2, 256)
    wv, wd = W.make_weights(dv, 31, True), W.make_weights(dd, 32, True)
    mv, md = O.model_from(dv, wv, mode="bf16"), O.model_from(dd, wd, mode="bf16")
    rng = np.random.default_rng(9)
    if long_keys:
        lens, tgts, max_src, max_tgt = (150, 97, 200, 64), [90, 70, 40, 80], 200, 96
    else:
        lens, tgts, max_src, max_tgt = (20, 7, 33, 12), [24, 18, 9, 20], 40, 24
    srcs = [W.zipf_ids(rng, n, 2000) for n in lens]
    sd = _handle(dv, wv, dd, wd, True, k_max=12, max_batch=4, max_src=max_src, max_tgt=max_tgt)
    sd.set_option("attn_stream", mode)                       # 2: four-stage ring here (few CTAs), 3: the two-stage ring
    rep = lockstep.run(sd, mv, md, srcs, tgts, 12, 3, 1.0, margin=1e-3, check_logits_every=2)
    print(rep.iterations, rep.draft_near_ties, rep.verify_near_ties, rep.max_logit_err, rep.max_stat_err)
    assert rep.ok, rep.notes
    assert rep.max_logit_err < 2e-2 and rep.max_stat_err < 2e-2
    sd.close()


@pytest.mark.parametrize("sk_cluster", [1, 0])
def test_base_shapes_batch1_lockstep(sk_cluster):
    """One config-2 sentence at batch 1 (26-row verify block): per-operation kernels with the weight-streaming GEMM,
    its LayerNorm prologue shared across clusters of 8 CTAs (the default) or computed by every CTA."""
    wl = W.config2_translation(1)
    wv = W.make_weights(wl.verifier, wl.seed_verifier, True)
    wd = W.make_weights(wl.drafter, wl.seed_drafter, True)
    mv, md = O.model_from(wl.verifier, wv, mode="bf16"), O.model_from(wl.drafter, wd, mode="bf16")
    sd = _handle(wl.verifier, wv, wl.drafter, wd, True, k_max=25, max_batch=1, max_src=40, max_tgt=64)
    sd.set_option("sk_cluster", sk_cluster)
    rep = lockstep.run(sd, mv, md, wl.src, wl.max_tgt, 25, 3, 1.0, margin=1e-3, check_logits_every=4, max_iters=8)
    print(rep.iterations, rep.draft_positions, rep.draft_near_ties, rep.verify_rows, rep.verify_near_ties,
          rep.max_logit_err, rep.max_stat_err, rep.notes[:5])
    assert rep.ok, rep.notes
    assert rep.max_logit_err < 2e-2 and rep.max_stat_err < 2e-2
    sd.close()


def test_base_shapes_bf16_lockstep_and_pure_tolerance():
    """Transformer-base shapes (config 2 recipe), a few sentences: lock-step against the oracle with bf16
    operand rounding, and logits against the pure-fp32 oracle within 2e-2 abs / 1e-2 rel."""
    wl = W.config2_translation(3)
    wv = W.make_weights(wl.verifier, wl.seed_verifier, True)
    wd = W.make_weights(wl.drafter, wl.seed_drafter, True)
    mv, md = O.model_from(wl.verifier, wv, mode="bf16"), O.model_from(wl.drafter, wd, mode="bf16")
    sd = _handle(wl.verifier, wv, wl.drafter, wd, True, k_max=25, max_batch=4, max_src=40, max_tgt=64)
    rep = lockstep.run(sd, mv, md, wl.src, wl.max_tgt, 25, 3, 1.0, margin=1e-3, check_logits_every=8, max_iters=10)
    print(rep.iterations, rep.draft_positions, rep.draft_near_ties, rep.verify_rows, rep.verify_near_ties,
          rep.max_logit_err, rep.max_stat_err, rep.notes[:5])
    assert rep.ok, rep.notes
    assert rep.max_logit_err < 2e-2 and rep.max_stat_err < 2e-2
    # pure fp32 oracle: 2e-2 absolute + 1e-2 relative for bf16 operands
    mp = O.model_from(wl.verifier, wv)
    s = wl.src[0]
    sd.encode(s[None], [len(s)], [32])
    drafts = np.arange(100, 125, dtype=np.int32)[None]
    sd.verify(drafts, 3, 1.0)
    g = sd.debug_logits(0, 26).cpu().numpy()
    ref = O.verify_rows(mp, O.encode(mp, s), [], drafts[0].tolist(), BOS)
    err = np.abs(g - ref)
    assert (err <= 2e-2 + 1e-2 * np.abs(ref)).all(), err.max()
    sd.close()


# ---------------------------------------------------------------- failure reporting (no GPU fault, nothing waits)
def test_device_error_word_reaches_the_caller_and_the_handle_recovers(tiny):
    """A bounded device-side wait that gives up raises a code in a device word.  Here the host writes that word
    itself (option "inject_error"): specdec_verify and specdec_generate must return SPECDEC_ERR_TIMEOUT with a
    message, report it once, and the handle must work again after specdec_encode."""
    b = _binding()
    wl, wv, wd, mv, md = tiny
    sd = _handle(wl.verifier, wv, wl.drafter, wd, False)
    s = wl.src[0]
    ref, _ = O.specdec_generate(mv, md, s, 32, wl.k, 3, 1.0, BOS, EOS, MASK)
    # step API
    sd.encode(s[None], [len(s)], [32])
    sd.set_option("inject_error", 5)
    with pytest.raises(b.SpecDecError) as e:
        sd.verify(np.zeros((1, wl.k), np.int32), 3, 1.0)
    assert e.value.code == -6 and "wait gave up" in str(e.value) and "5" in str(e.value)
    sd.encode(s[None], [len(s)], [32])                       # reported once: the next session starts clean
    d = sd.draft(wl.k)
    acc, bif = sd.verify(d, 3, 1.0)
    assert 0 <= int(acc[0]) <= wl.k
    # the loop
    sd.set_option("inject_error", 9)
    with pytest.raises(b.SpecDecError) as e:
        sd.generate(s[None], [len(s)], [32], wl.k, 3, 1.0)
    assert e.value.code == -6 and "9" in str(e.value)
    for _ in range(2):                                       # and generate works again, twice (commit counter intact)
        out, n, st = sd.generate(s[None], [len(s)], [32], wl.k, 3, 1.0)
        assert out[0, :int(n[0])].cpu().tolist() == ref and st["status"] == 0
    sd.close()


@pytest.mark.parametrize("gate", [2, 0])
def test_generate_with_every_budget_zero(tiny, gate):
    """Five sequences whose target budgets are all 0: nothing to decode, no commit ever runs behind the device-side
    gate; the call must return five empty outputs, and a normal call afterwards must still be right."""
    wl, wv, wd, mv, md = tiny
    sd = _handle(wl.verifier, wv, wl.drafter, wd, False, max_batch=5)
    sd.set_option("gate", gate)
    sd.set_option("poll_flag", 1)
    srcs = [wl.src[i % 4] for i in range(5)]
    src, lens = W.pad_batch(srcs)
    out, n, st = sd.generate(src, lens, [0] * 5, wl.k, 3, 1.0)
    assert n.cpu().tolist() == [0] * 5 and st["emitted"] == 0 and st["status"] == 0
    out, n, st = sd.generate(src, lens, [0, 3, 0, 32, 1], wl.k, 3, 1.0)
    for i, mt in enumerate([0, 3, 0, 32, 1]):
        ref, _ = O.specdec_generate(mv, md, srcs[i], mt, wl.k, 3, 1.0, BOS, EOS, MASK)
        assert out[i, :int(n[i])].cpu().tolist() == ref
    sd.close()


# ---------------------------------------------------------------- the drafter's prefix-causal reading (cached drafter)
def test_prefix_causal_drafter_tiny_and_designed_pair(tiny):
    """Option "drafter_prefix_causal": fp32, every draft and decision in lock-step with the oracle's prefix-causal
    drafter, then whole generations.  The designed pair accepts several drafts per iteration, so the drafter's cache
    grows by more than one position at a time; the tiny pair grows it one by one."""
    wl, wv, wd, mv, md = tiny
    sd = _handle(wl.verifier, wv, wl.drafter, wd, False)
    rep = lockstep.run(sd, mv, md, wl.src, wl.max_tgt, wl.k, 3, 1.0, margin=0.0, check_logits_every=3,
                       drafter_reading="prefix_causal")
    assert rep.ok and rep.draft_near_ties == 0 and rep.verify_near_ties == 0, rep.notes
    src, lens = W.pad_batch(wl.src)
    for graphs in (1, 0):
        sd.set_option("graphs", graphs)
        out, n, st = sd.generate(src, lens, wl.max_tgt, wl.k, 3, 1.0)
        for b, s in enumerate(wl.src):
            ref, _ = O.specdec_generate(mv, md, s, 32, wl.k, 3, 1.0, BOS, EOS, MASK, drafter_reading="prefix_causal")
            assert out[b, :int(n[b])].cpu().tolist() == ref
    sd.close()
    dv, dwv, dd, dwd, T, D, dsrc = designed.case_study_pair()
    mv2, md2 = O.model_from(dv, dwv), O.model_from(dd, dwd)
    sd = _handle(dv, dwv, dd, dwd, False, k_max=10, max_batch=2, max_src=16, max_tgt=40)
    sd.set_option("drafter_prefix_causal", 1)
    ref, ost = O.specdec_generate(mv2, md2, dsrc, 40, 10, 3, 1.0, BOS, EOS, MASK, drafter_reading="prefix_causal")
    for rep_i in range(2):
        out, n, st = sd.generate(np.stack([dsrc, dsrc]), [len(dsrc)] * 2, [40, 7], 10, 3, 1.0)
        assert out[0, :int(n[0])].cpu().tolist() == ref and out[1, :int(n[1])].cpu().tolist() == ref[:7]
    assert ost.accepted >= 8                                  # several drafts accepted per iteration
    sd.close()


def test_prefix_causal_drafter_bf16_lockstep():
    """The same reading on the bf16 tensor-core path: mid-sized models, five sequences of different lengths, the
    oracle's decisions committed on both sides (prefixes grow by 1 .. k + 1 tokens per iteration)."""
    wv, wd = W.make_weights(MID_V, 21, True), W.make_weights(MID_D, 22, True)
    mv, md = O.model_from(MID_V, wv, mode="bf16"), O.model_from(MID_D, wd, mode="bf16")
    rng = np.random.default_rng(6)
    srcs = [W.zipf_ids(rng, n, 2000) for n in (20, 7, 33, 12, 25)]
    sd = _handle(MID_V, wv, MID_D, wd, True, k_max=12, max_batch=8, max_src=40, max_tgt=40)
    # drafts that the verifier partly accepts: its own greedy continuation with a wrong token every few positions
    greedy = [O.greedy_decode(mv, s, 40, BOS, EOS) for s in srcs]

    def draft_fn(b, committed, k):
        g = greedy[b][len(committed):len(committed) + k]
        g = g + [7] * (k - len(g))
        if len(g) > 4:
            g[4] = 9
        return g
    rep = lockstep.run(sd, mv, md, srcs, [30, 18, 40, 5, 33], 12, 3, 1.0, margin=1e-3, check_logits_every=2, pad_to=40,
                       drafter_reading="prefix_causal")
    print(rep.iterations, rep.draft_near_ties, rep.verify_near_ties, rep.max_logit_err, rep.max_stat_err)
    assert rep.ok, rep.notes
    assert rep.max_logit_err < 2e-2 and rep.draft_near_ties <= 0.05 * rep.draft_positions
    # with accepted drafts (the GPU drafter still runs and is compared; the committed prefix jumps by up to 5)
    sd.set_option("drafter_prefix_causal", 1)
    src, lens = W.pad_batch(srcs, 40)
    sd.encode(src, lens, np.asarray([30, 18, 40, 5, 33], np.int32))
    out = [[] for _ in srcs]
    mem_d = [O.encode(md, s) for s in srcs]
    for it in range(6):
        g_draft = sd.draft(12).cpu().numpy()
        keep, nxt = np.zeros(5, np.int32), np.zeros(5, np.int32)
        for b in range(5):
            j = len(out[b])
            if j >= [30, 18, 40, 5, 33][b]:
                continue
            logits = O.decoder_rows(md, [BOS] + out[b] + [MASK] * 12, mem_d[b], causal=False, n_causal=j + 1)[j + 1:]
            o_draft = logits.argmax(axis=1)
            for i in range(12):
                if g_draft[b, i] != o_draft[i]:
                    assert float(logits[i, o_draft[i]] - logits[i, g_draft[b, i]]) < 1e-3, (it, b, i)
            d = draft_fn(b, out[b], 12)
            keep[b] = min(4, [30, 18, 40, 5, 33][b] - j - 1) if [30, 18, 40, 5, 33][b] - j - 1 > 0 else 0
            nxt[b] = d[keep[b]] if keep[b] < len(d) else 7
        blk = np.stack([draft_fn(b, out[b], 12) for b in range(5)]).astype(np.int32)
        sd.verify(blk, 3, 1.0)
        sd.commit(keep, nxt)
        for b in range(5):
            mt = [30, 18, 40, 5, 33][b]
            if len(out[b]) < mt:
                O.commit(out[b], blk[b].tolist(), int(keep[b]), int(nxt[b]), mt, EOS)
    sd.close()


def test_prefix_causal_drafter_base_shapes_generate():
    """Transformer-base shapes, bf16, batch 4 with default options: whole generations with the cached drafter equal the
    oracle's prefix-causal generations (the output of a random-init pair is the verifier's greedy continuation either
    way, so the drafts themselves are compared in lock-step on one sentence first)."""
    wl = W.config2_translation(4)
    wv = W.make_weights(wl.verifier, wl.seed_verifier, True)
    wd = W.make_weights(wl.drafter, wl.seed_drafter, True)
    mv, md = O.model_from(wl.verifier, wv, mode="bf16"), O.model_from(wl.drafter, wd, mode="bf16")
    sd = _handle(wl.verifier, wv, wl.drafter, wd, True, k_max=25, max_batch=4, max_src=40, max_tgt=64)
    rep = lockstep.run(sd, mv, md, wl.src[:2], wl.max_tgt[:2], 25, 3, 1.0, margin=1e-3, check_logits_every=4, max_iters=6,
                       drafter_reading="prefix_causal")
    print(rep.iterations, rep.draft_positions, rep.draft_near_ties, rep.verify_near_ties, rep.max_logit_err, rep.notes[:3])
    assert rep.ok, rep.notes
    src, lens = W.pad_batch(wl.src, 40)
    out, n, st = sd.generate(src, lens, wl.max_tgt, 25, 3, 1.0)
    for b in (0, 3):
        ref, _ = O.specdec_generate(mv, md, wl.src[b], wl.max_tgt[b], 25, 3, 1.0, BOS, EOS, MASK, drafter_reading="prefix_causal")
        assert out[b, :int(n[b])].cpu().tolist() == ref
    sd.close()


def test_integrity_checks_find_a_damaged_red_zone_and_a_nan(tiny):
    """The arena's red zones and the non-finite scan: clean after real work; a red zone damaged from the host (an
    in-arena write: nothing faults) and a NaN placed in an activation buffer are found, named, and -- with option
    debug_checks -- fail the next step call with SPECDEC_ERR_CORRUPT; the handle works again once they are repaired."""
    wl, wv, wd, mv, md = tiny
    sd = _handle(wl.verifier, wv, wl.drafter, wd, False, k_max=wl.k)
    src, lens = W.pad_batch(wl.src)
    want = sd.generate(src, lens, np.array(wl.max_tgt, np.int32), wl.k, wl.beta, wl.tau)[0].cpu().numpy()
    rep = sd.integrity()
    assert rep["zones"] > 100 and rep["damaged_zones"] == 0 and rep["first_damaged_zone"] == -1, rep
    assert rep["nonfinite"] == 0 and rep["first_nonfinite_buffer"] == -1, rep
    sd.set_option("debug_checks", 1)
    got = sd.generate(src, lens, np.array(wl.max_tgt, np.int32), wl.k, wl.beta, wl.tau)[0].cpu().numpy()
    assert (got == want).all()
    # a damaged red zone
    sd.set_option("poke_zone", 7)
    rep = sd.integrity()
    assert rep["damaged_zones"] == 1 and rep["first_damaged_zone"] == 7, rep
    b = _binding()
    with pytest.raises(b.SpecDecError) as ei:
        sd.generate(src, lens, np.array(wl.max_tgt, np.int32), wl.k, wl.beta, wl.tau)
    assert ei.value.code == -8 and "red zone" in str(ei.value) and "block 7" in str(ei.value), str(ei.value)
    sd.set_option("heal_zones", 1)
    assert sd.integrity()["damaged_zones"] == 0
    # a NaN in the attention-output buffer (buffer 4 of the scan), in a row no pass of this test reaches
    sd.set_option("poke_nan", 1)
    rep = sd.integrity()
    assert rep["nonfinite"] == 1 and rep["first_nonfinite_buffer"] == 4, rep
    with pytest.raises(b.SpecDecError) as ei:
        sd.generate(src, lens, np.array(wl.max_tgt, np.int32), wl.k, wl.beta, wl.tau)
    assert ei.value.code == -8 and "attention output" in str(ei.value), str(ei.value)
    sd.set_option("poke_nan", 0)
    got = sd.generate(src, lens, np.array(wl.max_tgt, np.int32), wl.k, wl.beta, wl.tau)[0].cpu().numpy()
    assert (got == want).all()
    sd.close()
