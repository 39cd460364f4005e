"""Seeded sweep over odd shapes through the C ABI, lock-step against the oracle, with the integrity check (red zones behind
every arena block, NaN / Inf scan) after every call: widths that are not powers of two, vocabularies that do not fill the
last tile, one to three layers, ragged sources, block sizes from 1 to 25, both precisions, both drafter readings, both
feed-forward activations.
Test infrastructure: the oracle is the reference, the CUDA library is what is tested."""
import numpy as np
import pytest

from oracle import specdec_oracle as O
from paper_2203_16487_b200 import workloads as W
from tests import lockstep

pytestmark = pytest.mark.gpu

# (d_model, heads, d_ffn, vocab, verifier enc/dec layers, drafter enc/dec layers, k, source lengths, bf16)
CASES = [
    (64, 1, 192, 1000, 1, 1, 1, 1, 1, (3, 9), False),
    (96, 3, 160, 517, 1, 2, 2, 1, 5, (12, 1, 7), False),
    (128, 2, 320, 3001, 2, 1, 1, 2, 13, (5, 16, 11, 2), True),
    (192, 3, 448, 4099, 1, 2, 2, 2, 7, (14, 6), True),
    (256, 4, 576, 2113, 2, 2, 1, 1, 9, (8, 15, 3, 10, 16), True),
    (320, 5, 640, 1601, 1, 1, 1, 3, 4, (16, 13, 9), True),
    (64, 2, 128, 130, 1, 3, 1, 1, 11, (4, 4, 4, 4, 4, 4, 4), True),
    (512, 8, 1024, 8257, 1, 1, 1, 1, 25, (16, 7), True),
    # the prefix-causal drafter reading with its K/V cache; exact GELU in the feed-forward blocks
    (192, 3, 320, 2050, 1, 2, 1, 2, 6, (10, 16, 2, 7, 13, 5), True, "prefix_causal", "relu"),
    (128, 2, 384, 1537, 2, 1, 1, 2, 8, (9, 12, 16, 1), True, "bidirectional", "gelu"),
    (96, 3, 224, 777, 1, 2, 1, 2, 5, (6, 11, 3), False, "prefix_causal", "gelu"),
]


@pytest.mark.parametrize("case", range(len(CASES)))
def test_odd_shapes_lockstep_with_integrity_checks(case):
    from paper_2203_16487_b200 import binding
    d, H, f, V, ve, vd, de, dd_, k, lens, bf16 = CASES[case][:11]
    reading, act = (CASES[case][11:] + ("bidirectional", "relu"))[:2]
    dv = W.ModelDims(d, H, f, V, ve, vd, 64)
    dd = W.ModelDims(d, H, f, V, de, dd_, 64)
    wv, wd = W.make_weights(dv, 500 + case, bf16), W.make_weights(dd, 600 + case, bf16)
    mode = "bf16" if bf16 else "pure"
    mv, md = O.model_from(dv, wv, mode=mode, act=act), O.model_from(dd, wd, mode=mode, act=act)
    rng = np.random.default_rng(700 + case)
    srcs = [W.zipf_ids(rng, n, V) for n in lens]
    tgts = [int(rng.integers(6, 20)) for _ in lens]
    sd = binding.SpecDec(dv, wv, dd, wd, k_max=k, max_batch=len(lens), max_src=16, max_tgt=20, bf16=bf16, activation=act)
    sd.set_option("debug_checks", 1)
    rep = lockstep.run(sd, mv, md, srcs, tgts, k, 3, 1.0, margin=1e-3 if bf16 else 0.0, check_logits_every=2, max_iters=6,
                       logit_tol=2e-2 if bf16 else 1e-4, drafter_reading=reading)
    print(case, rep.iterations, rep.draft_positions, rep.draft_near_ties, rep.verify_rows, rep.verify_near_ties,
          rep.max_logit_err, rep.max_stat_err, rep.notes[:4])
    assert rep.ok, rep.notes
    assert rep.max_logit_err < (2e-2 if bf16 else 1e-4) and rep.max_stat_err < (2e-2 if bf16 else 1e-4)
    # the same handle free-running, every call checked as well
    out, n, st = sd.generate(*W.pad_batch(srcs), np.array(tgts, np.int32), k, 3, 1.0)
    assert sd.integrity()["damaged_zones"] == 0 and sd.integrity()["nonfinite"] == 0
    n = n.cpu().numpy()
    assert (n <= np.array(tgts)).all() and (n >= 1).all()
    sd.close()
