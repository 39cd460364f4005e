"""The library's diagnostics entry points answer with plausible numbers."""
import pytest

from paper_2203_16487_b200 import workloads as W

pytestmark = pytest.mark.gpu


def test_link_cost_and_mma_rate():
    from paper_2203_16487_b200 import binding
    dims = W.ModelDims(128, 2, 512, 2000, 1, 1, 64)
    wv, wd = W.make_weights(dims, 1, True), W.make_weights(dims, 2, True)
    sd = binding.SpecDec(dims, wv, dims, wd, k_max=8, max_batch=32, max_src=16, max_tgt=16, bf16=True)
    us = sd.link_cost(32, 148)
    assert 0.05 < us < 50.0                                   # a kernel boundary costs on the order of a microsecond
    issue, done = sd.mma_rate(128, False, 2048)
    assert 16 <= done <= 1024 and issue <= done + 1           # a 128 x 128 x 16 MMA takes tens of clocks
    issue2, done2 = sd.mma_rate(256, True, 2048)
    assert done2 > 0.9 * done                                 # twice the columns over twice the SMs: not faster per instruction
    with pytest.raises(binding.SpecDecError):                 # the background stream wants an embedding table of 8 MB
        sd.mma_rate_bg(128, False, 2048, 2, 1)
    ns0, ns1 = sd.cluster_round(16, 0, 32), sd.cluster_round(16, 4096, 32)
    assert 50 < ns0 < 50000 and ns1 > ns0                     # an exchange round costs hundreds of nanoseconds, more with data
    # and the handle still works afterwards
    import numpy as np
    src = np.arange(4, 12, dtype=np.int32)[None]
    out, n, st = sd.generate(src, [8], [6], 4, 3, 1.0)
    assert int(n[0]) >= 1 and st["status"] == 0
    sd.close()


def test_mma_rate_with_commits_and_a_background_stream():
    """A commit per k-block and a producer's bulk copies into the same shared memory leave the MMA rate where it was."""
    from paper_2203_16487_b200 import binding
    dims = W.ModelDims(128, 2, 512, 32768, 1, 1, 64)
    wv, wd = W.make_weights(dims, 1, True), W.make_weights(dims, 2, True)
    sd = binding.SpecDec(dims, wv, dims, wd, k_max=8, max_batch=4, max_src=16, max_tgt=16, bf16=True)
    _, base, _ = sd.mma_rate_bg(256, False, 4096, 0, 0)
    _, done, bpc = sd.mma_rate_bg(256, False, 4096, 4, 1)
    assert done < 1.25 * base and bpc > 4.0                   # tens of bytes per clock land while the pipe keeps its pace
    _, done2, bpc2 = sd.mma_rate_bg(256, True, 4096, 2, 1)
    assert done2 < 1.25 * base and bpc2 > 2.0
    assert sd.integrity()["damaged_zones"] == 0
    sd.close()
