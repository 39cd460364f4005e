"""specdec_accept_scan_static -- the acceptance rule for callers that cannot allocate device memory
(for example inside a server whose pool already owns all of HBM): its intermediate statistics sit in a
fixed array inside the library.  Checked through the C ABI against the oracle's rule row by row and against
specdec_accept_scan, on two calls in a row that share that array, the second smaller than the first so stale
entries would show.  Collected last on purpose, so a run that stops at the first failure has already run
everything else."""
import numpy as np
import pytest
import torch

from oracle import specdec_oracle as O

pytestmark = pytest.mark.gpu


def _case(rng, B, k, V):
    logits = (rng.standard_normal((B, k + 1, V)) * 3).astype(np.float32)
    top = logits.argmax(axis=2)
    drafts = np.where(rng.random((B, k)) < 0.75, top[:, :k], rng.integers(0, V, (B, k))).astype(np.int32)
    logits[0, 0, :4] = logits[0, 0].max() + 0.5             # exact ties at the top of one row
    drafts[0, 0] = 2
    return logits, drafts


def _oracle(logits, drafts, beta, tau):
    res = [O.verify(logits[b], drafts[b].tolist(), beta, tau) for b in range(logits.shape[0])]
    return [a for a, _ in res], [t for _, t in res]


def test_static_scratch_variant_matches_on_two_calls_in_a_row():
    from paper_2203_16487_b200 import binding
    rng = np.random.default_rng(2024)
    cases = [_case(rng, 9, 25, 32768), _case(rng, 3, 4, 1500)]   # 2nd call: fewer rows, fewer tiles
    dev = [(torch.from_numpy(l).cuda(), torch.from_numpy(d).cuda()) for l, d in cases]
    acc = torch.empty(9, dtype=torch.int32, device="cuda")
    bif = torch.empty(9, dtype=torch.int32, device="cuda")
    torch.cuda.synchronize()
    for beta, tau in [(3, 1.0), (1, 0.0), (5, 3.0)]:
        for (logits, drafts), (lg, dr) in zip(cases, dev):
            B = lg.shape[0]
            ref_a, ref_b = binding.accept_scan(lg, dr, beta, tau)
            a, b = binding.accept_scan_static(lg, dr, beta, tau, acc[:B], bif[:B])
            torch.cuda.synchronize()
            o_a, o_b = _oracle(logits, drafts, beta, tau)
            assert a.cpu().tolist() == o_a and b.cpu().tolist() == o_b, (beta, tau, B)   # integer results: bit-exact
            assert torch.equal(a.cpu(), ref_a.cpu()) and torch.equal(b.cpu(), ref_b.cpu()), (beta, tau, B)


def test_static_scratch_variant_long_blocks():
    """Blocks of more than 256 rows per sequence take the scan's second code path (no per-row flag byte)."""
    from paper_2203_16487_b200 import binding
    rng = np.random.default_rng(7)
    B, k, V = 2, 300, 700
    logits = (rng.standard_normal((B, k + 1, V)) * 3).astype(np.float32)
    drafts = logits.argmax(axis=2)[:, :k].astype(np.int32)
    drafts[0, 280] = int(np.argmin(logits[0, 280]))          # sequence 0 stops beyond row 256, sequence 1 accepts everything
    lg, dr = torch.from_numpy(logits).cuda(), torch.from_numpy(drafts).cuda()
    for _ in range(2):
        a, b = binding.accept_scan_static(lg, dr, 2, 0.5)
        torch.cuda.synchronize()
        o_a, o_b = _oracle(logits, drafts, 2, 0.5)
        assert o_a == [280, 300]
        assert a.cpu().tolist() == o_a and b.cpu().tolist() == o_b


def test_static_scratch_variant_rejects_sizes_beyond_its_array():
    from paper_2203_16487_b200 import binding
    lg = torch.zeros((200, 26, 8), dtype=torch.float32, device="cuda")          # 5200 rows > 4096
    dr = torch.zeros((200, 25), dtype=torch.int32, device="cuda")
    with pytest.raises(binding.SpecDecError) as e:
        binding.accept_scan_static(lg, dr, 3, 1.0)
    assert e.value.code == -3 and "4096" in str(e.value)
    lg = torch.zeros((1, 2, 70000), dtype=torch.float32, device="cuda")         # V > 65536
    dr = torch.zeros((1, 1), dtype=torch.int32, device="cuda")
    with pytest.raises(binding.SpecDecError) as e:
        binding.accept_scan_static(lg, dr, 3, 1.0)
    assert e.value.code == -3
    lg = torch.zeros((1, 3501, 4), dtype=torch.float32, device="cuda")          # k + 1 > 2048 rows in one block
    dr = torch.zeros((1, 3500), dtype=torch.int32, device="cuda")
    with pytest.raises(binding.SpecDecError) as e:
        binding.accept_scan_static(lg, dr, 3, 1.0)
    assert e.value.code == -3 and "2048" in str(e.value)
