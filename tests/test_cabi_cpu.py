"""CPU-side checks of the boundary: the library builds for sm_100a, loads, and exports every
symbol include/specdec.h declares.  No compute call is made here."""
import ctypes as C
import os
import re

import pytest

from paper_2203_16487_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "specdec.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(specdec_[a-z_]+)\s*\(", text)))


def test_library_builds_and_exports_every_declared_symbol():
    path = build.build()
    assert os.path.exists(path)
    lib = binding.load_library(path)
    names = _declared()
    assert len(names) >= 14
    for n in names:
        assert hasattr(lib, n), n
    assert set(names) == set(binding.EXPORTS)


def test_no_device_means_error_not_fallback():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    lib = binding.load_library()
    cfg = binding.Config()
    for m in (cfg.verifier, cfg.drafter):
        m.d_model, m.n_heads, m.d_ffn, m.vocab, m.enc_layers, m.dec_layers, m.max_pos = 64, 4, 256, 100, 1, 1, 64
    cfg.k_max, cfg.max_batch, cfg.max_src, cfg.max_tgt, cfg.page_tokens = 4, 1, 8, 8, 16
    t = (binding.Tensor * 1)(binding.Tensor(b"verifier.embed", None, 0, 2, (C.c_longlong * 4)(100, 64, 0, 0)))
    h = C.c_void_p()
    rc = lib.specdec_create(C.byref(cfg), t, 1, None, C.byref(h))
    assert rc == -5 and not h.value
    assert b"no CUDA device" in lib.specdec_last_error(None)
    # argument validation happens before any device work
    cfg.page_tokens = 12
    assert lib.specdec_create(C.byref(cfg), t, 1, None, C.byref(h)) == -1
    cfg.page_tokens, cfg.ffn_activation = 16, 7
    assert lib.specdec_create(C.byref(cfg), t, 1, None, C.byref(h)) == -1
    assert b"ffn_activation" in lib.specdec_last_error(None)
    with pytest.raises(RuntimeError):
        binding.SpecDec(None, {}, None, {}, k_max=1, max_batch=1, max_src=1, max_tgt=1, bf16=False)
