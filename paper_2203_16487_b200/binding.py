"""Thin ctypes binding of the C ABI in include/specdec.h.

Argument marshalling only: every step of the draft -> verify -> commit path
runs in the CUDA library.  PyTorch provides device memory and streams.  If the
library is missing the import of this module fails loudly; there is no
fallback of any kind.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, Optional

import numpy as np
import torch

from . import build as _build

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libspecdec_b200.so")

EXPORTS = [
    "specdec_create", "specdec_destroy", "specdec_encode", "specdec_draft", "specdec_verify",
    "specdec_commit", "specdec_generate", "specdec_generate_host", "specdec_get_output",
    "specdec_accept_scan", "specdec_debug_logits", "specdec_debug_row_stats", "specdec_set_option",
    "specdec_launch_count", "specdec_last_error", "specdec_set_draft_script", "specdec_profile_read",
    "specdec_accept_scan_static", "specdec_debug_trace", "specdec_debug_link_cost", "specdec_debug_mma_rate", "specdec_debug_cluster_round",
    "specdec_debug_integrity", "specdec_debug_mma_rate_bg",
]


class ModelDims(C.Structure):
    _fields_ = [(n, C.c_int) for n in
                ("d_model", "n_heads", "d_ffn", "vocab", "enc_layers", "dec_layers", "max_pos")]


class Config(C.Structure):
    _fields_ = [("verifier", ModelDims), ("drafter", ModelDims)] + [(n, C.c_int) for n in (
        "k_max", "max_batch", "max_src", "max_tgt", "page_tokens",
        "pad_id", "bos_id", "eos_id", "mask_id", "compute_dtype", "ffn_activation")]


class Integrity(C.Structure):
    _fields_ = [("zones", C.c_int32), ("damaged_zones", C.c_int32), ("first_damaged_zone", C.c_int32),
                ("first_nonfinite_buffer", C.c_int32), ("nonfinite", C.c_int64)]


class Tensor(C.Structure):
    _fields_ = [("name", C.c_char_p), ("d_ptr", C.c_void_p), ("dtype", C.c_int), ("ndim", C.c_int),
                ("shape", C.c_longlong * 4)]


class Stats(C.Structure):
    _fields_ = [("iterations", C.c_longlong), ("seq_iterations", C.c_longlong), ("drafted", C.c_longlong),
                ("accepted", C.c_longlong), ("emitted", C.c_longlong),
                ("ms_encode", C.c_double), ("ms_draft", C.c_double), ("ms_verify", C.c_double),
                ("ms_commit", C.c_double), ("ms_total", C.c_double), ("status", C.c_int)]

    def as_dict(self):
        return {n: getattr(self, n) for n, _ in self._fields_}


def load_library(path: str = LIB_PATH) -> C.CDLL:
    if path == LIB_PATH and _build.needs_build():
        try:
            _build.build()              # compile step (nvcc, sm_100a); not a fallback
        except Exception as e:          # a stale library must never pass for the current source
            raise RuntimeError(f"cannot build {path}: {e}") from e
    if not os.path.exists(path):
        raise RuntimeError(f"{path} is missing: build it with `python -m paper_2203_16487_b200.build` "
                           "(there is no fallback path)")
    lib = C.CDLL(path)
    vp, ip, i, f = C.c_void_p, C.c_void_p, C.c_int, C.c_float
    lib.specdec_create.argtypes = [C.POINTER(Config), C.POINTER(Tensor), i, vp, C.POINTER(vp)]
    lib.specdec_destroy.argtypes = [vp]
    lib.specdec_encode.argtypes = [vp, ip, ip, ip, i, i, vp]
    lib.specdec_draft.argtypes = [vp, i, ip, vp]
    lib.specdec_verify.argtypes = [vp, ip, i, i, f, ip, ip, vp]
    lib.specdec_commit.argtypes = [vp, ip, ip, vp]
    lib.specdec_generate.argtypes = [vp, ip, ip, ip, i, i, i, i, f, ip, i, ip, C.POINTER(Stats), vp]
    lib.specdec_generate_host.argtypes = [vp, ip, ip, ip, i, i, i, i, f, ip, i, ip, C.POINTER(Stats), vp]
    lib.specdec_get_output.argtypes = [vp, ip, i, ip, ip, vp]
    lib.specdec_accept_scan.argtypes = [vp, ip, i, i, i, i, f, ip, ip, vp]
    lib.specdec_accept_scan_static.argtypes = [vp, ip, i, i, i, i, f, ip, ip, vp]
    lib.specdec_debug_logits.argtypes = [vp, i, vp, vp]
    lib.specdec_debug_row_stats.argtypes = [vp, vp, vp]
    lib.specdec_debug_link_cost.argtypes = [vp, i, i, C.POINTER(C.c_double)]
    lib.specdec_debug_mma_rate.argtypes = [vp, i, i, i, C.POINTER(C.c_double), C.POINTER(C.c_double)]
    lib.specdec_debug_cluster_round.argtypes = [vp, i, i, i, C.POINTER(C.c_double)]
    lib.specdec_debug_trace.argtypes = [vp, C.POINTER(C.c_longlong), i]
    lib.specdec_set_option.argtypes = [vp, C.c_char_p, i]
    lib.specdec_set_draft_script.argtypes = [vp, ip, i, i, vp]
    lib.specdec_profile_read.argtypes = [vp, C.POINTER(C.c_double), C.POINTER(C.c_longlong)]
    lib.specdec_launch_count.argtypes = [vp]
    lib.specdec_launch_count.restype = C.c_longlong
    lib.specdec_last_error.argtypes = [vp]
    lib.specdec_last_error.restype = C.c_char_p
    for name in EXPORTS:
        if name not in ("specdec_launch_count", "specdec_last_error"):
            getattr(lib, name).restype = i
    return lib


_lib: Optional[C.CDLL] = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        _lib = load_library()
    return _lib


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else C.c_void_p(t.data_ptr())


def _dims(d) -> ModelDims:
    return ModelDims(d.d_model, d.n_heads, d.d_ffn, d.vocab, d.enc_layers, d.dec_layers, d.max_pos)


class SpecDecError(RuntimeError):
    def __init__(self, code, msg):
        super().__init__(f"specdec error {code}: {msg}")
        self.code = code


class SpecDec:
    """One handle: two models, their arena and one decoding session at a time."""

    def __init__(self, verifier_dims, verifier_w: Dict[str, np.ndarray], drafter_dims,
                 drafter_w: Dict[str, np.ndarray], *, k_max: int, max_batch: int, max_src: int, max_tgt: int,
                 bf16: bool, page_tokens: int = 16, pad_id=0, bos_id=1, eos_id=2, mask_id=3, device="cuda:0",
                 activation: str = "relu"):
        if not torch.cuda.is_available():
            raise RuntimeError("SpecDec needs a CUDA device: the library has no CPU path")
        self._lib = lib()
        self.device = torch.device(device)
        self.k_max, self.max_batch, self.max_src, self.max_tgt = k_max, max_batch, max_src, max_tgt
        self.vocab = verifier_dims.vocab
        cfg = Config(_dims(verifier_dims), _dims(drafter_dims), k_max, max_batch, max_src, max_tgt, page_tokens,
                     pad_id, bos_id, eos_id, mask_id, 1 if bf16 else 0, {"relu": 0, "gelu": 1}[activation])
        keep, tensors = [], []
        for prefix, w in (("verifier.", verifier_w), ("drafter.", drafter_w)):
            for name, a in w.items():
                t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(self.device)
                keep.append(t)
                shape = (C.c_longlong * 4)(*(list(t.shape) + [0] * (4 - t.dim())))
                tensors.append(Tensor((prefix + name).encode(), t.data_ptr(), 0, t.dim(), shape))
        arr = (Tensor * len(tensors))(*tensors)
        h = C.c_void_p()
        with torch.cuda.device(self.device):
            rc = self._lib.specdec_create(C.byref(cfg), arr, len(tensors), _stream(), C.byref(h))
        if rc != 0:
            raise SpecDecError(rc, self._lib.specdec_last_error(None).decode())
        self._h = h
        del keep
        self.B = 0
        if os.environ.get("SPECDEC_DEBUG_CHECKS") == "1":        # every step call ends with the integrity check
            self.set_option("debug_checks", 1)
        self._bufs = {}

    # ------------------------------------------------------------------ helpers
    def _check(self, rc):
        if rc != 0:
            raise SpecDecError(rc, self._lib.specdec_last_error(self._h).decode())

    def _i32(self, a) -> torch.Tensor:
        if isinstance(a, torch.Tensor):
            return a.to(device=self.device, dtype=torch.int32).contiguous()
        return torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(self.device)

    def close(self):
        if getattr(self, "_h", None):
            self._lib.specdec_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def set_option(self, name: str, value: int):
        self._check(self._lib.specdec_set_option(self._h, name.encode(), int(value)))

    def set_draft_script(self, script):
        """script [B, n] int32 (or None): entries >= 0 replace the drafter's output at that target index."""
        if script is None:
            self._check(self._lib.specdec_set_draft_script(self._h, None, 0, 0, _stream()))
            return
        t = self._i32(script)
        self._check(self._lib.specdec_set_draft_script(self._h, _ptr(t), int(t.shape[0]), int(t.shape[1]), _stream()))
        torch.cuda.current_stream().synchronize()

    def profile_read(self):
        ms, n = C.c_double(), C.c_longlong()
        self._check(self._lib.specdec_profile_read(self._h, C.byref(ms), C.byref(n)))
        return ms.value, n.value

    def link_cost(self, n_links: int = 64, grid: int = 148) -> float:
        """Microseconds per kernel boundary in a chain of dependent launches (diagnostics)."""
        us = C.c_double()
        self._check(self._lib.specdec_debug_link_cost(self._h, n_links, grid, C.byref(us)))
        return us.value

    def mma_rate(self, bn: int, two_sm: bool = False, n_mma: int = 4096):
        """(issue, completion) clocks per tcgen05.mma with shared-memory-resident operands (diagnostics)."""
        a, b = C.c_double(), C.c_double()
        self._check(self._lib.specdec_debug_mma_rate(self._h, bn, 1 if two_sm else 0, n_mma, C.byref(a), C.byref(b)))
        return a.value, b.value

    def mma_rate_bg(self, bn: int, two_sm: bool, n_mma: int, bg_stages: int, commit_every: int = 0):
        """(issue clocks, completion clocks) per tcgen05.mma and the bytes per clock a background bulk-copy stream
        landed in shared memory meanwhile; commit_every > 0 adds a tcgen05.commit after that many MMAs (diagnostics)."""
        a, b, c = C.c_double(), C.c_double(), C.c_double()
        self._check(self._lib.specdec_debug_mma_rate_bg(self._h, bn, 1 if two_sm else 0, n_mma, bg_stages, commit_every,
                                                        C.byref(a), C.byref(b), C.byref(c)))
        return a.value, b.value, c.value

    def cluster_round(self, cluster_size: int = 16, bytes_per_peer: int = 0, rounds: int = 64) -> float:
        """Nanoseconds per all-to-all exchange round inside one thread-block cluster (diagnostics)."""
        ns = C.c_double()
        self._check(self._lib.specdec_debug_cluster_round(self._h, cluster_size, bytes_per_peer, rounds, C.byref(ns)))
        return ns.value

    def integrity(self) -> dict:
        """Red zones behind every arena block and a NaN / Inf scan of activations and caches (synchronises)."""
        rep = Integrity()
        self._check(self._lib.specdec_debug_integrity(self._h, C.byref(rep), _stream()))
        return {n: int(getattr(rep, n)) for n, _ in Integrity._fields_}

    def trace(self, n: int):
        buf = (C.c_longlong * n)()
        self._check(self._lib.specdec_debug_trace(self._h, buf, n))
        return list(buf)

    def last_error(self) -> str:
        return self._lib.specdec_last_error(self._h).decode()

    def launch_count(self) -> int:
        return int(self._lib.specdec_launch_count(self._h))

    # ------------------------------------------------------------------ the path
    def encode(self, src, src_len, max_tgt=None):
        src, src_len = self._i32(src), self._i32(src_len)
        mt = None if max_tgt is None else self._i32(max_tgt)
        self.B, S = int(src.shape[0]), int(src.shape[1])
        self._check(self._lib.specdec_encode(self._h, _ptr(src), _ptr(src_len), _ptr(mt), self.B, S, _stream()))

    def _buf(self, name, shape):
        """Persistent device buffers: stable addresses let the library replay its CUDA graphs."""
        key = (name,) + tuple(shape)
        if key not in self._bufs:
            self._bufs[key] = torch.zeros(shape, dtype=torch.int32, device=self.device)
        return self._bufs[key]

    def draft(self, k: int) -> torch.Tensor:
        """Drafts [B,k]; the returned tensor is reused by the next call of the same shape."""
        out = self._buf("draft", (self.B, k))
        out.fill_(-1)
        self._check(self._lib.specdec_draft(self._h, k, _ptr(out), _stream()))
        return out

    def verify(self, drafts, beta: int, tau: float):
        """(accepted [B], bifurcation token [B]); the returned tensors are reused by the next call."""
        k = int(drafts.shape[1])
        buf = self._buf("vdraft", (self.B, k))
        buf.copy_(self._i32(drafts))
        return self.verify_raw(buf, beta, tau, self._buf("acc", (self.B,)), self._buf("bif", (self.B,)))

    def verify_raw(self, drafts: torch.Tensor, beta: int, tau: float, acc: torch.Tensor, bif: torch.Tensor):
        """No staging: `drafts` [B,k], `acc`, `bif` [B] are int32 device tensors owned by the caller."""
        k = int(drafts.shape[1])
        self._check(self._lib.specdec_verify(self._h, _ptr(drafts), k, beta, float(tau), _ptr(acc), _ptr(bif), _stream()))
        return acc, bif

    def commit(self, keep=None, nxt=None):
        keep = None if keep is None else self._i32(keep)
        nxt = None if nxt is None else self._i32(nxt)
        self._check(self._lib.specdec_commit(self._h, _ptr(keep), _ptr(nxt), _stream()))

    def output(self):
        out = torch.zeros((self.B, self.max_tgt), dtype=torch.int32, device=self.device)
        n = torch.zeros(self.B, dtype=torch.int32, device=self.device)
        fin = torch.zeros(self.B, dtype=torch.int32, device=self.device)
        self._check(self._lib.specdec_get_output(self._h, _ptr(out), self.max_tgt, _ptr(n), _ptr(fin), _stream()))
        return out, n, fin

    def generate(self, src, src_len, max_tgt, k: int, beta: int, tau: float, want_stats: bool = True):
        """Device-resident inputs -> (ids [B,max_tgt] tensor, lengths [B] tensor, stats dict)."""
        src, src_len = self._i32(src), self._i32(src_len)
        mt = None if max_tgt is None else self._i32(max_tgt)
        self.B, S = int(src.shape[0]), int(src.shape[1])
        out = torch.zeros((self.B, self.max_tgt), dtype=torch.int32, device=self.device)
        n = torch.zeros(self.B, dtype=torch.int32, device=self.device)
        st = Stats()
        self._check(self._lib.specdec_generate(self._h, _ptr(src), _ptr(src_len), _ptr(mt), self.B, S, k, beta,
                                               float(tau), _ptr(out), self.max_tgt, _ptr(n),
                                               C.byref(st) if want_stats else None, _stream()))
        return out, n, st.as_dict()

    def generate_host(self, src: torch.Tensor, src_len: torch.Tensor, max_tgt: Optional[torch.Tensor],
                      out: torch.Tensor, out_len: torch.Tensor, k: int, beta: int, tau: float,
                      want_stats: bool = False):
        """HOST int32 tensors in (ideally pinned), HOST tensors out; copies are inside the call."""
        assert not src.is_cuda and not out.is_cuda and src.dtype == torch.int32 and out.dtype == torch.int32
        B, S = int(src.shape[0]), int(src.shape[1])
        self.B = B
        st = Stats()
        self._check(self._lib.specdec_generate_host(self._h, _ptr(src), _ptr(src_len), _ptr(max_tgt), B, S, k, beta,
                                                    float(tau), _ptr(out), int(out.shape[1]), _ptr(out_len),
                                                    C.byref(st) if want_stats else None, _stream()))
        return st.as_dict()

    # ------------------------------------------------------------------ parity helpers
    def debug_logits(self, which: int, rows: int) -> torch.Tensor:
        out = torch.zeros((rows, self.vocab), dtype=torch.float32, device=self.device)
        self._check(self._lib.specdec_debug_logits(self._h, which, _ptr(out), _stream()))
        return out

    def debug_row_stats(self, k: int) -> torch.Tensor:
        out = torch.zeros((self.B, k + 1, 6), dtype=torch.float32, device=self.device)
        self._check(self._lib.specdec_debug_row_stats(self._h, _ptr(out), _stream()))
        return out


def accept_scan(logits: torch.Tensor, drafts: torch.Tensor, beta: int, tau: float):
    """The acceptance rule alone on fp32 logits [B,k+1,V] (device tensors)."""
    assert logits.is_cuda and logits.dtype == torch.float32 and logits.is_contiguous()
    B, k1, V = logits.shape
    drafts = drafts.to(device=logits.device, dtype=torch.int32).contiguous()
    acc = torch.empty(B, dtype=torch.int32, device=logits.device)
    bif = torch.empty(B, dtype=torch.int32, device=logits.device)
    rc = lib().specdec_accept_scan(_ptr(logits), _ptr(drafts), B, k1 - 1, V, beta, float(tau), _ptr(acc), _ptr(bif),
                                   _stream())
    if rc != 0:
        raise SpecDecError(rc, lib().specdec_last_error(None).decode())
    return acc, bif


def accept_scan_static(logits: torch.Tensor, drafts: torch.Tensor, beta: int, tau: float,
                       acc: Optional[torch.Tensor] = None, bif: Optional[torch.Tensor] = None):
    """specdec_accept_scan_static: the acceptance rule for callers that cannot allocate device memory
    (the partial statistics sit in an array compiled into the library).  Pass preallocated `acc` and
    `bif` [B] int32 device tensors to keep the call itself free of any allocation."""
    assert logits.is_cuda and logits.dtype == torch.float32 and logits.is_contiguous()
    B, k1, V = logits.shape
    assert drafts.is_cuda and drafts.dtype == torch.int32 and drafts.is_contiguous()
    if acc is None:
        acc = torch.empty(B, dtype=torch.int32, device=logits.device)
    if bif is None:
        bif = torch.empty(B, dtype=torch.int32, device=logits.device)
    rc = lib().specdec_accept_scan_static(_ptr(logits), _ptr(drafts), B, k1 - 1, V, beta, float(tau), _ptr(acc),
                                          _ptr(bif), _stream())
    if rc != 0:
        raise SpecDecError(rc, lib().specdec_last_error(None).decode())
    return acc, bif
