"""ctypes face of the C oracle (oracle/sonic_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by tests, by the smoke check and by the
benchmark's CPU-baseline leg.  The product package never imports this module.
All arrays are host numpy arrays; bf16 logits are widened to fp32 exactly
before they reach the C code.
"""
from __future__ import annotations

import ctypes as C
from typing import Optional

import numpy as np

from . import build as _build

_lib = None


class _Args(C.Structure):
    _fields_ = [
        ("B", C.c_int32), ("V", C.c_int32), ("K", C.c_int32),
        ("logits", C.c_void_p), ("row_stride", C.c_int64),
        ("mode", C.c_void_p),
        ("bitmask", C.c_void_p), ("bitmask_stride", C.c_int64),
        ("temperature", C.c_void_p), ("top_k", C.c_void_p), ("top_p", C.c_void_p), ("min_p", C.c_void_p),
        ("rep_penalty", C.c_void_p), ("freq_penalty", C.c_void_p), ("pres_penalty", C.c_void_p),
        ("hist_ids", C.c_void_p), ("hist_counts", C.c_void_p), ("hist_len", C.c_void_p),
        ("hist_stride", C.c_int32),
        ("bias_ids", C.c_void_p), ("bias_vals", C.c_void_p), ("bias_len", C.c_void_p),
        ("bias_stride", C.c_int32),
        ("seed", C.c_void_p), ("offset", C.c_void_p),
        ("draft_tokens", C.c_void_p), ("draft_probs", C.c_void_p),
    ]


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(_build.build())
        _lib.oracle_u01.restype = C.c_double
        _lib.oracle_u01.argtypes = [C.c_uint32]
        _lib.oracle_support.restype = C.c_int
        _lib.oracle_processed_row.restype = C.c_int
        _lib.oracle_prologue.restype = C.c_int
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data


def _c(a, dtype):
    return None if a is None else np.ascontiguousarray(a, dtype=dtype)


class _Packed:
    """Keeps the contiguous arrays alive next to the struct that points at them."""

    def __init__(self, w, K=0, draft_tokens=None, draft_probs=None, logits=None):
        x = w.logits_f32() if logits is None else logits
        self.logits = _c(x, np.float32)
        rows, V = self.logits.shape
        self.keep = dict(
            mode=_c(w.mode, np.uint32), bitmask=_c(w.bitmask, np.uint32),
            temperature=_c(w.temperature, np.float32), top_k=_c(w.top_k, np.int32),
            top_p=_c(w.top_p, np.float32), min_p=_c(w.min_p, np.float32),
            rep_penalty=_c(w.rep_penalty, np.float32), freq_penalty=_c(w.freq_penalty, np.float32),
            pres_penalty=_c(w.pres_penalty, np.float32),
            hist_ids=_c(w.hist_ids, np.int32), hist_counts=_c(w.hist_counts, np.int32),
            hist_len=_c(w.hist_len, np.int32),
            bias_ids=_c(w.bias_ids, np.int32), bias_vals=_c(w.bias_vals, np.float32),
            bias_len=_c(w.bias_len, np.int32),
            seed=_c(w.seed, np.uint64), offset=_c(w.offset, np.uint64),
            draft_tokens=_c(draft_tokens, np.int32), draft_probs=_c(draft_probs, np.float32),
        )
        k = self.keep
        a = _Args()
        a.B = w.B
        a.V = V
        a.K = K
        a.logits = _p(self.logits)
        a.row_stride = V
        a.mode = _p(k["mode"])
        a.bitmask = _p(k["bitmask"])
        a.bitmask_stride = 0 if k["bitmask"] is None else k["bitmask"].shape[-1]
        for name in ("temperature", "top_k", "top_p", "min_p", "rep_penalty", "freq_penalty", "pres_penalty",
                     "hist_ids", "hist_counts", "hist_len", "bias_ids", "bias_vals", "bias_len", "seed",
                     "offset", "draft_tokens", "draft_probs"):
            setattr(a, name, _p(k[name]))
        a.hist_stride = 0 if k["hist_ids"] is None else k["hist_ids"].shape[1]
        a.bias_stride = 0 if k["bias_ids"] is None else k["bias_ids"].shape[1]
        self.args = a


def philox4x32_10(ctr, key):
    c = (C.c_uint32 * 4)(*[int(v) & 0xFFFFFFFF for v in ctr])
    k = (C.c_uint32 * 2)(*[int(v) & 0xFFFFFFFF for v in key])
    o = (C.c_uint32 * 4)()
    lib().oracle_philox4x32_10(c, k, o)
    return [int(v) for v in o]


def u01(r: int) -> float:
    return float(lib().oracle_u01(C.c_uint32(int(r) & 0xFFFFFFFF)))


def uniforms(seed: int, pos: int, request: int):
    ua, ud = C.c_double(), C.c_double()
    lib().oracle_uniforms(C.c_uint64(seed), C.c_uint64(pos), C.c_uint32(request), C.byref(ua), C.byref(ud))
    return ua.value, ud.value


def processed_row(w, b: int) -> np.ndarray:
    """Processed (post-prologue) fp32 logits of row b of a singular-mode workload."""
    pk = _Packed(w)
    y = np.empty(pk.args.V, dtype=np.float32)
    lib().oracle_processed_row(C.byref(pk.args), C.c_int(b), C.c_void_p(y.ctypes.data))
    return y


def support(w, b: int):
    """Final support of row b in ranking order: (indices, probabilities, margin)."""
    pk = _Packed(w)
    V = pk.args.V
    idx = np.empty(V, dtype=np.int32)
    pr = np.empty(V, dtype=np.float64)
    m = C.c_double()
    n = lib().oracle_support(C.byref(pk.args), C.c_int(b), C.c_void_p(idx.ctypes.data),
                             C.c_void_p(pr.ctypes.data), C.byref(m))
    return idx[:n].copy(), pr[:n].copy(), m.value


def sample(w):
    """Singular mode over a SampleWorkload -> dict(token, prob, flags, support, margin)."""
    pk = _Packed(w)
    B = w.B
    tok = np.empty(B, np.int32)
    prob = np.empty(B, np.float32)
    flags = np.empty(B, np.uint32)
    sup = np.empty(B, np.int32)
    margin = np.empty(B, np.float64)
    lib().oracle_sample(C.byref(pk.args), C.c_void_p(tok.ctypes.data), C.c_void_p(prob.ctypes.data),
                        C.c_void_p(flags.ctypes.data), C.c_void_p(sup.ctypes.data),
                        C.c_void_p(margin.ctypes.data))
    return dict(token=tok, prob=prob, flags=flags, support=sup, margin=margin)


def verify(vw):
    """Multistep mode over a VerifyWorkload -> dict(tokens, accept_len, p_draft, flags, margin)."""
    w = vw.sample
    pk = _Packed(w, K=vw.K, draft_tokens=vw.draft_tokens, draft_probs=vw.draft_probs)
    B, K = vw.B, vw.K
    toks = np.empty((B, K + 1), np.int32)
    acc = np.empty(B, np.int32)
    pd = np.empty((B, max(K, 1)), np.float32)
    flags = np.empty(B, np.uint32)
    margin = np.empty(B, np.float64)
    lib().oracle_verify(C.byref(pk.args), C.c_void_p(toks.ctypes.data), C.c_void_p(acc.ctypes.data),
                        C.c_void_p(pd.ctypes.data), C.c_void_p(flags.ctypes.data),
                        C.c_void_p(margin.ctypes.data))
    return dict(tokens=toks, accept_len=acc, p_draft=pd[:, :K], flags=flags, margin=margin)


def topk(logits_f32: np.ndarray, k: int):
    """Sorted top-k of each row: (values [B,k] descending, indices [B,k]); ties to the lowest index."""
    x = np.ascontiguousarray(logits_f32, dtype=np.float32)
    B, V = x.shape
    vals = np.empty((B, k), np.float32)
    idx = np.empty((B, k), np.int32)
    lib().oracle_topk(C.c_void_p(x.ctypes.data), C.c_int(B), C.c_int(V), C.c_int64(V), C.c_int(k),
                      C.c_void_p(vals.ctypes.data), C.c_void_p(idx.ctypes.data))
    return vals, idx
