"""Small builders shared by the tests (inputs only, no method arithmetic)."""
from __future__ import annotations

import numpy as np

from paper_2607_20475_b200 import workloads as wl


def make_sample(logits, mode, *, dtype=wl.DTYPE_F32, temperature=None, top_k=None, top_p=None, min_p=None,
                rep=None, freq=None, pres=None, seed=None, offset=None, bitmask=None,
                hist=None, bias=None, name="custom") -> wl.SampleWorkload:
    """hist: list (per row) of dict id->count; bias: list (per row) of dict id->value."""
    x = np.asarray(logits, dtype=np.float32)
    B, V = x.shape
    d = wl._defaults(B)
    d["mode"][:] = np.asarray(mode, dtype=np.uint32)
    for key, val in (("temperature", temperature), ("top_k", top_k), ("top_p", top_p), ("min_p", min_p),
                     ("rep_penalty", rep), ("freq_penalty", freq), ("pres_penalty", pres),
                     ("seed", seed), ("offset", offset)):
        if val is not None:
            d[key][:] = np.asarray(val, dtype=d[key].dtype)
    kw = {}
    if hist is not None:
        H = max(1, max(len(h) for h in hist))
        ids = np.zeros((B, H), np.int32); cnt = np.zeros((B, H), np.int32); ln = np.zeros(B, np.int32)
        for r, h in enumerate(hist):
            for j, (i, c) in enumerate(h.items()):
                ids[r, j] = i; cnt[r, j] = c
            ln[r] = len(h)
        kw.update(hist_ids=ids, hist_counts=cnt, hist_len=ln)
    if bias is not None:
        L = max(1, max(len(h) for h in bias))
        ids = np.zeros((B, L), np.int32); vals = np.zeros((B, L), np.float32); ln = np.zeros(B, np.int32)
        for r, h in enumerate(bias):
            for j, (i, v) in enumerate(h.items()):
                ids[r, j] = i; vals[r, j] = v
            ln[r] = len(h)
        kw.update(bias_ids=ids, bias_vals=vals, bias_len=ln)
    if bitmask is not None:
        kw["bitmask"] = np.asarray(bitmask, dtype=np.uint32).reshape(B, -1)
    lg = wl.f32_to_bf16_bits(x) if dtype == wl.DTYPE_BF16 else x
    return wl.SampleWorkload(name=name, B=B, V=V, dtype=dtype, logits=lg, **d, **kw)


def pack_bits(allowed: np.ndarray) -> np.ndarray:
    """bool [B, V] -> packed uint32 [B, ceil(V/32)], bit (i&31) of word (i>>5)."""
    B, V = allowed.shape
    W = (V + 31) // 32
    bits = np.zeros((B, W * 32), dtype=bool)
    bits[:, :V] = allowed
    return np.packbits(bits.reshape(B, W, 32), axis=2, bitorder="little").view(np.uint32).reshape(B, W)


def py_philox4x32_10(ctr, key):
    """Independent pure-Python Philox4x32-10 (second implementation, pins the oracle's)."""
    c = [int(v) & 0xFFFFFFFF for v in ctr]
    k = [int(v) & 0xFFFFFFFF for v in key]
    for _ in range(10):
        p0 = 0xD2511F53 * c[0]
        p1 = 0xCD9E8D57 * c[2]
        c = [((p1 >> 32) ^ c[1] ^ k[0]) & 0xFFFFFFFF, p1 & 0xFFFFFFFF,
             ((p0 >> 32) ^ c[3] ^ k[1]) & 0xFFFFFFFF, p0 & 0xFFFFFFFF]
        k = [(k[0] + 0x9E3779B9) & 0xFFFFFFFF, (k[1] + 0xBB67AE85) & 0xFFFFFFFF]
    return c


def py_uniforms(seed, pos, request):
    r = py_philox4x32_10([pos & 0xFFFFFFFF, (pos >> 32) & 0xFFFFFFFF, request, 0],
                         [seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF])
    u = lambda v: ((v >> 8) + 0.5) / 16777216.0
    return u(r[0]), u(r[1])
