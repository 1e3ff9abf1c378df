"""Seeded synthetic inputs shaped like the paper's sampling workloads.

This module only *draws inputs*: logit matrices, per-request parameters, mode
bits, grammar bitmasks, token histories, bias lists, draft tokens and draft
distributions.  Neither the CUDA path nor the CPU oracle lives here and neither
is imported; both consume what these functions return, as numpy arrays on the
host.  The sizes follow the paper's evaluation range (vocabularies 2^13..2^18,
bf16 and fp32 logits, low-entropy spiked rows, rank-Zipf rows and flat rows,
Section 4 of the paper); they are stand-ins for real model logits, which are
not available offline.

Mode bits follow the paper's bit-level indicator table (Section 3.5).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, Optional

import numpy as np

# Bit-level indicators (Section 3.5, indicator table).
GRAMMAR = 0x001
REPETITION = 0x002
FREQUENCY = 0x004
PRESENCE = 0x008
BIAS = 0x010
TEMPERATURE = 0x020
GREEDY = 0x040
TOP_K = 0x080
TOP_P = 0x100
MIN_P = 0x200
LOGPROBS = 0x400  # reserved, not consumed

DTYPE_F32 = 0
DTYPE_BF16 = 1

BASE_SEED = 20260000


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even fp32 -> bf16, returned as uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to fp32."""
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


@dataclass
class SampleWorkload:
    """Inputs of one singular-mode call (all host numpy arrays)."""

    name: str
    B: int
    V: int
    dtype: int                      # DTYPE_F32 / DTYPE_BF16
    logits: np.ndarray              # [B, V] float32, or uint16 bf16 bit patterns
    mode: np.ndarray                # [B] uint32
    temperature: np.ndarray         # [B] float32
    top_k: np.ndarray               # [B] int32
    top_p: np.ndarray               # [B] float32
    min_p: np.ndarray               # [B] float32
    rep_penalty: np.ndarray         # [B] float32
    freq_penalty: np.ndarray        # [B] float32
    pres_penalty: np.ndarray        # [B] float32
    seed: np.ndarray                # [B] uint64
    offset: np.ndarray              # [B] uint64
    bitmask: Optional[np.ndarray] = None      # [B, ceil(V/32)] uint32
    hist_ids: Optional[np.ndarray] = None     # [B, Hmax] int32 (unique per row)
    hist_counts: Optional[np.ndarray] = None  # [B, Hmax] int32
    hist_len: Optional[np.ndarray] = None     # [B] int32
    bias_ids: Optional[np.ndarray] = None     # [B, Lmax] int32 (unique per row)
    bias_vals: Optional[np.ndarray] = None    # [B, Lmax] float32
    bias_len: Optional[np.ndarray] = None     # [B] int32
    meta: Dict = field(default_factory=dict)

    def logits_f32(self) -> np.ndarray:
        if self.dtype == DTYPE_BF16:
            return bf16_bits_to_f32(self.logits)
        return self.logits

    def input_bytes(self) -> int:
        """Bytes the call must read at least once (logits, mask, lists)."""
        n = self.logits.nbytes
        if self.bitmask is not None and np.any(self.mode & GRAMMAR):
            n += self.bitmask.nbytes
        if self.hist_len is not None:
            n += int(self.hist_len.sum()) * 8
        if self.bias_len is not None:
            n += int(self.bias_len.sum()) * 8
        return n


@dataclass
class VerifyWorkload:
    """Inputs of one multistep (speculative verification) call."""

    name: str
    B: int
    K: int
    V: int
    sample: SampleWorkload          # per-request parameters; logits = target [B*(K+1), V]
    draft_tokens: np.ndarray        # [B, K] int32
    draft_probs: np.ndarray         # [B, K, V] float32
    meta: Dict = field(default_factory=dict)


@dataclass
class TopKWorkload:
    name: str
    B: int
    V: int
    dtype: int
    logits: np.ndarray
    meta: Dict = field(default_factory=dict)

    def logits_f32(self) -> np.ndarray:
        if self.dtype == DTYPE_BF16:
            return bf16_bits_to_f32(self.logits)
        return self.logits


# --------------------------------------------------------------------------- rows
def _row_spiked(rng, V, boost, n_ids, sigma=1.0):
    x = rng.standard_normal(V).astype(np.float32) * np.float32(sigma)
    ids = rng.choice(V, size=n_ids, replace=False)
    x[ids] += np.float32(boost)
    return x


def _row_zipf(rng, V, s):
    """Rank-Zipf row: logit = -s*ln(rank), ranks a random permutation, so that
    probabilities at unit temperature are proportional to rank^-s."""
    rank = rng.permutation(V).astype(np.float64) + 1.0
    return (-s * np.log(rank)).astype(np.float32)


def _row_flat(rng, V, sigma):
    return (rng.standard_normal(V) * sigma).astype(np.float32)


def _mixture_row(rng, r, V, boost=10.0, zipf_s=1.1, flat_sigma=0.5):
    regime = r % 3
    if regime == 0:
        return _row_spiked(rng, V, boost, int(rng.integers(1, 5)))
    if regime == 1:
        return _row_zipf(rng, V, zipf_s)
    return _row_flat(rng, V, flat_sigma)


def _history(rng, B, V, n_tokens):
    """Token history of n_tokens ids drawn uniformly with replacement per row,
    aggregated to unique (id, count) lists padded to a common width."""
    ids = np.zeros((B, n_tokens), dtype=np.int32)
    cnt = np.zeros((B, n_tokens), dtype=np.int32)
    ln = np.zeros(B, dtype=np.int32)
    for r in range(B):
        toks = rng.integers(0, V, size=n_tokens)
        u, c = np.unique(toks, return_counts=True)
        perm = rng.permutation(len(u))          # lists carry no ordering promise
        ids[r, : len(u)] = u[perm]
        cnt[r, : len(u)] = c[perm]
        ln[r] = len(u)
    return ids, cnt, ln


def _bias(rng, B, V, n_entries, lo=-5.0, hi=5.0):
    ids = np.zeros((B, n_entries), dtype=np.int32)
    vals = np.zeros((B, n_entries), dtype=np.float32)
    for r in range(B):
        ids[r] = rng.choice(V, size=n_entries, replace=False)
        vals[r] = rng.uniform(lo, hi, size=n_entries).astype(np.float32)
    return ids, vals, np.full(B, n_entries, dtype=np.int32)


def _defaults(B):
    return dict(
        mode=np.zeros(B, dtype=np.uint32),
        temperature=np.ones(B, dtype=np.float32),
        top_k=np.zeros(B, dtype=np.int32),
        top_p=np.ones(B, dtype=np.float32),
        min_p=np.zeros(B, dtype=np.float32),
        rep_penalty=np.ones(B, dtype=np.float32),
        freq_penalty=np.zeros(B, dtype=np.float32),
        pres_penalty=np.zeros(B, dtype=np.float32),
        seed=np.zeros(B, dtype=np.uint64),
        offset=np.zeros(B, dtype=np.uint64),
    )


def _stochastic_params(rng, d, r, ks, ps, thetas):
    d["temperature"][r] = np.float32(rng.uniform(0.5, 1.5))
    d["mode"][r] |= TEMPERATURE
    k = int(rng.choice(ks))
    p = float(rng.choice(ps))
    th = float(rng.choice(thetas))
    if k > 0:
        d["top_k"][r] = k
        d["mode"][r] |= TOP_K
    if p < 1.0:
        d["top_p"][r] = np.float32(p)
        d["mode"][r] |= TOP_P
    if th > 0.0:
        d["min_p"][r] = np.float32(th)
        d["mode"][r] |= MIN_P


# --------------------------------------------------------------------------- configs
def config1(B: int = 4, V: int = 32768) -> SampleWorkload:
    """Singular mode, tiny: greedy / temp+top-k / temp+top-p / temp+min-p rows."""
    rng = np.random.default_rng(BASE_SEED + 1)
    x = rng.standard_normal((B, V)).astype(np.float32)
    ids = rng.choice(V, size=3, replace=False)
    x[0, ids] += np.float32(8.0)
    d = _defaults(B)
    for r in range(B):
        kind = r % 4
        if kind == 0:
            d["mode"][r] = GREEDY
        elif kind == 1:
            d["mode"][r] = TEMPERATURE | TOP_K
            d["temperature"][r] = 0.7
            d["top_k"][r] = 50
        elif kind == 2:
            d["mode"][r] = TEMPERATURE | TOP_P
            d["temperature"][r] = 1.0
            d["top_p"][r] = 0.9
        else:
            d["mode"][r] = TEMPERATURE | MIN_P
            d["temperature"][r] = 1.0
            d["min_p"][r] = 0.05
    return SampleWorkload(name="c1", B=B, V=V, dtype=DTYPE_F32, logits=x, **d)


def config2(B: int = 64, V: int = 131072, dtype: int = DTYPE_BF16, data_seed: int = BASE_SEED + 2,
            n_history: int = 512, n_bias: int = 16) -> SampleWorkload:
    """Singular mode, heterogeneous batch (mixed entropy, half greedy, penalties, bias)."""
    rng = np.random.default_rng(data_seed)
    x = np.empty((B, V), dtype=np.float32)
    for r in range(B):
        x[r] = _mixture_row(rng, r, V)
    d = _defaults(B)
    for r in range(B):
        if r % 2 == 1:
            d["mode"][r] |= GREEDY
        else:
            _stochastic_params(rng, d, r, ks=(0, 20, 50, 1000), ps=(1.0, 0.9, 0.95), thetas=(0.0, 0.05))
        d["mode"][r] |= REPETITION | FREQUENCY | PRESENCE | BIAS
        d["offset"][r] = r
    d["rep_penalty"][:] = 1.1
    d["freq_penalty"][:] = 0.2
    d["pres_penalty"][:] = 0.3
    n_history = min(n_history, V)
    n_bias = min(n_bias, V)
    hi, hc, hl = _history(rng, B, V, n_history)
    bi, bv, bl = _bias(rng, B, V, n_bias)
    logits = f32_to_bf16_bits(x) if dtype == DTYPE_BF16 else x
    return SampleWorkload(name="c2", B=B, V=V, dtype=dtype, logits=logits, hist_ids=hi, hist_counts=hc,
                          hist_len=hl, bias_ids=bi, bias_vals=bv, bias_len=bl, **d)


def config3(B: int = 128, V: int = 262144, data_seed: int = BASE_SEED + 3,
            n_history: int = 512, n_bias: int = 16) -> SampleWorkload:
    """Grammar-constrained singular mode: 2% of ids allowed, masked-argmax rows."""
    rng = np.random.default_rng(data_seed)
    x = np.empty((B, V), dtype=np.float32)
    for r in range(B):
        x[r] = _mixture_row(rng, r, V)
    W = (V + 31) // 32
    bitmask = np.zeros((B, W), dtype=np.uint32)
    n_allowed = max(1, int(0.02 * V))
    for r in range(B):
        allowed = rng.choice(V, size=n_allowed, replace=False)
        bits = np.zeros(W * 32, dtype=bool)
        bits[allowed] = True
        am = int(np.argmax(x[r]))
        bits[am] = (r % 2 == 0)      # even rows keep the raw argmax, odd rows mask it
        packed = np.packbits(bits.reshape(W, 32), axis=1, bitorder="little")
        bitmask[r] = packed.view(np.uint32).reshape(W)
    d = _defaults(B)
    for r in range(B):
        d["mode"][r] |= GRAMMAR | REPETITION | FREQUENCY | PRESENCE | BIAS
        if r % 4 == 0:
            d["mode"][r] |= GREEDY
        else:
            d["mode"][r] |= TEMPERATURE | TOP_K | TOP_P
            d["temperature"][r] = np.float32(rng.uniform(0.5, 1.5))
            d["top_k"][r] = 64
            d["top_p"][r] = 0.95
        d["offset"][r] = r
    d["rep_penalty"][:] = 1.1
    d["freq_penalty"][:] = 0.2
    d["pres_penalty"][:] = 0.3
    hi, hc, hl = _history(rng, B, V, min(n_history, V))
    bi, bv, bl = _bias(rng, B, V, min(n_bias, V))
    return SampleWorkload(name="c3", B=B, V=V, dtype=DTYPE_F32, logits=x, bitmask=bitmask, hist_ids=hi,
                          hist_counts=hc, hist_len=hl, bias_ids=bi, bias_vals=bv, bias_len=bl, **d)


def _draft_distribution(raw: np.ndarray, tau: float, k: int, p: float) -> np.ndarray:
    """Stand-in for a draft model's own sampler settings: the distribution the
    draft tokens are drawn from (temperature, then keep the k most likely, then
    the smallest most-likely set of mass >= p, renormalised).  It is an *input*
    of the verification call; neither implementation under test calls this."""
    z = raw.astype(np.float64) / float(tau)
    order = np.argsort(-z, kind="stable")
    n = len(z)
    if k > 0:
        n = min(n, k)
    w = np.exp(z[order[:n]] - z[order[0]])
    if p < 1.0:
        c = np.cumsum(w)
        n = min(n, int(np.searchsorted(c, p * c[-1], side="left")) + 1)
        w = w[:n]
    q = np.zeros(len(z), dtype=np.float64)
    q[order[:n]] = w / w.sum()
    return q


def config4(B: int = 32, K: int = 4, V: int = 131072, data_seed: int = BASE_SEED + 4) -> VerifyWorkload:
    """Multistep speculative verification, mixed greedy and stochastic requests."""
    rng = np.random.default_rng(data_seed)
    tgt = np.empty((B, K + 1, V), dtype=np.float32)
    for b in range(B):
        for l in range(K + 1):
            tgt[b, l] = _row_spiked(rng, V, 10.0, int(rng.integers(1, 5)))
    d = _defaults(B)
    for b in range(B):
        if b % 2 == 1:
            d["mode"][b] |= GREEDY
        else:
            _stochastic_params(rng, d, b, ks=(0, 20, 50), ps=(1.0, 0.9, 0.95), thetas=(0.0,))
        d["seed"][b] = 1
    tok_rng = np.random.default_rng(1)
    draft_tokens = np.zeros((B, K), dtype=np.int32)
    draft_probs = np.zeros((B, K, V), dtype=np.float32)
    for b in range(B):
        greedy = bool(d["mode"][b] & GREEDY)
        tau = float(d["temperature"][b]) if d["mode"][b] & TEMPERATURE else 1.0
        k = int(d["top_k"][b]) if d["mode"][b] & TOP_K else 0
        p = float(d["top_p"][b]) if d["mode"][b] & TOP_P else 1.0
        for l in range(K):
            raw = tgt[b, l].astype(np.float64) + rng.standard_normal(V) * 0.5
            q = _draft_distribution(raw, tau, k, p).astype(np.float32)
            draft_probs[b, l] = q
            if greedy:
                draft_tokens[b, l] = int(np.argmax(q))
            else:
                q64 = q.astype(np.float64)
                draft_tokens[b, l] = int(tok_rng.choice(V, p=q64 / q64.sum()))
    sw = SampleWorkload(name="c4", B=B, V=V, dtype=DTYPE_F32, logits=tgt.reshape(B * (K + 1), V), **d)
    return VerifyWorkload(name="c4", B=B, K=K, V=V, sample=sw, draft_tokens=draft_tokens,
                          draft_probs=draft_probs)


TOPK_REGIMES = ("spike", "zipf", "normal")
TOPK_KS = (1, 8, 64, 256, 1024, 4096)


def config5(regime: str, B: int = 256, V: int = 262144, dtype: int = DTYPE_F32,
            data_seed: int = BASE_SEED + 5) -> TopKWorkload:
    """Standalone hierarchical top-k sweep input for one regime."""
    rng = np.random.default_rng(data_seed + TOPK_REGIMES.index(regime) if regime in TOPK_REGIMES
                                else data_seed + 17)
    x = np.empty((B, V), dtype=np.float32)
    for r in range(B):
        if regime == "spike":
            x[r] = _row_spiked(rng, V, 12.0, min(8, V))
        elif regime == "zipf":
            x[r] = _row_zipf(rng, V, 1.0)
        elif regime == "normal":
            x[r] = rng.standard_normal(V).astype(np.float32)
        elif regime == "zeros":                    # all ties
            x[r] = 0.0
        elif regime == "const129":                 # U(128.6,128.7) rounds to 129 in bf16
            x[r] = 129.0
        elif regime == "twovalued":
            x[r] = np.where(rng.random(V) < 0.5, 1.0, -1.0).astype(np.float32)
        elif regime == "ascending":                # all of the top-k in the last tile
            x[r] = np.arange(V, dtype=np.float32) / np.float32(V)
        elif regime == "descending":
            x[r] = -np.arange(V, dtype=np.float32) / np.float32(V)
        elif regime == "signedzeros":
            x[r] = np.where(rng.random(V) < 0.5, 0.0, -0.0).astype(np.float32)
        else:
            raise ValueError(regime)
    logits = f32_to_bf16_bits(x) if dtype == DTYPE_BF16 else x
    return TopKWorkload(name=f"c5-{regime}", B=B, V=V, dtype=dtype, logits=logits, meta={"regime": regime})


def sweep_case(B: int, V: int, dtype: int, regime: str, copy: int = 0) -> SampleWorkload:
    """Throughput-sweep input beyond the five configurations: B stochastic rows, all "spiked" (N(0,1) with +10 on
    three ids: low entropy) or all "flat" (N(0,1): high entropy), temperature 0.8, top-k 50, top-p 0.9."""
    rng = np.random.default_rng(BASE_SEED + 700 + 31 * copy + (0 if regime == "spiked" else 1))
    x = rng.standard_normal((B, V)).astype(np.float32)
    if regime == "spiked":
        for r in range(B):
            x[r, rng.choice(V, size=3, replace=False)] += np.float32(10.0)
    d = _defaults(B)
    d["mode"][:] = TEMPERATURE | TOP_K | TOP_P
    d["temperature"][:] = 0.8
    d["top_k"][:] = 50
    d["top_p"][:] = 0.9
    d["offset"][:] = np.arange(B)
    lg = f32_to_bf16_bits(x) if dtype == DTYPE_BF16 else x
    return SampleWorkload(name=f"sweep-{regime}", B=B, V=V, dtype=dtype, logits=lg, **d)
