"""Comparison rules between the CUDA path and the CPU oracle (used by the gpu tests).

Integer results (top-k index sets, greedy tokens, accept lengths) must be
bit-exact.  Sampled / accepted tokens must be bit-exact unless the oracle's
margin for the row (relative distance of a floating-point decision to its
threshold) is below 1e-6; such rows are counted and reported.  Probabilities
agree within 1e-5 relative for fp32 inputs and 2e-3 for bf16 inputs.
"""
from __future__ import annotations

import numpy as np

from paper_2607_20475_b200 import workloads as wl

MARGIN = 1e-6
FLAG_MASK = 0x3     # NO_TOKEN | BADPARAM (FALLBACK is a diagnostic of the CUDA path only)


def compare_sample(got, ref, w, max_near=None):
    B = w.B
    near = ref["margin"] < MARGIN
    rtol = 2e-3 if w.dtype == wl.DTYPE_BF16 else 1e-5
    assert np.array_equal(got["flags"] & FLAG_MASK, ref["flags"] & FLAG_MASK), \
        (np.nonzero((got["flags"] & FLAG_MASK) != (ref["flags"] & FLAG_MASK))[0][:10])
    greedy = (w.mode & wl.GREEDY) != 0
    bad = []
    for b in range(B):
        if greedy[b] or not near[b]:
            if got["token"][b] != ref["token"][b] or got["support"][b] != ref["support"][b]:
                bad.append((b, int(got["token"][b]), int(ref["token"][b]), int(got["support"][b]),
                            int(ref["support"][b]), float(ref["margin"][b]), hex(int(w.mode[b]))))
            elif ref["token"][b] >= 0:
                assert abs(got["prob"][b] - ref["prob"][b]) <= rtol * ref["prob"][b] + 1e-12, \
                    (b, got["prob"][b], ref["prob"][b])
    assert not bad, f"{len(bad)} rows differ (row, got, ref, got_support, ref_support, margin, mode): {bad[:8]}"
    n_near = int(near.sum())
    if max_near is not None:
        assert n_near <= max_near, f"{n_near} near-margin rows"
    return n_near


def compare_verify(got, ref, vw, max_near=None):
    near = ref["margin"] < MARGIN
    assert np.array_equal(got["flags"] & FLAG_MASK, ref["flags"] & FLAG_MASK)
    bad = []
    for b in range(vw.B):
        if near[b] and not (vw.sample.mode[b] & wl.GREEDY):
            continue
        if got["accept_len"][b] != ref["accept_len"][b] or not np.array_equal(got["tokens"][b], ref["tokens"][b]):
            bad.append((b, got["tokens"][b].tolist(), ref["tokens"][b].tolist(), float(ref["margin"][b])))
    assert not bad, f"{len(bad)} requests differ: {bad[:6]}"
    assert np.allclose(got["p_draft"], ref["p_draft"], rtol=1e-5, atol=1e-9), \
        np.abs(got["p_draft"] - ref["p_draft"]).max()
    n_near = int(near.sum())
    if max_near is not None:
        assert n_near <= max_near
    return n_near


def compare_topk(got_vals, got_idx, ref_vals, ref_idx):
    assert np.array_equal(got_idx, ref_idx), np.argwhere(got_idx != ref_idx)[:10]
    assert np.array_equal(got_vals.view(np.uint32), ref_vals.view(np.uint32))
