"""Pins of the CPU oracle against things other than itself: published Philox
vectors, closed forms, hand-worked examples, brute force on tiny vocabularies,
library routines used as definitions (stable argsort, softmax), the exact
enumeration identity of rejection sampling and chi-squared on many draws."""
import math
import os

import numpy as np
import pytest
from scipy import stats
from scipy.special import softmax

from oracle import oracle
from paper_2607_20475_b200 import workloads as wl
from tests.helpers import make_sample, pack_bits, py_philox4x32_10, py_uniforms

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ------------------------------------------------------------------ Philox
def test_philox_known_answers():
    for line in open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")):
        if line.startswith("#") or not line.strip():
            continue
        v = [int(t, 16) for t in line.split()]
        assert oracle.philox4x32_10(v[0:4], v[4:6]) == v[6:10]
        assert py_philox4x32_10(v[0:4], v[4:6]) == v[6:10]


def test_philox_matches_second_implementation_on_random_counters():
    rng = np.random.default_rng(7)
    for _ in range(200):
        ctr = rng.integers(0, 2**32, size=4).tolist()
        key = rng.integers(0, 2**32, size=2).tolist()
        assert oracle.philox4x32_10(ctr, key) == py_philox4x32_10(ctr, key)


def test_uniform_mapping_is_exact_dyadic_and_keyed_by_seed_position_request():
    # ((r >> 8) + 1/2) / 2^24, so r = 0 -> 2^-25 and r = 2^32-1 -> 1 - 2^-25
    assert oracle.u01(0) == 2.0 ** -25
    assert oracle.u01(0xFFFFFFFF) == 1.0 - 2.0 ** -25
    assert oracle.u01(0x6627E8D5) == ((0x6627E8D5 >> 8) + 0.5) / 2 ** 24
    # counter = (pos_lo, pos_hi, request, 0), key = (seed_lo, seed_hi)
    for seed, pos, req in [(0, 0, 0), (1, 3, 5), (0x123456789ABCDEF0, 0x100000002, 7)]:
        assert oracle.uniforms(seed, pos, req) == py_uniforms(seed, pos, req)
    # (0,0,0) is the all-zero known-answer vector
    ua, ud = oracle.uniforms(0, 0, 0)
    assert ua == ((0x6627E8D5 >> 8) + 0.5) / 2 ** 24 and ud == ((0xE169C58D >> 8) + 0.5) / 2 ** 24


# ---------------------------------------------------------------- prologue
X8 = np.array([[1.0, 3.0, 2.0, 2.0, 0.0, -1.0, 0.5, 2.5]], dtype=np.float32)


def test_prologue_identity_cases():
    rng = np.random.default_rng(3)
    x = rng.standard_normal((1, 257)).astype(np.float32)
    w = make_sample(x, [0])
    assert np.array_equal(oracle.processed_row(w, 0), x[0] + np.float32(0))
    # alpha = 1, beta = gamma = 0 recovers the unpenalised logits
    w = make_sample(x, [wl.REPETITION | wl.FREQUENCY | wl.PRESENCE], rep=[1.0], freq=[0.0], pres=[0.0],
                    hist=[{5: 3, 17: 1, 200: 9}])
    assert np.array_equal(oracle.processed_row(w, 0), x[0] + np.float32(0))
    # parameters are ignored when their bit is clear
    w = make_sample(x, [0], rep=[1.5], freq=[0.3], pres=[0.2], temperature=[0.5],
                    hist=[{5: 3}], bias=[{7: 1.0}])
    assert np.array_equal(oracle.processed_row(w, 0), x[0] + np.float32(0))


def test_prologue_mask_only():
    allowed = np.array([[0, 1, 1, 1, 1, 0, 1, 1]], dtype=bool)
    w = make_sample(X8, [wl.GRAMMAR], bitmask=pack_bits(allowed))
    y = oracle.processed_row(w, 0)
    assert np.all(np.isneginf(y[[0, 5]])) and np.array_equal(y[allowed[0]], X8[0][allowed[0]])


def test_prologue_hand_worked_vector():
    # history {2: twice, 5: once}, alpha=1.25, beta=0.5, gamma=0.25; bias {1: -1.5, 6: +2.25}; tau = 0.7.
    # token 2: ((2/1.25) - 0.5*2) - 0.25 = 0.35 (fp32: 0x1.666668p-2), then /0.7;
    # token 5: ((-1*1.25) - 0.5*1) - 0.25 = -2.0, then /0.7; others x/0.7 (1 and 6 after the bias add).
    mode = wl.REPETITION | wl.FREQUENCY | wl.PRESENCE | wl.BIAS | wl.TEMPERATURE
    w = make_sample(X8, [mode], rep=[1.25], freq=[0.5], pres=[0.25], temperature=[0.7],
                    hist=[{2: 2, 5: 1}], bias=[{1: -1.5, 6: 2.25}])
    y = oracle.processed_row(w, 0)
    expect = [float.fromhex(h) for h in
              ["0x1.6db6dcp+0", "0x1.124924p+1", "0x1.000002p-1", "0x1.6db6dcp+1", "0x0p+0",
               "-0x1.6db6dcp+1", "0x1.f6db6ep+1", "0x1.c92492p+1"]]
    assert y.tolist() == expect
    # without temperature the penalised entries are exactly these fp32 values
    w = make_sample(X8, [mode & ~wl.TEMPERATURE & ~wl.BIAS], rep=[1.25], freq=[0.5], pres=[0.25],
                    hist=[{2: 2, 5: 1}])
    y = oracle.processed_row(w, 0)
    assert y[2] == float.fromhex("0x1.666668p-2") and y[5] == -2.0


def test_prologue_sign_asymmetry_and_zero():
    # positive logits are divided, non-positive ones multiplied (zero stays zero); -0 becomes +0
    x = np.array([[4.0, -4.0, 0.0, -0.0]], dtype=np.float32)
    w = make_sample(x, [wl.REPETITION], rep=[2.0], hist=[{0: 1, 1: 1, 2: 1, 3: 1}])
    y = oracle.processed_row(w, 0)
    assert y.tolist() == [2.0, -8.0, 0.0, 0.0] and not np.signbit(y[3])


# ------------------------------------------------------- ordering / top-k
def brute_rank_order(x):
    """O(V^2) definition: rank = #{j: x_j > x_i or (x_j == x_i and j < i)}."""
    V = len(x)
    order = np.empty(V, dtype=np.int64)
    for i in range(V):
        r = sum(1 for j in range(V) if x[j] > x[i] or (x[j] == x[i] and j < i))
        order[r] = i
    return order


def test_topk_brute_force_with_ties():
    rng = np.random.default_rng(11)
    for V in (1, 2, 7, 33, 64):
        x = rng.integers(-3, 4, size=(3, V)).astype(np.float32)   # many ties
        for k in sorted({1, min(3, V), V}):
            vals, idx = oracle.topk(x, k)
            for b in range(3):
                o = brute_rank_order(x[b])[:k]
                assert idx[b].tolist() == o.tolist()
                assert vals[b].tolist() == x[b][o].tolist()


def test_topk_matches_stable_argsort_and_tie_stress():
    rng = np.random.default_rng(12)
    x = rng.standard_normal((4, 5000)).astype(np.float32)
    x[1] = wl.bf16_bits_to_f32(wl.f32_to_bf16_bits(x[1]))          # coarse values: thousands of ties
    vals, idx = oracle.topk(x, 300)
    for b in range(4):
        o = np.argsort(-x[b], kind="stable")[:300]
        assert idx[b].tolist() == o.tolist()
    for const in (0.0, 129.0):                                     # all-equal rows: indices 0..k-1
        vals, idx = oracle.topk(np.full((2, 1000), const, np.float32), 17)
        assert idx.tolist() == [list(range(17))] * 2 and np.all(vals == const)
    z = np.array([[0.0, -0.0, 0.0, -0.0, 1.0]], dtype=np.float32)  # -0 == +0, lowest index first
    vals, idx = oracle.topk(z, 5)
    assert idx[0].tolist() == [4, 0, 1, 2, 3]


# ------------------------------------------------------------- truncation
def test_support_hand_worked_examples():
    # x = [1, 3, 2, 2, 0, -1, 0.5, 2.5]: ranking 1, 7, 2, 3, 0, 6, 4, 5 (2 before 3: tie -> lowest index)
    e = math.exp
    # top-k 3: softmax over {3, 2.5, 2}
    idx, pr, _ = oracle.support(make_sample(X8, [wl.TOP_K], top_k=[3]), 0)
    z3 = 1 + e(-0.5) + e(-1.0)
    assert idx.tolist() == [1, 7, 2]
    assert np.allclose(pr, [1 / z3, e(-0.5) / z3, e(-1.0) / z3], rtol=1e-14)
    # top-p 0.9 over the full vocabulary: cumulative fractions .3805 .6114 .7514 .8913 .9428 -> five tokens
    idx, pr, _ = oracle.support(make_sample(X8, [wl.TOP_P], top_p=[0.9]), 0)
    assert idx.tolist() == [1, 7, 2, 3, 0]
    z5 = 1 + e(-0.5) + 2 * e(-1.0) + e(-2.0)
    assert np.allclose(pr, np.array([1, e(-0.5), e(-1), e(-1), e(-2)]) / z5, rtol=1e-14)
    # min-p 0.3: threshold 3 + ln 0.3 = 1.796 -> {3, 2.5, 2, 2}
    idx, pr, _ = oracle.support(make_sample(X8, [wl.MIN_P], min_p=[0.3]), 0)
    assert idx.tolist() == [1, 7, 2, 3]
    # k=5, p=0.9, theta=0.3: top-p is taken over the top-5 renormalised mass (.4036 .6484 .7969 .9454) -> 4
    idx, pr, _ = oracle.support(make_sample(X8, [wl.TOP_K | wl.TOP_P | wl.MIN_P], top_k=[5], top_p=[0.9],
                                            min_p=[0.3]), 0)
    assert idx.tolist() == [1, 7, 2, 3]
    z4 = 1 + e(-0.5) + 2 * e(-1.0)
    assert np.allclose(pr, np.array([1, e(-0.5), e(-1), e(-1)]) / z4, rtol=1e-14)


def test_top_p_invariants_random_rows():
    rng = np.random.default_rng(21)
    for trial in range(40):
        V = int(rng.integers(2, 300))
        x = (rng.standard_normal((1, V)) * rng.uniform(0.3, 4)).astype(np.float32)
        p = float(np.float32(rng.uniform(0.05, 0.999)))
        idx, pr, margin = oracle.support(make_sample(x, [wl.TOP_P], top_p=[p]), 0)
        full = softmax(x[0].astype(np.float64))
        kept = full[idx]
        order = np.argsort(-x[0], kind="stable")
        assert idx.tolist() == order[: len(idx)].tolist()          # a prefix of the ranking
        assert kept.sum() >= p * (1 - 1e-12)                        # retained mass >= p
        assert kept.sum() - kept[-1] < p * (1 + 1e-12)              # minimal
        assert np.allclose(pr, kept / kept.sum(), rtol=1e-12)
    # p -> 0+ keeps exactly the most likely token
    idx, _, _ = oracle.support(make_sample(X8, [wl.TOP_P], top_p=[1e-30]), 0)
    assert idx.tolist() == [1]
    # p = 1 keeps everything finite
    idx, _, _ = oracle.support(make_sample(X8, [wl.TOP_P], top_p=[1.0]), 0)
    assert sorted(idx.tolist()) == list(range(8))


def test_min_p_equals_probability_form():
    rng = np.random.default_rng(22)
    for trial in range(40):
        V = int(rng.integers(2, 200))
        x = (rng.standard_normal((1, V)) * 2).astype(np.float32)
        th = float(np.float32(rng.uniform(0.01, 0.9)))
        idx, pr, margin = oracle.support(make_sample(x, [wl.MIN_P], min_p=[th]), 0)
        full = softmax(x[0].astype(np.float64))
        if margin < 1e-9:
            continue
        expect = np.nonzero(full >= th * full.max())[0]
        assert sorted(idx.tolist()) == expect.tolist()


def test_top_k_then_top_p_uses_renormalised_mass():
    # two equal leaders and a long tail: over the full vocabulary top-p 0.6 needs three tokens,
    # over the top-2 survivors it needs two.
    x = np.array([[2.0, 2.0] + [0.0] * 30], dtype=np.float32)
    idx, _, _ = oracle.support(make_sample(x, [wl.TOP_P], top_p=[0.6]), 0)
    full = softmax(x[0].astype(np.float64))
    assert len(idx) == int(np.searchsorted(np.cumsum(np.sort(full)[::-1]), 0.6)) + 1
    idx, _, _ = oracle.support(make_sample(x, [wl.TOP_K | wl.TOP_P], top_k=[2], top_p=[0.6]), 0)
    assert idx.tolist() == [0, 1]


def test_masked_and_penalised_support():
    # hand-worked: processed = [1.4286, 2.1429, 0.5, 2.8571, 0, -2.8571, 3.9286, 3.5714], ids 0 and 5 masked
    mode = (wl.GRAMMAR | wl.REPETITION | wl.FREQUENCY | wl.PRESENCE | wl.BIAS | wl.TEMPERATURE
            | wl.TOP_K | wl.TOP_P | wl.MIN_P)
    allowed = np.array([[0, 1, 1, 1, 1, 0, 1, 1]], dtype=bool)
    w = make_sample(X8, [mode], rep=[1.25], freq=[0.5], pres=[0.25], temperature=[0.7], top_k=[4],
                    top_p=[0.95], min_p=[0.05], hist=[{2: 2, 5: 1}], bias=[{1: -1.5, 6: 2.25}],
                    bitmask=pack_bits(allowed))
    idx, pr, _ = oracle.support(w, 0)
    assert idx.tolist() == [6, 7, 3, 1]
    y = np.array([3.9285715, 3.5714285, 2.8571429, 2.1428571])
    ww = np.exp(y - y[0])
    assert np.allclose(pr, ww / ww.sum(), rtol=1e-6)
    g = make_sample(X8, [wl.GRAMMAR | wl.GREEDY], bitmask=pack_bits(allowed))
    assert oracle.sample(g)["token"].tolist() == [1]                # unmasked argmax
    g = make_sample(X8, [wl.GRAMMAR | wl.GREEDY], bitmask=pack_bits(~allowed))
    assert oracle.sample(g)["token"].tolist() == [0]                # only ids 0 and 5 allowed


# ------------------------------------------------------------------- draws
def test_draw_closed_form_two_tokens():
    # V = 2: token 0 iff u < p0 (index-order inverse CDF: first i with F_i > u*W)
    N = 4000
    x = np.tile(np.array([[math.log(0.3), math.log(0.7)]], dtype=np.float32), (N, 1))
    w = make_sample(x, np.full(N, 0), offset=np.arange(N))
    out = oracle.sample(w)
    p0 = softmax(x[0].astype(np.float64))[0]
    for b in range(N):
        _, ud = py_uniforms(0, b, b)
        if abs(ud - p0) < 1e-9:
            continue
        assert out["token"][b] == (0 if ud < p0 else 1)
        assert abs(out["prob"][b] - (p0 if out["token"][b] == 0 else 1 - p0)) < 1e-6


def test_greedy_is_argmax_lowest_index():
    x = np.array([[1.0, 5.0, 5.0, -2.0], [0.0, 0.0, 0.0, 0.0]], dtype=np.float32)
    out = oracle.sample(make_sample(x, [wl.GREEDY, wl.GREEDY]))
    assert out["token"].tolist() == [1, 0] and out["prob"].tolist() == [1.0, 1.0]


def test_draw_chi_squared_against_truncated_distribution():
    N = 200000
    rng = np.random.default_rng(31)
    x1 = (rng.standard_normal(24) * 1.5).astype(np.float32)
    x = np.tile(x1[None, :], (N, 1))
    w = make_sample(x, np.full(N, wl.TEMPERATURE | wl.TOP_K | wl.TOP_P), temperature=np.full(N, 0.8),
                    top_k=np.full(N, 12), top_p=np.full(N, 0.9), seed=np.full(N, 1234), offset=np.arange(N))
    out = oracle.sample(w)
    # expected distribution from the definitions, written independently in fp64
    y = x1.astype(np.float64) / np.float64(np.float32(0.8))
    order = np.argsort(-y, kind="stable")[:12]
    pk = softmax(y[order])
    n = int(np.searchsorted(np.cumsum(pk), 0.9 * (1 - 1e-15))) + 1
    keep = order[:n]
    expect = np.zeros(24)
    expect[keep] = softmax(y[keep])
    counts = np.bincount(out["token"], minlength=24)
    assert counts[expect == 0].sum() == 0
    chi2 = ((counts[keep] - N * expect[keep]) ** 2 / (N * expect[keep])).sum()
    assert chi2 < stats.chi2.ppf(0.999, len(keep) - 1)


def test_no_token_and_bad_parameters():
    x = np.full((3, 16), -np.inf, dtype=np.float32)
    x[1, 3] = 0.5
    out = oracle.sample(make_sample(x, [0, 0, wl.TEMPERATURE], temperature=[1.0, 1.0, 0.0]))
    assert out["token"].tolist() == [-1, 3, -1]
    assert out["flags"].tolist() == [1, 0, 2]


def test_top_p_one_keeps_every_survivor():
    # Appendix "Probability Truncation": the nucleus of mass >= p * Z.  At p = 1 only the whole set reaches the whole
    # mass; in floating point the running sum of a peaked row stops growing long before the last token (here after
    # the first: 1 + e^-50 == 1 in fp64), so the literal comparison would keep one token.  p = 1 means no truncation.
    x = np.array([[0.0, -50.0, -60.0, -np.inf, -55.0, -70.0]], dtype=np.float32).repeat(3, 0)
    w = make_sample(x, [wl.TOP_P, wl.TOP_P | wl.TOP_K, wl.TOP_P | wl.MIN_P], top_p=[1.0, 1.0, 1.0], top_k=[0, 3, 0],
                    min_p=[0.0, 0.0, 1e-25])
    out = oracle.sample(w)
    assert out["support"].tolist() == [5, 3, 3]          # every finite token; the 3 best; those above ln(1e-25) = -57.6
    assert out["token"].tolist() == [0, 0, 0] and np.all(out["margin"] > 1e-3)
    # just below 1 the nucleus is decided by the masses again
    out = oracle.sample(make_sample(x[:1], [wl.TOP_P], top_p=[np.float32(1.0 - 2.0 ** -20)]))
    assert out["support"].tolist() == [1]


def test_penalty_coefficients_outside_their_domain_are_bad_parameters():
    # Appendix "Repetition Penalties" states alpha >= 1, beta >= 0, gamma >= 0; a coefficient that would make a logit NaN
    # or infinite (divisor not positive and finite, coefficient not finite) is reported like any bad parameter,
    # for greedy rows as well; a clear mode bit hides the value
    x = np.linspace(-1.0, 1.0, 12, dtype=np.float32)[None, :].repeat(7, 0)
    R, F, Pn = wl.REPETITION, wl.FREQUENCY, wl.PRESENCE
    out = oracle.sample(make_sample(x, [R | wl.GREEDY, R, F | wl.GREEDY, Pn, wl.GREEDY, R | F | Pn | wl.GREEDY, R | wl.GREEDY],
                                    rep=[0.0, np.nan, 1.0, 1.0, np.nan, 0.5, np.inf], freq=[0, 0, np.inf, 0, np.inf, -1.0, 0],
                                    pres=[0, 0, 0, np.nan, np.nan, -1.0, 0], hist=[{11: 1}] * 7))
    assert out["flags"].tolist() == [2, 2, 2, 2, 0, 0, 2]
    assert out["token"].tolist()[:4] == [-1, -1, -1, -1] and out["token"][4] == 11 and out["token"][6] == -1
    # row 5: alpha = 0.5 is inside (0, inf): x[11] = 1.0 / 0.5 + 1 + 1 = 4
    assert out["token"][5] == 11


# ----------------------------------------------------------- verification
def _verify_workload(p_rows, q_rows, drafts, mode, seed, **kw):
    """p_rows [B, K+1, V] target probabilities, q_rows [B, K, V] draft probabilities."""
    p_rows = np.asarray(p_rows, dtype=np.float64)
    B, K1, V = p_rows.shape
    with np.errstate(divide="ignore"):
        logits = np.log(p_rows).astype(np.float32).reshape(B * K1, V)
    sw = make_sample(np.zeros((B, V), np.float32), mode, seed=np.full(B, seed), **kw)
    sw.logits = logits
    return wl.VerifyWorkload(name="t", B=B, K=K1 - 1, V=V, sample=sw,
                             draft_tokens=np.asarray(drafts, np.int32).reshape(B, K1 - 1),
                             draft_probs=np.asarray(q_rows, np.float32).reshape(B, K1 - 1, V))


def test_verify_hand_worked_accept_rule():
    # p = (.5,.3,.2), q = (.2,.5,.3): d=0 always accepted; d=1 iff u <= 0.6; d=2 iff u <= 2/3;
    # residual = (1,0,0), so every rejection emits token 0.
    p = [0.5, 0.3, 0.2]
    q = [0.2, 0.5, 0.3]
    B = 3000
    drafts = np.arange(B) % 3
    vw = _verify_workload(np.tile(np.array(p), (B, 2, 1)), np.tile(np.array(q), (B, 1, 1)), drafts,
                          np.zeros(B), seed=5)
    out = oracle.verify(vw)
    pf = softmax(np.log(np.array(p)).astype(np.float32).astype(np.float64))
    qf = np.array(q, np.float32).astype(np.float64)
    for b in range(B):
        d = int(drafts[b])
        ua, _ = py_uniforms(5, 0, b)
        lhs, rhs = ua * qf[d], pf[d]
        if abs(lhs - rhs) < 1e-7:
            continue
        if lhs <= rhs:
            assert out["accept_len"][b] == 1 and out["tokens"][b, 0] == d and out["tokens"][b, 1] >= 0
        else:
            assert out["accept_len"][b] == 0 and out["tokens"][b].tolist() == [0, -1]
        assert abs(out["p_draft"][b, 0] - pf[d]) < 1e-6


def test_verify_preserves_target_distribution_chi_squared():
    # drafts truly sampled from q; the first emitted token must be distributed as p (Leviathan et al.)
    rng = np.random.default_rng(41)
    V, B = 12, 200000
    p = softmax(rng.standard_normal(V) * 1.2)
    q = softmax(rng.standard_normal(V) * 1.2)
    drafts = rng.choice(V, size=B, p=q)
    vw = _verify_workload(np.tile(p, (B, 2, 1)), np.tile(q, (B, 1, 1)), drafts, np.zeros(B), seed=99)
    out = oracle.verify(vw)
    pf = softmax(np.log(p).astype(np.float32).astype(np.float64))
    counts = np.bincount(out["tokens"][:, 0], minlength=V)
    chi2 = ((counts - B * pf) ** 2 / (B * pf)).sum()
    assert chi2 < stats.chi2.ppf(0.999, V - 1)
    # exact enumeration identity behind it: sum_d q(d) [a(d) 1{x=d} + (1-a(d)) r(x)] = p(x)
    a = np.minimum(1.0, p / q)
    r = np.maximum(0.0, p - q)
    r /= r.sum()
    assert np.allclose(q * a + (q * (1 - a)).sum() * r, p, atol=1e-12)
    # the acceptance rate is sum_x min(p, q)
    assert abs(out["accept_len"].mean() - np.minimum(pf, q).sum()) < 4 * math.sqrt(0.25 / B)


def test_verify_greedy_prefix_and_bonus():
    V, K = 9, 3
    rng = np.random.default_rng(42)
    logits = rng.standard_normal((4, K + 1, V)).astype(np.float32)
    am = logits.argmax(axis=2)
    drafts = am[:, :K].copy()
    drafts[1, 1] = (drafts[1, 1] + 1) % V        # mismatch at position 1
    drafts[2, 0] = (drafts[2, 0] + 1) % V        # mismatch at position 0
    drafts[3, 2] = (drafts[3, 2] + 1) % V        # mismatch at position 2
    sw = make_sample(np.zeros((4, V), np.float32), [wl.GREEDY] * 4)
    sw.logits = logits.reshape(-1, V)
    vw = wl.VerifyWorkload(name="g", B=4, K=K, V=V, sample=sw, draft_tokens=drafts.astype(np.int32),
                           draft_probs=np.full((4, K, V), 1.0 / V, np.float32))
    out = oracle.verify(vw)
    assert out["accept_len"].tolist() == [3, 1, 0, 2]
    assert out["tokens"][0].tolist() == am[0].tolist()                       # all accepted + bonus
    assert out["tokens"][1].tolist() == [am[1, 0], am[1, 1], -1, -1]
    assert out["tokens"][2].tolist() == [am[2, 0], -1, -1, -1]
    assert out["tokens"][3].tolist() == [am[3, 0], am[3, 1], am[3, 2], -1]


def test_verify_with_no_drafts_equals_singular_mode():
    rng = np.random.default_rng(43)
    B, V = 64, 50
    x = (rng.standard_normal((B, V)) * 2).astype(np.float32)
    mode = np.full(B, wl.TEMPERATURE | wl.TOP_P)
    kw = dict(temperature=np.full(B, 0.9), top_p=np.full(B, 0.8), seed=np.full(B, 77), offset=np.arange(B) * 3)
    s = oracle.sample(make_sample(x, mode, **kw))
    sw = make_sample(x, mode, **kw)
    vw = wl.VerifyWorkload(name="k0", B=B, K=0, V=V, sample=sw, draft_tokens=np.zeros((B, 0), np.int32),
                           draft_probs=np.zeros((B, 0, V), np.float32))
    v = oracle.verify(vw)
    assert v["tokens"][:, 0].tolist() == s["token"].tolist() and v["accept_len"].tolist() == [0] * B


def test_verify_zero_probability_draft_is_rejected():
    # a draft outside the target's support (top-k 1 keeps only token 2) is never accepted, and the
    # resampled token comes from the support
    p = np.tile(np.array([0.2, 0.3, 0.5]), (50, 2, 1))
    q = np.tile(np.array([0.9, 0.05, 0.05]), (50, 1, 1))
    vw = _verify_workload(p, q, np.zeros(50), np.full(50, wl.TOP_K), seed=3, top_k=np.full(50, 1))
    out = oracle.verify(vw)
    assert out["accept_len"].tolist() == [0] * 50 and out["tokens"][:, 0].tolist() == [2] * 50
    assert np.all(out["p_draft"] == 0)


# ------------------------------------------ positions, bonus draw, margins, end-to-end tokens
def _index_order_pick(ids, probs, u):
    """Closed form of the draw over a hand-worked support: ids ascending with their probabilities;
    the first id whose cumulative probability exceeds u (probabilities sum to 1)."""
    F = 0.0
    for i, p in zip(ids, probs):
        F += p
        if F > u:
            return i
    return ids[-1]


def test_verify_positions_use_offset_plus_l_and_bonus_uses_the_draw_word():
    # K = 2, V = 3, the same p and q at every position.  p = (.5,.3,.2), q = (.2,.5,.3), hand-worked:
    # draft 0 always accepted, draft 1 iff u_acc <= .6, draft 2 iff u_acc <= 2/3; the residual is (1,0,0), so a
    # rejection emits token 0; the bonus token (both accepted) is the index-order draw from p with the DRAW word of
    # position 2: token 0 if u_draw < .5, 1 if < .8, else 2.  Position l of request b uses the Philox counter
    # offset + l (word 0 accept, word 1 draw): predicted here from the second Philox implementation.
    p = np.array([0.5, 0.3, 0.2])
    q = np.array([0.2, 0.5, 0.3])
    pf = softmax(np.log(p).astype(np.float32).astype(np.float64))
    qf = q.astype(np.float32).astype(np.float64)
    B, K, seed = 4000, 2, 21
    rng = np.random.default_rng(8)
    drafts = rng.integers(0, 3, size=(B, K))
    offset = rng.integers(0, 2 ** 40, size=B).astype(np.uint64)
    vw = _verify_workload(np.tile(p, (B, K + 1, 1)), np.tile(q, (B, K, 1)), drafts, np.zeros(B), seed=seed, offset=offset)
    out = oracle.verify(vw)
    n_bonus = n_second = 0
    for b in range(B):
        expect, acc, near = [], 0, False
        for l in range(K + 1):
            ua, ud = py_uniforms(seed, int(offset[b]) + l, b)
            if l < K:
                d = int(drafts[b, l])
                lhs = ua * qf[d]
                near |= abs(lhs - pf[d]) < 1e-7
                if lhs <= pf[d]:
                    expect.append(d); acc += 1
                    continue
                expect.append(0)                                   # residual (1, 0, 0)
                break
            near |= min(abs(ud - pf[0]), abs(ud - pf[0] - pf[1])) < 1e-7
            expect.append(_index_order_pick([0, 1, 2], pf, ud))   # bonus token from position K
        if near:
            continue
        expect += [-1] * (K + 1 - len(expect))
        assert out["tokens"][b].tolist() == expect, (b, out["tokens"][b], expect)
        assert out["accept_len"][b] == acc
        n_bonus += acc == K
        n_second += acc >= 1
    assert n_bonus > 300 and n_second > 1500                      # positions 1 and 2 were really exercised
    # using the position-0 counter for every position, or the accept word for the bonus draw, gives other tokens
    b = next(b for b in range(B) if out["accept_len"][b] == K
             and _index_order_pick([0, 1, 2], pf, py_uniforms(seed, int(offset[b]) + K, b)[0]) != out["tokens"][b, K])
    assert out["tokens"][b, K] == _index_order_pick([0, 1, 2], pf, py_uniforms(seed, int(offset[b]) + K, b)[1])


def test_end_to_end_tokens_of_the_hand_worked_rows():
    # Row A: x8 with top-k 5, top-p 0.9, min-p 0.3 -> support {1, 7, 2, 3}, probabilities
    # (.426933, .258948, .157060, .157060); index-order CDF over ids 1, 2, 3, 7 = (.426933, .583992, .741052, 1).
    # Row B: mask + penalties + bias + tau 0.7, k 4, p .95, theta .05 -> support {6, 7, 3, 1}; index-order CDF over
    # ids 1, 3, 6, 7 = (.075877, .230872, .683387, 1).  (seed, offset, row) = (0, 0, 0) draws
    # u = ((0xe169c58d >> 8) + .5) / 2^24 = 0.88052019 from the second Philox word: token 7 in both rows.
    u = ((0xE169C58D >> 8) + 0.5) / 2 ** 24
    assert py_uniforms(0, 0, 0)[1] == u
    wa = make_sample(X8, [wl.TOP_K | wl.TOP_P | wl.MIN_P], top_k=[5], top_p=[0.9], min_p=[0.3])
    out = oracle.sample(wa)
    assert out["token"].tolist() == [7] and out["support"].tolist() == [4]
    assert abs(out["prob"][0] - 0.258948) < 1e-6
    mode = (wl.GRAMMAR | wl.REPETITION | wl.FREQUENCY | wl.PRESENCE | wl.BIAS | wl.TEMPERATURE
            | wl.TOP_K | wl.TOP_P | wl.MIN_P)
    allowed = np.array([[0, 1, 1, 1, 1, 0, 1, 1]], dtype=bool)
    wb = make_sample(X8, [mode], rep=[1.25], freq=[0.5], pres=[0.25], temperature=[0.7], top_k=[4],
                     top_p=[0.95], min_p=[0.05], hist=[{2: 2, 5: 1}], bias=[{1: -1.5, 6: 2.25}],
                     bitmask=pack_bits(allowed))
    out = oracle.sample(wb)
    assert out["token"].tolist() == [7] and out["support"].tolist() == [4]
    assert abs(out["prob"][0] - 0.316613) < 1e-6
    # other offsets walk the same hand-worked CDFs
    cdf_a = ([1, 2, 3, 7], [0.426933, 0.157060, 0.157060, 0.258948])
    cdf_b = ([1, 3, 6, 7], [0.075877, 0.154995, 0.452516, 0.316613])
    for off in range(1, 60):
        u = py_uniforms(0, off, 0)[1]
        for w, (ids, pr) in ((wa, cdf_a), (wb, cdf_b)):
            edges = np.cumsum(pr)
            if np.min(np.abs(edges - u)) < 1e-5:
                continue
            w.offset[:] = off
            assert oracle.sample(w)["token"][0] == _index_order_pick(ids, pr, u)


def test_margins_of_the_hand_worked_rows():
    # top-p 0.9 on x8: the cumulative fractions around the cut are .891346 (4 tokens) and .942847 (5 tokens), so the
    # cut's margin is min(|.942847 - .9|, |.891346 - .9|) = .008654; the row's margin is the smaller of that and
    # the draw's distance to the nearer edge of its CDF step (index-order CDF over ids 0, 1, 2, 3, 7 =
    # .054623, .458235, .606716, .755197, 1).
    z = 1 + math.exp(-0.5) + 2 * math.exp(-1) + math.exp(-2) + math.exp(-2.5) + math.exp(-3) + math.exp(-4)
    c4 = (1 + math.exp(-0.5) + 2 * math.exp(-1)) / z
    c5 = c4 + math.exp(-2) / z
    p32 = float(np.float32(0.9))
    cut_margin = min(abs(c5 - p32), abs(c4 - p32))
    assert abs(cut_margin - 0.008654) < 2e-6
    edges = np.cumsum(np.array([math.exp(-2), 1, math.exp(-1), math.exp(-1), math.exp(-0.5)]) / (c5 * z))
    w = make_sample(X8, [wl.TOP_P], top_p=[0.9])
    seen_draw = seen_cut = 0
    for off in range(200):
        w.offset[:] = off
        u = py_uniforms(0, off, 0)[1]
        j = int(np.searchsorted(edges, u, side="right"))
        lo = edges[j - 1] if j > 0 else 0.0
        draw_margin = min(abs(edges[min(j, 4)] - u), abs(lo - u))
        got = oracle.sample(w)["margin"][0]
        assert abs(got - min(cut_margin, draw_margin)) < 1e-9, (off, got, cut_margin, draw_margin)
        seen_draw += draw_margin < cut_margin
        seen_cut += draw_margin >= cut_margin
    assert seen_draw > 0 and seen_cut > 0
    # min-p 0.3 on x8: threshold 3 + ln(0.3) = 1.796027; the entries next to the cut are 2.0 and 1.0
    w = make_sample(X8, [wl.MIN_P], min_p=[0.3])
    _, _, m = oracle.support(w, 0)
    thr = 3 + math.log(float(np.float32(0.3)))
    assert abs(m - min(2.0 - thr, thr - 1.0)) < 1e-12
    # verification: the accept test's margin |u q - p| / max(u q, p), draft 1 of p = (.5,.3,.2), q = (.2,.5,.3)
    p, q = np.array([0.5, 0.3, 0.2]), np.array([0.2, 0.5, 0.3])
    pf = softmax(np.log(p).astype(np.float32).astype(np.float64))
    qf = q.astype(np.float32).astype(np.float64)
    B = 64
    vw = _verify_workload(np.tile(p, (B, 2, 1)), np.tile(q, (B, 1, 1)), np.ones(B), np.zeros(B), seed=9)
    out = oracle.verify(vw)
    for b in range(B):
        ua, ud = py_uniforms(9, 0, b)
        lhs = ua * qf[1]
        acc_margin = abs(lhs - pf[1]) / max(lhs, pf[1])
        if lhs <= pf[1]:
            # accepted: the bonus token's draw margin joins in (CDF .5, .8, 1 with position 1's draw word)
            ud1 = py_uniforms(9, 1, b)[1]
            e = np.array([0.0, pf[0], pf[0] + pf[1], 1.0])
            j = int(np.searchsorted(e, ud1, side="right"))
            expect = min(acc_margin, abs(e[min(j, 3)] - ud1), abs(e[j - 1] - ud1))
        else:
            expect = min(acc_margin, min(abs(1.0 - ud), abs(0.0 - ud)))      # residual (1, 0, 0): one step from 0 to 1
        assert abs(out["margin"][b] - expect) < 1e-7, (b, out["margin"][b], expect)
