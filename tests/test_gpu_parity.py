"""CUDA path vs CPU oracle, element by element, through the C ABI (needs a B200)."""
import numpy as np
import pytest

from paper_2607_20475_b200 import workloads as wl
from tests.helpers import make_sample, pack_bits
from tests.parity import compare_sample, compare_topk, compare_verify

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def sonic():
    from paper_2607_20475_b200 import harness as binding
    binding.lib()
    return binding


@pytest.fixture(scope="module")
def oracle():
    from oracle import oracle as o
    return o


def run_sample(sonic, oracle, w, twice=True, max_near=None):
    dev = sonic.DeviceSample(w)
    dev.run()
    got = dev.results()
    ref = oracle.sample(w)
    n = compare_sample(got, ref, w, max_near)
    if twice:                                   # the workspace is restored by the kernels: a replay must agree
        dev.run()
        got2 = dev.results()
        for key in got:
            assert np.array_equal(got[key], got2[key]), key
    return got, ref, n


# ------------------------------------------------------------------ top-k
@pytest.mark.parametrize("regime", ["spike", "zipf", "normal", "zeros", "const129", "twovalued", "ascending",
                                    "descending", "signedzeros"])
@pytest.mark.parametrize("dtype", [wl.DTYPE_F32, wl.DTYPE_BF16])
def test_topk_small(sonic, oracle, regime, dtype):
    # several CTA tiles and a ragged tail (V is not a multiple of the tile, nor of the vector width for fp32)
    for B, V in ((3, 20001), (2, 70000)):
        tw = wl.config5(regime, B=B, V=V, dtype=dtype)
        x = tw.logits_f32()
        for k in (1, 8, 64, 1000, 4096):
            dev = sonic.DeviceTopK(tw, k)
            dev.run()
            gv, gi = dev.results()
            rv, ri = oracle.topk(x, k)
            compare_topk(gv, gi, rv, ri)


def test_topk_tiny_vocabularies(sonic, oracle):
    rng = np.random.default_rng(5)
    for V in (1, 2, 3, 31, 33, 1000, 4096, 8192, 8193):
        x = rng.integers(-4, 5, size=(4, V)).astype(np.float32)
        x[1, :] = -np.inf
        if V > 2:
            x[2, V // 2] = -np.inf
        tw = wl.TopKWorkload(name="t", B=4, V=V, dtype=wl.DTYPE_F32, logits=x)
        for k in sorted({1, min(V, 5), min(V, 4096)}):
            dev = sonic.DeviceTopK(tw, k)
            dev.run()
            gv, gi = dev.results()
            rv, ri = oracle.topk(x, k)
            compare_topk(gv, gi, rv, ri)


@pytest.mark.parametrize("regime", wl.TOPK_REGIMES)
def test_topk_config5_full(sonic, oracle, regime):
    tw = wl.config5(regime)
    x = tw.logits_f32()
    rv, ri = oracle.topk(x, 4096)
    ws = sonic.new_workspace(tw.B, tw.V)
    for k in wl.TOPK_KS:
        dev = sonic.DeviceTopK(tw, k, ws=ws)
        dev.run()
        gv, gi = dev.results()
        compare_topk(gv, gi, rv[:, :k].copy(), ri[:, :k].copy())


# --------------------------------------------------------------- singular mode
def test_config1_full(sonic, oracle):
    w = wl.config1()
    got, ref, n = run_sample(sonic, oracle, w)
    assert got["token"][0] == int(np.argmax(w.logits[0]))


@pytest.mark.parametrize("dtype", [wl.DTYPE_BF16, wl.DTYPE_F32])
@pytest.mark.parametrize("V", [9000, 40000])
def test_config2_reduced(sonic, oracle, dtype, V):
    w = wl.config2(B=24, V=V, dtype=dtype)
    run_sample(sonic, oracle, w)


def test_config2_full(sonic, oracle):
    w = wl.config2()
    got, ref, n = run_sample(sonic, oracle, w, max_near=4)
    print("config2 near-margin rows:", n, "fallback rows:", int(((got["flags"] & 4) != 0).sum()))


def test_config3_reduced(sonic, oracle):
    w = wl.config3(B=16, V=50000)
    run_sample(sonic, oracle, w)


def test_config3_full(sonic, oracle):
    w = wl.config3()
    got, ref, n = run_sample(sonic, oracle, w, max_near=4)
    # masked-argmax rows: the raw argmax of odd rows is not allowed and must not be chosen
    raw_am = np.argmax(w.logits, axis=1)
    odd = np.arange(w.B) % 2 == 1
    assert np.all(got["token"][odd] != raw_am[odd])


def test_edge_rows(sonic, oracle):
    V = 20000
    rng = np.random.default_rng(9)
    x = rng.standard_normal((10, V)).astype(np.float32)
    x[0, :] = -np.inf                                   # no finite logit
    x[1, :] = 0.0                                       # all ties
    x[2, :] = -np.inf; x[2, 12345] = 1.0                # single allowed token
    x[3, 7] = x[3].max() + 1; x[3, 19999] = x[3, 7]     # tie for the maximum: lowest index wins
    x[9, :] = np.where(rng.random(V) < 0.5, 0.0, -0.0)  # signed zeros
    mode = [wl.TOP_K, wl.TOP_K | wl.TEMPERATURE, wl.TOP_P, wl.GREEDY, wl.TEMPERATURE, wl.TOP_K | wl.TOP_P | wl.MIN_P,
            wl.MIN_P | wl.TEMPERATURE, wl.TOP_K, wl.TOP_K | wl.TEMPERATURE, wl.GREEDY]
    w = make_sample(x, mode, temperature=[1, .7, 1, 1, 0.0, 1, 1.3, 1, 2.0, 1], top_k=[5, 3, 0, 0, 0, 40000, 0, -1, 1, 0],
                    top_p=[1, 1, .5, 1, 1, .9, 1, 1, 1, 1], min_p=[0, 0, 0, 0, 0, .01, .2, 0, 0, 0],
                    seed=np.arange(10) + 3, offset=np.arange(10) * 1000003)
    got, ref, n = run_sample(sonic, oracle, w)
    assert got["flags"][0] & 1 and got["flags"][4] & 2 and got["flags"][7] & 2
    assert got["token"][3] == 7 and got["token"][9] == 0 and got["token"][2] == 12345


def test_top_p_one_keeps_every_survivor(sonic, oracle):
    # p = 1 with the bit set is "no truncation" on peaked rows whose tail no longer moves a floating-point sum:
    # with top-k off (histogram path), with top-k (merge), with min-p, in a verification-free sampling call
    V = 30000
    rng = np.random.default_rng(13)
    x = (rng.standard_normal((6, V)) * 3).astype(np.float32)
    x[:, 17] += 60.0                                      # one token holds all but 1e-20 of the mass
    mode = [wl.TOP_P, wl.TOP_P | wl.TEMPERATURE, wl.TOP_P | wl.TOP_K, wl.TOP_P | wl.MIN_P, wl.TOP_P | wl.TOP_K | wl.TEMPERATURE,
            wl.TOP_P]
    w = make_sample(x, mode, temperature=[1, 0.3, 1, 1, 0.5, 1], top_p=[1, 1, 1, 1, 1, np.float32(1 - 2.0 ** -16)],
                    top_k=[0, 0, 700, 0, 50, 0], min_p=[0, 0, 0, 1e-30, 0, 0], seed=np.arange(6) + 70)
    got, ref, n = run_sample(sonic, oracle, w)
    assert n == 0
    assert ref["support"].tolist()[:3] == [V, V, 700] and ref["support"][4] == 50 and ref["support"][5] == 1
    assert got["support"].tolist() == ref["support"].tolist()
    assert np.all(got["token"] == 17)


def test_penalty_coefficients_outside_their_domain(sonic, oracle):
    # Appendix "Repetition Penalties": alpha >= 1, beta >= 0, gamma >= 0.  A divisor that is not positive and finite, or a
    # coefficient that is not finite, is a bad parameter (greedy rows too); a clear bit hides any value
    V = 9000
    rng = np.random.default_rng(12)
    x = rng.standard_normal((9, V)).astype(np.float32) * 2
    inf, nan = np.inf, np.nan
    R, F, Pn = wl.REPETITION, wl.FREQUENCY, wl.PRESENCE
    mode = [R | wl.TOP_K, R | wl.GREEDY, R | wl.TOP_P, F | wl.TOP_K, Pn | wl.MIN_P, F | wl.GREEDY, wl.TOP_K, R | F | Pn | wl.TOP_K, R | wl.TOP_K]
    w = make_sample(x, mode, top_k=[5, 0, 0, 7, 0, 0, 5, 9, 5], top_p=[1, 1, .8, 1, 1, 1, 1, 1, 1], min_p=[0, 0, 0, 0, .1, 0, 0, 0, 0],
                    rep=[0.0, -2.0, nan, 1.0, 1.0, 1.0, nan, 0.5, inf], freq=[0, 0, 0, inf, 0, nan, inf, -0.25, 0],
                    pres=[0, 0, 0, 0, -inf, 0, nan, -0.5, 0],
                    hist=[{3: 1, 77: 2}] * 9, seed=np.arange(9) + 40)
    got, ref, n = run_sample(sonic, oracle, w)
    bad = (got["flags"] & 2) != 0
    assert list(bad) == [True, True, True, True, True, True, False, False, True]
    assert np.all(got["token"][bad] == -1)


def test_temperature_ties_in_topk(sonic, oracle):
    # distinct logits that collide after the temperature division: the boundary group of the top-k
    # must be broken by index exactly as the definition does
    V = 30000
    rng = np.random.default_rng(10)
    base = rng.integers(0, 2000, size=(6, V)).astype(np.float32)
    x = (np.float32(1.0) + base * np.float32(2.0 ** -23)).astype(np.float32)   # consecutive fp32 values
    w = make_sample(x, [wl.TOP_K | wl.TEMPERATURE] * 3 + [wl.GREEDY | wl.TEMPERATURE] * 3,
                    temperature=[3.0, 1.7, 0.9, 3.0, 1.7, 0.9], top_k=[7, 50, 300, 0, 0, 0], seed=np.arange(6))
    run_sample(sonic, oracle, w)


def test_mode_bits_gate_parameters(sonic, oracle):
    # parameters whose bit is clear must be ignored; NULL arrays are fine when no row sets the bit
    V = 12000
    rng = np.random.default_rng(11)
    x = rng.standard_normal((4, V)).astype(np.float32) * 3
    w = make_sample(x, [0, wl.GREEDY, wl.TOP_K, wl.TOP_P], temperature=[0.1] * 4, top_k=[3, 3, 3, 3],
                    top_p=[0.1, 0.1, 0.1, 0.1], min_p=[0.9] * 4, rep=[3.0] * 4, hist=[{1: 2}] * 4, bias=[{2: 9.0}] * 4,
                    seed=[5, 6, 7, 8])
    run_sample(sonic, oracle, w)
    w2 = make_sample(x, [wl.GREEDY, wl.GREEDY, wl.TOP_K, wl.TOP_K], top_k=[3, 3, 3, 3])
    w2.temperature = w2.top_p = w2.min_p = w2.rep_penalty = w2.freq_penalty = w2.pres_penalty = None
    got, ref, _ = run_sample(sonic, oracle, make_sample(x, [wl.GREEDY, wl.GREEDY, wl.TOP_K, wl.TOP_K], top_k=[3] * 4))
    dev = sonic.DeviceSample(w2)
    dev.run()
    got2 = dev.results()
    assert np.array_equal(got["token"], got2["token"])


def test_bad_list_id_and_long_lists(sonic, oracle):
    V = 33000
    rng = np.random.default_rng(12)
    x = rng.standard_normal((3, V)).astype(np.float32)
    hist = [{int(i): int(c) for i, c in zip(rng.choice(V, 3000, replace=False), rng.integers(0, 5, 3000))},
            {int(V + 5): 1, 4: 2}, {3: 1}]
    bias = [{int(i): float(v) for i, v in zip(rng.choice(V, 700, replace=False), rng.uniform(-8, 8, 700))},
            {1: 1.0}, {-1: 2.0}]
    mode = wl.REPETITION | wl.FREQUENCY | wl.PRESENCE | wl.BIAS | wl.TOP_K | wl.TEMPERATURE
    w = make_sample(x, [mode, mode, mode | wl.GREEDY], rep=[1.3] * 3, freq=[0.1] * 3, pres=[0.4] * 3,
                    temperature=[0.8] * 3, top_k=[40] * 3, hist=hist, bias=bias)
    got, ref, _ = run_sample(sonic, oracle, w)
    assert got["flags"][1] & 2 and got["flags"][2] & 2 and got["token"][0] >= 0


def test_sample_distribution_chi_squared_on_gpu(sonic, oracle):
    # many draws of one truncated distribution: the CUDA path's own RNG stream and CDF inversion
    from scipy import stats
    from scipy.special import softmax
    N, V = 20000, 9000
    rng = np.random.default_rng(13)
    x1 = (rng.standard_normal(V) * 2).astype(np.float32)
    x = np.tile(x1[None], (N, 1))
    w = make_sample(x, np.full(N, wl.TOP_K | wl.TEMPERATURE), temperature=np.full(N, 0.9), top_k=np.full(N, 16),
                    seed=np.full(N, 2024), offset=np.arange(N))
    dev = sonic.DeviceSample(w)
    dev.run()
    got = dev.results()
    y = x1.astype(np.float64) / np.float64(np.float32(0.9))
    keep = np.argsort(-y, kind="stable")[:16]
    pr = softmax(y[keep])
    counts = np.array([(got["token"] == i).sum() for i in keep])
    assert counts.sum() == N
    chi2 = ((counts - N * pr) ** 2 / (N * pr)).sum()
    assert chi2 < stats.chi2.ppf(0.999, 15)


# --------------------------------------------------------------- multistep mode
def run_verify(sonic, oracle, vw, max_near=None):
    dev = sonic.DeviceVerify(vw)
    dev.run()
    got = dev.results()
    ref = oracle.verify(vw)
    n = compare_verify(got, ref, vw, max_near)
    dev.run()
    got2 = dev.results()
    for key in got:
        assert np.array_equal(got[key], got2[key]), key
    return got, ref, n


def test_config4_reduced(sonic, oracle):
    vw = wl.config4(B=8, K=3, V=30000)
    run_verify(sonic, oracle, vw)


def test_config4_full(sonic, oracle):
    vw = wl.config4()
    got, ref, n = run_verify(sonic, oracle, vw, max_near=8)   # dense top-p rows: a token carries ~1e-6 of the mass
    print("config4 accept lengths:", got["accept_len"].tolist(), "near-margin:", n)


def test_verify_no_drafts_equals_sample(sonic, oracle):
    w = wl.config2(B=12, V=20000, dtype=wl.DTYPE_F32)
    vw = wl.VerifyWorkload(name="k0", B=w.B, K=0, V=w.V, sample=w, draft_tokens=np.zeros((w.B, 0), np.int32),
                           draft_probs=np.zeros((w.B, 0, w.V), np.float32))
    got, ref, _ = run_verify(sonic, oracle, vw)
    dev = sonic.DeviceSample(w)
    dev.run()
    s = dev.results()
    assert np.array_equal(s["token"], got["tokens"][:, 0])


def test_verify_greedy_and_rejections(sonic, oracle):
    # greedy requests with a mismatch at every possible position; stochastic requests whose drafts are
    # outside the target support (always rejected) or identical to the target (always accepted)
    V, K, B = 17000, 3, 8
    rng = np.random.default_rng(14)
    tgt = rng.standard_normal((B, K + 1, V)).astype(np.float32) * 2
    am = tgt.argmax(axis=2)
    drafts = am[:, :K].copy().astype(np.int32)
    for b in range(4):
        if b < K:
            drafts[b, b] = (drafts[b, b] + 1) % V
    mode = [wl.GREEDY] * 4 + [wl.TOP_K] * 2 + [wl.TOP_K | wl.TEMPERATURE] * 2
    sw = make_sample(np.zeros((B, V), np.float32), mode, top_k=[0, 0, 0, 0, 1, 1, 30, 30],
                     temperature=[1, 1, 1, 1, 1, 1, 0.8, 0.8], seed=np.arange(B) + 40)
    sw.logits = tgt.reshape(-1, V)
    q = np.full((B, K, V), 1.0 / V, np.float32)
    drafts[5, 1] = (am[5, 1] + 7) % V                    # outside the top-1 support: rejected at position 1
    vw = wl.VerifyWorkload(name="g", B=B, K=K, V=V, sample=sw, draft_tokens=drafts, draft_probs=q)
    got, ref, _ = run_verify(sonic, oracle, vw)
    assert got["accept_len"][:6].tolist() == [0, 1, 2, 3, 3, 1]
