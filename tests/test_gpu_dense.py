"""GPU parity tests of the histogram path (rows with top-k off: top-p, min-p, plain temperature sampling and their
verification variants) at the edges of its own design: a call with one such row (tiles cut into parts), crossing bins
crowded with ties (low-precision logits), top-p against min-p in the same bin, ragged vocabularies, sparse masks,
rejected drafts (residual pass), rows without a token, and replays interleaved between call shapes on one workspace."""
import numpy as np
import pytest

from paper_2607_20475_b200 import workloads as wl
from tests.helpers import make_sample, pack_bits
from tests.parity import compare_sample, compare_verify

pytestmark = pytest.mark.gpu

DENSE = 8


@pytest.fixture(scope="module")
def sonic():
    from paper_2607_20475_b200 import harness
    harness.lib()
    return harness


@pytest.fixture(scope="module")
def oracle():
    from oracle import oracle as o
    return o


def run(sonic, oracle, w, max_near=None, twice=True):
    dev = sonic.DeviceSample(w)
    dev.run()
    got = dev.results()
    ref = oracle.sample(w)
    n = compare_sample(got, ref, w, max_near)
    if twice:
        dev.run()
        again = dev.results()
        for key in got:
            assert np.array_equal(got[key], again[key]), key
    return got, ref, n


@pytest.mark.parametrize("V,dtype", [(131072, wl.DTYPE_BF16), (262144, wl.DTYPE_F32), (32768, wl.DTYPE_F32), (8192, wl.DTYPE_F32),
                                     (700, wl.DTYPE_BF16), (100001, wl.DTYPE_F32)])
def test_single_row_calls_of_every_kind(sonic, oracle, V, dtype):
    # one row per call: the passes cut their tiles into parts; top-p, min-p, both, neither
    rng = np.random.default_rng(V)
    x = rng.standard_normal((1, V)).astype(np.float32) * 1.3
    for mode, kw in ((wl.TOP_P | wl.TEMPERATURE, dict(top_p=[0.9], temperature=[0.9])),
                     (wl.MIN_P, dict(min_p=[0.02])),
                     (wl.TOP_P | wl.MIN_P | wl.TEMPERATURE, dict(top_p=[0.97], min_p=[0.001], temperature=[1.3])),
                     (wl.TEMPERATURE, dict(temperature=[0.8])),
                     (wl.TOP_P, dict(top_p=[1.0]))):
        w = make_sample(x, [mode], dtype=dtype, seed=[V + mode], offset=[3], **kw)
        got, ref, _ = run(sonic, oracle, w, max_near=1)
        assert got["flags"][0] & DENSE


def test_crossing_bins_crowded_with_ties(sonic, oracle):
    # low-precision logits: a few values in the crossing bin, hundreds or thousands of ties each (a Zipf tail in bf16
    # repeats a value about 5000 times); all-equal and two-valued rows: the cut falls among ties, by lowest index
    V = 131072
    rng = np.random.default_rng(9)
    rank = rng.permutation(V) + 1
    zipf = (-1.1 * np.log(rank)).astype(np.float32)
    flat = (rng.standard_normal(V) * 0.5).astype(np.float32)
    two = np.where(rng.random(V) < 0.3, 1.0, 0.0).astype(np.float32)
    const = np.full(V, 129.0, np.float32)
    x = np.stack([zipf, zipf, flat, flat, two, two, const, const, zipf, flat])
    B = x.shape[0]
    mode = np.full(B, wl.TOP_P | wl.TEMPERATURE, np.uint32)
    mode[8:] |= wl.MIN_P
    w = make_sample(x, mode, dtype=wl.DTYPE_BF16, temperature=[1.0, 1.4, 0.8, 1.2, 1.0, 0.7, 1.0, 1.0, 1.1, 1.0],
                    top_p=[0.9, 0.95, 0.9, 0.5, 0.5, 0.99, 0.25, 0.999, 0.98, 0.9], min_p=np.full(B, 0.01),
                    seed=np.arange(B) + 40, offset=np.arange(B) * 5)
    # (equal weights put the cumulative mass exactly on p * Z now and then - margin zero - so most of these rows are
    #  near-margin by construction; each is still held to one of its two admissible outcomes)
    got, ref, _ = run(sonic, oracle, w, max_near=B)
    assert (got["flags"] & DENSE).all() and not (got["flags"] & 4).any()        # none needed the cluster kernel
    # the same rows in fp32 with a mask that allows 2 % of the ids (supports of a few thousand) and a ragged width
    Vr = 100003
    allowed = rng.random((B, Vr)) < 0.02
    w = make_sample(x[:, :Vr], mode | wl.GRAMMAR, temperature=np.full(B, 1.1), top_p=np.full(B, 0.9), min_p=np.full(B, 0.01),
                    bitmask=pack_bits(allowed), seed=np.arange(B) + 70, offset=np.arange(B))
    run(sonic, oracle, w, max_near=B)


def test_top_p_against_min_p_in_one_row(sonic, oracle):
    # the min-p threshold above, inside and below the bin where top-p cuts
    V = 65536
    rng = np.random.default_rng(12)
    x = np.tile((rng.standard_normal(V) * 2).astype(np.float32), (9, 1))
    thetas = [0.5, 0.2, 0.1, 0.05, 0.02, 0.01, 0.005, 0.001, 1e-6]
    w = make_sample(x, np.full(9, wl.TOP_P | wl.MIN_P), top_p=np.full(9, 0.6), min_p=thetas, seed=np.arange(9), offset=np.arange(9))
    got, ref, _ = run(sonic, oracle, w)
    assert len(set(ref["support"].tolist())) > 3                              # the cases really differ
    # a dense sweep of theta around the top-p cut: for some the threshold key falls in the crossing bin itself
    idx, pr, _ = oracle.support(make_sample(x[:1], [wl.TOP_P], top_p=[0.6]), 0)
    y = x[0].astype(np.float64)
    cut_val = y[idx[-1]]
    th = np.exp((cut_val - y.max()) + np.linspace(-0.004, 0.004, 33))
    w = make_sample(np.tile(x[0], (33, 1)), np.full(33, wl.TOP_P | wl.MIN_P), top_p=np.full(33, 0.6), min_p=th.astype(np.float32),
                    seed=np.arange(33) + 9, offset=np.arange(33))
    run(sonic, oracle, w)


def test_top_p_just_below_and_just_above_a_cumulative_fraction_with_the_mass_in_the_ragged_tile(sonic, oracle):
    # p set a hair below and a hair above the cumulative fraction of the n-th ranked token (relative distance 2e-5, far
    # outside the near-margin band): the support is n, then n + 1.  The heavy tokens sit in the row's ragged last tile
    # (V = 2 tiles + 300), so the cut element, most of the support and the drawn tokens are found there.
    V = 2 * 8192 + 300
    rng = np.random.default_rng(21)
    base = (rng.standard_normal(V) * 1.5).astype(np.float32)
    base[-300:] += np.float32(6.0)
    y = base.astype(np.float64)
    order = np.lexsort((np.arange(V), -y))
    wts = np.exp(y[order] - y.max())
    frac = np.cumsum(wts) / wts.sum()
    rows, ps, want = [], [], []
    for n in (1, 2, 17, 120, 299, 300, 301, 2000):
        f = frac[n - 1]                                        # mass of the n best tokens
        if frac[n] - f < 1e-4 * f:                             # (the next token must clear the band too)
            continue
        for p_, n_ in ((f * (1 - 2e-5), n), (f * (1 + 2e-5), n + 1)):
            rows.append(base); ps.append(np.float32(p_)); want.append(n_)
    B = len(rows)
    assert B >= 10
    w = make_sample(np.stack(rows), np.full(B, wl.TOP_P), top_p=ps, seed=np.arange(B) + 3, offset=np.arange(B) * 7)
    got, ref, near = run(sonic, oracle, w, max_near=0)
    assert near == 0
    assert ref["support"].tolist() == want and got["support"].tolist() == want
    assert np.all((got["flags"] & DENSE) != 0)
    assert np.mean(got["token"] >= 2 * 8192) > 0.5            # drawn from the ragged tile


def test_rows_without_token_and_bad_rows_of_the_class(sonic, oracle):
    V = 20000
    rng = np.random.default_rng(13)
    x = rng.standard_normal((6, V)).astype(np.float32)
    x[1] = -np.inf
    allowed = np.ones((6, V), bool)
    allowed[2] = False                                                        # everything masked
    allowed[3] = False
    allowed[3, 777] = True                                                    # a single allowed token
    mode = np.array([wl.TOP_P, wl.TOP_P, wl.MIN_P | wl.GRAMMAR, wl.TOP_P | wl.GRAMMAR, wl.TOP_P | wl.TEMPERATURE, wl.BIAS | wl.MIN_P], np.uint32)
    w = make_sample(x, mode, top_p=[0.9, 0.9, 1.0, 0.9, 0.0 + 1.5, 1.0], min_p=[0, 0, 0.1, 0, 0, 0.1], temperature=np.ones(6),
                    bitmask=pack_bits(allowed), bias=[{}, {}, {}, {}, {}, {V + 5: 1.0}], seed=np.arange(6), offset=np.arange(6))
    got, ref, _ = run(sonic, oracle, w)
    assert got["token"].tolist()[1:4] == [-1, -1, 777] and got["flags"][4] & 2 and got["flags"][5] & 2


def test_verification_rows_with_rejected_and_foreign_drafts(sonic, oracle):
    # top-k off on every stochastic request: accepted drafts, rejected drafts (residual pass), drafts outside the
    # support, the bonus position; greedy requests beside them
    vw = wl.config4(B=10, K=3, V=50000)
    vw.sample.top_k[:] = 0
    vw.sample.mode[:] = (vw.sample.mode & ~np.uint32(wl.TOP_K)).astype(np.uint32)
    rng = np.random.default_rng(14)
    vw.draft_tokens[0, 0] = int(np.argmin(vw.sample.logits_f32()[0]))            # surely outside a top-p support
    vw.draft_tokens[2, 1] = rng.integers(0, vw.V)
    dev = sonic.DeviceVerify(vw)
    dev.run()
    got = dev.results()
    ref = oracle.verify(vw)
    compare_verify(got, ref, vw, max_near=5)
    assert (ref["accept_len"] < vw.K).any() and (ref["accept_len"] == vw.K).any()
    dev.run()
    again = dev.results()
    for key in got:
        assert np.array_equal(got[key], again[key]), key


def test_replays_interleaved_between_call_shapes_on_one_workspace(sonic, oracle):
    # three calls of different shapes share one workspace sized for the largest; their graphs are replayed in turn a
    # thousand times: every replay leaves the same outputs (only the header of the workspace carries state between calls)
    import torch
    wa = wl.config2(B=24, V=50000)
    wb = wl.config1()
    vw = wl.config4(B=4, K=2, V=30000)
    vw.sample.top_k[:2] = 0
    vw.sample.mode[:2] = (vw.sample.mode[:2] & ~np.uint32(wl.TOP_K)).astype(np.uint32)
    nbytes = max(sonic.sonic_workspace_bytes(24, 50000), sonic.sonic_workspace_bytes(4, 32768), sonic.sonic_workspace_bytes(12, 30000))
    ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    sonic.sonic_workspace_init(ws)
    devs = [sonic.DeviceSample(wa, ws=ws), sonic.DeviceSample(wb, ws=ws), sonic.DeviceVerify(vw, ws=ws)]
    first, graphs = [], []
    for d in devs:
        d.run()
        first.append(d.results())
    compare_sample(first[0], oracle.sample(wa), wa)
    compare_sample(first[1], oracle.sample(wb), wb)
    compare_verify(first[2], oracle.verify(vw), vw, max_near=2)
    for d in devs:
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            d.run()
        graphs.append(g)
    for i in range(1000):
        graphs[i % 3].replay()
        if i % 97 == 0 or i >= 997:
            again = devs[i % 3].results()
            for key in first[i % 3]:
                assert np.array_equal(first[i % 3][key], again[key]), (i, key)
    hdr = ws[:32].view(torch.int32).cpu().numpy()
    assert not hdr[[0, 2, 3, 4, 5, 6, 7]].any(), hdr[:8]        # (word 1 counts the last call's rows for the cluster kernel)
