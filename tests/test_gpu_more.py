"""More CUDA-vs-oracle parity: the launch configuration the benchmark times (CUDA graphs over rotating
input copies that share one workspace), the largest vocabulary, rows the streaming path hands to the
exact kernel, mixed verification with grammar masks and penalties, replay determinism."""
import numpy as np
import pytest

from paper_2607_20475_b200 import workloads as wl
from tests.helpers import make_sample, pack_bits
from tests.parity import compare_sample, compare_verify, compare_topk

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


def header_error_word(dev):
    import torch
    torch.cuda.synchronize()
    return int(dev.ws[:4].view(torch.int32).cpu().numpy()[0])


def test_bench_launch_configuration_full_size(sonic, oracle):
    # exactly what bench.py times: one graph of back-to-back calls over distinct full-size c2 copies on a shared
    # workspace, replayed; every copy's outputs must match the oracle afterwards
    import torch
    import bench
    devs = bench.build_device_copies("c2", 3, sonic)
    g = bench.capture(devs, 3)
    for _ in range(5):
        g.replay()
    torch.cuda.synchronize()
    for c, dev in enumerate(devs):
        got = dev.results()
        ref = oracle.sample(dev.w)
        compare_sample(got, ref, dev.w, max_near=6)
    assert header_error_word(devs[0]) == 0


def test_replays_are_bit_identical(sonic):
    import torch
    w = wl.config2(B=32, V=50000)
    dev = sonic.DeviceSample(w)
    dev.run()
    first = dev.results()
    for _ in range(30):
        dev.run()
    again = dev.results()
    for key in first:
        assert np.array_equal(first[key], again[key]), key
    assert header_error_word(dev) == 0


def test_largest_vocabulary_all_paths(sonic, oracle):
    V = 262144
    rng = np.random.default_rng(77)
    x = (rng.standard_normal((8, V)) * 1.5).astype(np.float32)
    x[0, rng.choice(V, 3, replace=False)] += 9
    mode = [wl.GREEDY, wl.TOP_K | wl.TEMPERATURE, wl.TOP_P | wl.TEMPERATURE, wl.MIN_P, wl.TEMPERATURE,
            wl.TOP_K | wl.TOP_P, wl.TOP_K | wl.TEMPERATURE | wl.MIN_P, wl.TOP_K]
    w = make_sample(x, mode, temperature=[1, .6, .5, 1, 1.2, 1, .9, 1], top_k=[0, 40, 0, 0, 0, 6000, 2048, 300],
                    top_p=[1, 1, .9, 1, 1, .8, 1, 1], min_p=[0, 0, 0, .02, 0, 0, .001, 0],
                    seed=np.arange(8) + 100, offset=np.arange(8) * 7)
    dev = sonic.DeviceSample(w)
    dev.run()
    got = dev.results()
    ref = oracle.sample(w)
    compare_sample(got, ref, w)
    # rows 2..4 (top-k off) take the histogram passes, row 5 (k beyond the streaming path) the cluster kernel
    assert all(got["flags"][r] & 8 for r in (2, 3, 4)) and got["flags"][5] & 4
    assert not (got["flags"][[2, 3, 4]] & 4).any()
    assert header_error_word(dev) == 0


def test_topk_bf16_full_width_and_k_limits(sonic, oracle):
    tw = wl.config5("normal", B=16, V=262144, dtype=wl.DTYPE_BF16)      # bf16: thousands of ties per row
    x = tw.logits_f32()
    rv, ri = oracle.topk(x, 4096)
    for k in (1, 100, 2048, 4096):
        dev = sonic.DeviceTopK(tw, k)
        dev.run()
        gv, gi = dev.results()
        compare_topk(gv, gi, rv[:, :k].copy(), ri[:, :k].copy())


def test_verify_with_mask_penalties_and_bf16(sonic, oracle):
    B, K, V = 6, 3, 40000
    rng = np.random.default_rng(78)
    base = wl.config2(B=B * (K + 1), V=V, dtype=wl.DTYPE_BF16)            # bf16 target rows, mixed regimes
    s = wl.config2(B=B, V=V, dtype=wl.DTYPE_BF16)                           # per-request parameters, lists
    s.logits = base.logits
    allowed = rng.random((B * (K + 1), V)) < 0.3
    s.bitmask = pack_bits(allowed)
    s.mode = (s.mode | wl.GRAMMAR).astype(np.uint32)
    tgt = base.logits_f32().reshape(B, K + 1, V)
    q = np.zeros((B, K, V), np.float32)
    drafts = np.zeros((B, K), np.int32)
    for b in range(B):
        for l in range(K):
            z = tgt[b, l].astype(np.float64) + rng.standard_normal(V) * 0.3
            z[~allowed[b * (K + 1) + l]] = -np.inf
            e = np.exp(z - z.max())
            q[b, l] = (e / e.sum()).astype(np.float32)
            drafts[b, l] = int(np.argmax(q[b, l])) if (s.mode[b] & wl.GREEDY) else int(rng.choice(V, p=e / e.sum()))
    vw = wl.VerifyWorkload(name="vm", B=B, K=K, V=V, sample=s, draft_tokens=drafts, draft_probs=q)
    dev = sonic.DeviceVerify(vw)
    dev.run()
    got = dev.results()
    ref = oracle.verify(vw)
    compare_verify(got, ref, vw)


def test_many_list_entries_in_one_tile(sonic, oracle):
    # all history and bias ids inside one 8192-element tile, more than a thread's prefetched share
    V = 30000
    rng = np.random.default_rng(79)
    x = rng.standard_normal((3, V)).astype(np.float32)
    ids = rng.choice(8192, 2000, replace=False) + 8192
    hist = [{int(i): int(c) for i, c in zip(ids, rng.integers(1, 4, 2000))}] * 3
    bias = [{int(i): float(v) for i, v in zip(ids[:900], rng.uniform(-3, 3, 900))}] * 3
    mode = wl.REPETITION | wl.FREQUENCY | wl.PRESENCE | wl.BIAS
    w = make_sample(x, [mode | wl.GREEDY, mode | wl.TOP_K | wl.TEMPERATURE, mode | wl.TOP_P], rep=[1.2] * 3,
                    freq=[0.1] * 3, pres=[0.2] * 3, temperature=[1, 0.8, 1], top_k=[0, 25, 0], top_p=[1, 1, 0.7],
                    hist=hist, bias=bias, seed=[9, 9, 9])
    dev = sonic.DeviceSample(w)
    dev.run()
    got = dev.results()
    ref = oracle.sample(w)
    compare_sample(got, ref, w)


@pytest.mark.parametrize("dtype", [wl.DTYPE_F32, wl.DTYPE_BF16])
@pytest.mark.parametrize("n_hist,n_bias", [(300, 50), (383, 64), (500, 20), (200, 100)])
def test_short_lists_per_tile_hit_lists(sonic, oracle, dtype, n_hist, n_bias):
    # lists short enough to be filtered per tile: below, at and above what one tile's hit lists hold (all ids in
    # one tile, which crowds it), ids present in both lists (penalty first, then bias), a ragged last tile
    V = 3 * 8192 + 17
    rng = np.random.default_rng(1000 + n_hist + n_bias)
    x = (rng.standard_normal((4, V)) * 2).astype(np.float32)
    ids = rng.choice(8192, max(n_hist, n_bias), replace=False) + 8192
    far = [0, 5, 8191, 2 * 8192, V - 1]                      # a few entries in the other tiles
    hist = [{**{int(i): int(c) for i, c in zip(ids[:n_hist], rng.integers(1, 5, n_hist))}, **{i: 2 for i in far}}] * 4
    bias = [{**{int(i): float(v) for i, v in zip(ids[:n_bias], rng.uniform(-4, 4, n_bias))}, **{i: 1.5 for i in far[:3]}}] * 4
    mode = wl.REPETITION | wl.FREQUENCY | wl.PRESENCE | wl.BIAS
    w = make_sample(x, [mode | wl.GREEDY, mode | wl.TOP_K | wl.TEMPERATURE, mode | wl.TOP_P, mode | wl.TOP_K | wl.TOP_P | wl.MIN_P],
                    dtype=dtype, rep=[1.3] * 4, freq=[0.15] * 4, pres=[0.25] * 4, temperature=[1, 0.7, 1, 1],
                    top_k=[0, 40, 0, 300], top_p=[1, 1, 0.8, 0.9], min_p=[1, 1, 1, 0.01], hist=hist, bias=bias,
                    seed=[3, 4, 5, 6])
    dev = sonic.DeviceSample(w)
    dev.run()
    got = dev.results()
    assert header_error_word(dev) == 0
    ref = oracle.sample(w)
    compare_sample(got, ref, w)


def test_many_short_rows_through_the_work_queue(sonic, oracle):
    # far more rows than resident CTAs, one ragged tile each: every CTA takes a run and then single tiles from the
    # queue; afterwards the queue counter in the workspace header is back at zero
    B, V = 1500, 777
    rng = np.random.default_rng(4242)
    x = (rng.standard_normal((B, V)) * 3).astype(np.float32)
    kinds = np.arange(B) % 3
    mode = np.where(kinds == 0, wl.GREEDY, np.where(kinds == 1, wl.TOP_K | wl.TEMPERATURE, wl.TOP_K | wl.TOP_P)).astype(np.uint32)
    w = make_sample(x, mode, temperature=np.where(kinds == 1, 0.7, 1.0), top_k=np.where(kinds == 0, 0, 12),
                    top_p=np.where(kinds == 2, 0.9, 1.0), seed=np.arange(B) + 5)
    dev = sonic.DeviceSample(w)
    for _ in range(2):
        dev.run()
    got = dev.results()
    assert header_error_word(dev) == 0
    import torch
    assert int(dev.ws[8:12].view(torch.int32).cpu().numpy()[0]) == 0      # header word 2: the work counter
    ref = oracle.sample(w)
    compare_sample(got, ref, w)


def test_two_host_threads_share_the_device(sonic, oracle):
    # two threads, each with its own stream and workspace, call into the library at the same time (each thread gets
    # an internal stream of its own for the histogram passes)
    import threading
    import torch
    ws = [wl.config1(), wl.config1()]
    ws[1] = make_sample(np.asarray(ws[1].logits)[::-1].copy(), ws[1].mode[::-1].copy(), temperature=ws[1].temperature[::-1].copy(),
                        top_k=ws[1].top_k[::-1].copy(), top_p=ws[1].top_p[::-1].copy(), min_p=ws[1].min_p[::-1].copy(),
                        seed=ws[1].seed[::-1].copy(), offset=ws[1].offset[::-1].copy())
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    devs = []
    for w, st in zip(ws, streams):
        with torch.cuda.stream(st):
            devs.append(sonic.DeviceSample(w))
    torch.cuda.synchronize()
    errors = []

    def work(i):
        try:
            with torch.cuda.stream(streams[i]):
                for _ in range(50):
                    devs[i].run()
            streams[i].synchronize()
        except Exception as exc:      # pragma: no cover - reported below
            errors.append(exc)

    threads = [threading.Thread(target=work, args=(i,)) for i in range(2)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors
    torch.cuda.synchronize()
    for w, dev in zip(ws, devs):
        assert header_error_word(dev) == 0
        compare_sample(dev.results(), oracle.sample(w), w)


@pytest.mark.parametrize("dtype", [wl.DTYPE_F32, wl.DTYPE_BF16])
def test_threshold_search_with_heavy_ties(sonic, oracle, dtype):
    # coarse-grained logits (a few dozen distinct values, so equal values differ only in their index) with k from
    # just above the small-sort limit to the largest the streaming path takes: the merge kernel has to cut the
    # candidate list inside a run of equal values
    V = 100000
    rng = np.random.default_rng(90210)
    ks = [513, 600, 777, 1000, 1023, 1025, 1500, 2047, 2048, 2049, 3000, 4095, 4096]
    x = (np.round(rng.standard_normal((len(ks), V)) * 4) / 4).astype(np.float32)
    x[1::2] = np.round(rng.standard_normal((len(ks[1::2]), V)) * 64).astype(np.float32) / 64
    w = make_sample(x, [wl.TOP_K | wl.TEMPERATURE] * len(ks), dtype=dtype, temperature=[0.9] * len(ks), top_k=ks,
                    seed=np.arange(len(ks)) + 31, offset=np.arange(len(ks)))
    dev = sonic.DeviceSample(w)
    dev.run()
    got = dev.results()
    assert header_error_word(dev) == 0
    compare_sample(got, oracle.sample(w), w)
    tw = wl.TopKWorkload(name="ties", B=len(ks), V=V, dtype=dtype, logits=w.logits)
    rv, ri = oracle.topk(tw.logits_f32(), 4096)
    for k in (513, 1000, 2049, 4096):
        dk = sonic.DeviceTopK(tw, k)
        dk.run()
        gv, gi = dk.results()
        compare_topk(gv, gi, rv[:, :k].copy(), ri[:, :k].copy())


def test_exact_row_counters_return_to_zero(sonic, oracle):
    # more exact-class rows than clusters (top-k off on every stochastic request, K + 1 positions each): the rows are
    # handed out from a counter in the workspace header, which the last cluster puts back to zero; replays must
    # therefore give the same answers and leave header words 3 and 6 at zero
    import torch
    vw = wl.config4(B=12, K=3, V=20000)
    vw.sample.top_k[:] = 0
    vw.sample.mode[:] = (vw.sample.mode & ~np.uint32(wl.TOP_K)).astype(np.uint32)
    dev = sonic.DeviceVerify(vw)
    dev.run()
    first = dev.results()
    for _ in range(3):
        dev.run()
    again = dev.results()
    for key in first:
        assert np.array_equal(first[key], again[key]), key
    hdr = dev.ws[:32].view(torch.int32).cpu().numpy()
    assert hdr[0] == 0 and hdr[3] == 0 and hdr[6] == 0
    compare_verify(again, oracle.verify(vw), vw)


def test_thousands_of_exact_rows_share_the_row_counter(sonic, oracle):
    # far more exact-class rows than clusters, short rows with a ragged slice per CTA: every cluster draws rows from
    # the counter until it runs dry; rows of the streaming classes are interleaved
    B, V = 3000, 300
    rng = np.random.default_rng(5150)
    x = (rng.standard_normal((B, V)) * 2).astype(np.float32)
    kinds = np.arange(B) % 4
    mode = np.select([kinds == 0, kinds == 1, kinds == 2], [wl.TOP_P | wl.TEMPERATURE, wl.MIN_P, wl.GREEDY],
                     wl.TOP_K | wl.TOP_P).astype(np.uint32)
    w = make_sample(x, mode, temperature=np.where(kinds == 0, 0.8, 1.0), top_k=np.where(kinds == 3, 7, 0),
                    top_p=np.where(kinds % 3 == 0, 0.85, 1.0), min_p=np.where(kinds == 1, 0.03, 0.0),
                    seed=np.arange(B) + 17, offset=np.arange(B) * 3)
    dev = sonic.DeviceSample(w)
    for _ in range(2):
        dev.run()
    got = dev.results()
    import torch
    hdr = dev.ws[:32].view(torch.int32).cpu().numpy()
    assert not hdr[[0, 2, 3, 4, 5, 6, 7]].any(), hdr       # error word and every work counter back at zero
    compare_sample(got, oracle.sample(w), w)
    assert all(got["flags"][r] & 8 for r in range(B) if kinds[r] in (0, 1))


@pytest.mark.parametrize("V", [262144, 200003, 128256, 100001])
def test_tile_cutoffs_ragged_rows_sparse_masks_and_empty_tiles(sonic, oracle, V):
    # small and medium k take their tile cutoff as the smallest group maximum of the whole tile; groups with no
    # finite element (past a ragged row's end, masked out, a whole tile masked) must not drag it down: every row
    # has to agree with the oracle, and the dense rows and small k be finished by the streaming path (no exact-kernel flag)
    rng = np.random.default_rng(V)
    ks = [8, 20, 50, 64, 200, 256, 600, 1000]
    B = 2 * len(ks)
    x = rng.standard_normal((B, V)).astype(np.float32)
    allowed = np.ones((B, V), dtype=bool)
    for r in range(len(ks), B):
        allowed[r] = rng.random(V) < 0.05                 # sparse: many groups of 128 hold no allowed id
        allowed[r, 3 * 8192:5 * 8192] = False             # two whole tiles masked
        allowed[r, 8192 + 1024:8192 + 4096] = False       # three warp tiles of one tile masked
    mode = [wl.TOP_K | wl.TEMPERATURE] * len(ks) + [wl.TOP_K | wl.TEMPERATURE | wl.GRAMMAR] * len(ks)
    w = make_sample(x, mode, temperature=rng.uniform(0.6, 1.4, B), top_k=ks + ks, bitmask=pack_bits(allowed),
                    seed=np.arange(B) + 5, offset=np.arange(B))
    dev = sonic.DeviceSample(w)
    dev.run()
    got = dev.results()
    compare_sample(got, oracle.sample(w), w)
    # (the sparse rows with a large k may legitimately miss their proof: few finite elements per group)
    must_stream = [r for r in range(B) if r < len(ks) or w.top_k[r] <= 64]
    assert not (got["flags"][must_stream] & 4).any(), np.nonzero(got["flags"] & 4)[0]
    assert header_error_word(dev) == 0
    tw = wl.TopKWorkload(name="ragged", B=B, V=V, dtype=wl.DTYPE_F32, logits=np.where(allowed, x, -np.inf).astype(np.float32))
    rv, ri = oracle.topk(tw.logits_f32(), 1024)
    for k in (8, 64, 256, 1024):
        d = sonic.DeviceTopK(tw, k)
        d.run()
        gv, gi = d.results()
        compare_topk(gv, gi, rv[:, :k].copy(), ri[:, :k].copy())
