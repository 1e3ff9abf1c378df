"""Seeded differential sweep: random shapes, mode bits, parameters, masks and sparse lists, the CUDA path against the
oracle.  Small enough for the oracle to finish each case in well under a second; the seeds are fixed, so a failure
names a reproducible case."""
import numpy as np
import pytest

from paper_2607_20475_b200 import workloads as wl
from tests.helpers import make_sample, pack_bits
from tests.parity import compare_sample, compare_verify

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


def random_rows(rng, B, V):
    """Logit rows of mixed character: smooth, spiked, quantised (many ties), mostly -inf."""
    x = np.empty((B, V), np.float32)
    for r in range(B):
        kind = int(rng.integers(0, 5))
        if kind == 0:
            row = rng.standard_normal(V) * rng.uniform(0.3, 4.0)
        elif kind == 1:
            row = rng.standard_normal(V)
            row[rng.choice(V, size=min(V, int(rng.integers(1, 6))), replace=False)] += rng.uniform(5, 15)
        elif kind == 2:
            row = np.round(rng.standard_normal(V) * 2) / 2            # ties everywhere
        elif kind == 3:
            row = -np.log(np.arange(1, V + 1)) * rng.uniform(0.5, 2.0)
            rng.shuffle(row)
        else:
            row = rng.standard_normal(V)
            row[rng.random(V) < 0.9] = -np.inf
        x[r] = row.astype(np.float32)
    return x


def random_case(seed, dtype):
    rng = np.random.default_rng(seed)
    V = int(rng.choice([1, 7, 33, 1000, 4097, 8192, 8193, 20011, 32768, 40000]))
    B = int(rng.integers(1, 7))
    x = random_rows(rng, B, V)
    mode = np.zeros(B, np.uint32)
    kw = dict(temperature=np.ones(B, np.float32), top_k=np.zeros(B, np.int32), top_p=np.ones(B, np.float32),
              min_p=np.zeros(B, np.float32), rep=np.ones(B, np.float32), freq=np.zeros(B, np.float32),
              pres=np.zeros(B, np.float32), seed=rng.integers(0, 2**62, B).astype(np.uint64),
              offset=rng.integers(0, 2**40, B).astype(np.uint64))
    for r in range(B):
        if rng.random() < 0.25:
            mode[r] |= wl.GREEDY
        if rng.random() < 0.6:
            mode[r] |= wl.TEMPERATURE
            kw["temperature"][r] = np.float32(rng.uniform(0.3, 2.0))
        if rng.random() < 0.6:
            mode[r] |= wl.TOP_K
            kw["top_k"][r] = int(rng.choice([1, 2, 5, 40, 300, 1000, 2048, 3000, V, V + 5]))
        if rng.random() < 0.5:
            mode[r] |= wl.TOP_P
            kw["top_p"][r] = np.float32(rng.choice([0.1, 0.5, 0.9, 0.99, 1.0]))
        if rng.random() < 0.3:
            mode[r] |= wl.MIN_P
            kw["min_p"][r] = np.float32(rng.choice([0.001, 0.05, 0.5, 1.0]))
        if rng.random() < 0.4:
            mode[r] |= wl.REPETITION
            kw["rep"][r] = np.float32(rng.uniform(1.0, 1.5))
        if rng.random() < 0.4:
            mode[r] |= wl.FREQUENCY
            kw["freq"][r] = np.float32(rng.uniform(0.0, 0.5))
        if rng.random() < 0.4:
            mode[r] |= wl.PRESENCE
            kw["pres"][r] = np.float32(rng.uniform(0.0, 0.5))
    hist = bias = bitmask = None
    if rng.random() < 0.7:
        n = int(rng.choice([1, 10, 200, 600, 1500]))
        hist = []
        for r in range(B):
            ids = rng.choice(V, size=min(V, n), replace=False)
            hist.append({int(i): int(c) for i, c in zip(ids, rng.integers(0, 5, len(ids)))})   # count 0: a no-op entry
    else:
        mode &= ~np.uint32(wl.REPETITION | wl.FREQUENCY | wl.PRESENCE)
    if rng.random() < 0.5:
        n = int(rng.choice([1, 8, 40]))
        bias = []
        for r in range(B):
            ids = rng.choice(V, size=min(V, n), replace=False)
            bias.append({int(i): float(v) for i, v in zip(ids, rng.uniform(-5, 5, len(ids)))})
        mode |= np.uint32(wl.BIAS)
    if rng.random() < 0.5:
        allowed = rng.random((B, V)) < rng.choice([0.02, 0.5, 0.98])
        if rng.random() < 0.3:
            allowed[0, :] = False                                                              # nothing allowed: NO_TOKEN
        bitmask = pack_bits(allowed)
        mode |= np.uint32(wl.GRAMMAR)
    return make_sample(x, mode, dtype=dtype, hist=hist, bias=bias, bitmask=bitmask, **kw)


@pytest.mark.parametrize("seed", range(40))
def test_random_sample_case(sonic, oracle, seed):
    dtype = wl.DTYPE_BF16 if seed % 3 == 2 else wl.DTYPE_F32
    w = random_case(77000 + seed, dtype)
    dev = sonic.DeviceSample(w)
    dev.run()
    got = dev.results()
    import torch
    assert int(dev.ws[:4].view(torch.int32).cpu().numpy()[0]) == 0
    ref = oracle.sample(w)
    compare_sample(got, ref, w)


def random_verify_case(seed):
    """A multistep case: the sample part from random_case (fp32), replicated positions, random draft distributions."""
    rng = np.random.default_rng(seed)
    base = random_case(seed, wl.DTYPE_F32)
    B, V = base.B, base.V
    K = int(rng.integers(0, 5))
    tgt = random_rows(rng, B * (K + 1), V)
    import dataclasses
    kw = {}
    if base.bitmask is not None:                      # one mask row per logit row
        kw["bitmask"] = np.repeat(base.bitmask, K + 1, axis=0)
    sw = dataclasses.replace(base, logits=tgt, **kw)
    draft_probs = np.zeros((B, max(K, 1), V), np.float32)
    draft_tokens = np.zeros((B, max(K, 1)), np.int32)
    for b in range(B):
        for l in range(K):
            z = tgt[b * (K + 1) + l].astype(np.float64) + rng.standard_normal(V) * 0.7
            z[~np.isfinite(z)] = -50.0
            q = np.exp(z - z.max())
            if rng.random() < 0.5:                    # a truncated draft distribution
                cut = np.sort(q)[::-1][min(V - 1, int(rng.integers(0, 50)))]
                q[q < cut] = 0.0
            q /= q.sum()
            draft_probs[b, l] = q.astype(np.float32)
            draft_tokens[b, l] = int(rng.choice(V, p=q))
    return wl.VerifyWorkload(name="fuzz", B=B, K=K, V=V, sample=sw, draft_tokens=draft_tokens[:, :K].copy() if K else draft_tokens[:, :0].copy(),
                             draft_probs=draft_probs[:, :K].copy() if K else draft_probs[:, :0].copy())


@pytest.mark.parametrize("seed", range(24))
def test_random_verify_case(sonic, oracle, seed):
    vw = random_verify_case(88000 + seed)
    dev = sonic.DeviceVerify(vw)
    dev.run()
    got = dev.results()
    ref = oracle.verify(vw)
    compare_verify(got, ref, vw)


@pytest.mark.parametrize("seed", range(16))
def test_random_topk_case(sonic, oracle, seed):
    from tests.parity import compare_topk
    rng = np.random.default_rng(99000 + seed)
    V = int(rng.choice([1, 9, 1000, 8192, 8193, 30000, 65536]))
    B = int(rng.integers(1, 6))
    x = random_rows(rng, B, V)
    k = int(min(V, rng.choice([1, 2, 7, 64, 500, 2048, 4096])))
    dtype = wl.DTYPE_BF16 if seed % 2 else wl.DTYPE_F32
    lg = wl.f32_to_bf16_bits(x) if dtype == wl.DTYPE_BF16 else x
    tw = wl.TopKWorkload(name="fuzz", B=B, V=V, dtype=dtype, logits=lg)
    dev = sonic.DeviceTopK(tw, k)
    dev.run()
    vals, idx = dev.results()
    rv, ri = oracle.topk(tw.logits_f32(), k)
    compare_topk(vals, idx, rv, ri)
