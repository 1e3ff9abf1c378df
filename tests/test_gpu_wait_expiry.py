"""A bounded wait of the streaming kernel that really runs out, in the form that neither faults nor hangs a GPU: a
test-only build of the library (wait limit 4096 rounds; a header word under which the producer announces one tile's bytes
but never issues its copy) runs in a child process; the kernel returns by itself, the call reports SONIC_FLAG_TIMEOUT on
every row, the error is sticky until sonic_workspace_init, and afterwards the results equal the oracle's."""
import json
import os
import subprocess
import sys

import numpy as np
import pytest

from oracle import oracle
from paper_2607_20475_b200 import build as lib_build, workloads as wl
from tests.helpers import make_sample

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
FLAG_TIMEOUT = 0x10


@pytest.mark.gpu
def test_a_wait_that_runs_out_is_reported_and_the_workspace_recovers():
    if not os.path.exists(lib_build.WAITTEST_LIB):
        lib_build.build_waittest()
    run = subprocess.run([sys.executable, os.path.join(ROOT, "tests", "wait_expiry", "child.py")],
                         capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert run.returncode == 0, run.stdout[-2000:] + run.stderr[-2000:]
    line = [ln for ln in run.stdout.splitlines() if ln.startswith("RESULT ")][-1]
    r = json.loads(line[len("RESULT "):])
    B = len(r["good_tokens"])
    # the same inputs as the child builds, through the oracle
    V = 40000
    rng = np.random.default_rng(77)
    x = rng.standard_normal((B, V)).astype(np.float32) * 2
    mode = [wl.GREEDY, wl.TOP_K | wl.TEMPERATURE, wl.TOP_P, wl.MIN_P | wl.TEMPERATURE, wl.TOP_K | wl.TOP_P, wl.TEMPERATURE]
    w = make_sample(x, mode, temperature=[1, .8, 1, 1.2, 1, .9], top_k=[0, 40, 0, 0, 300, 0], top_p=[1, 1, .9, 1, .8, 1],
                    min_p=[0, 0, 0, .05, 0, 0], seed=np.arange(B) + 5)
    ref = oracle.sample(w)
    sure = ref["margin"] >= 1e-6
    assert sure.sum() >= B - 1
    # before: a normal call
    assert r["error_word_before"] == 0
    assert np.array_equal(np.asarray(r["good_tokens"])[sure], ref["token"][sure])
    assert all((f & FLAG_TIMEOUT) == 0 for f in r["good_flags"])
    # the call whose tile copy never came: it returned, and every row says so
    assert r["error_word_after"] & 1
    assert all(f & FLAG_TIMEOUT for f in r["expired_flags"]) and all(t == -1 for t in r["expired_tokens"])
    # sticky: the next call on the same workspace reports it too
    assert all(f & FLAG_TIMEOUT for f in r["sticky_flags"]) and all(t == -1 for t in r["sticky_tokens"])
    # after sonic_workspace_init the workspace serves correct calls again
    assert r["error_word_recovered"] == 0
    assert all((f & FLAG_TIMEOUT) == 0 for f in r["recovered_flags"])
    assert np.array_equal(np.asarray(r["recovered_tokens"])[sure], ref["token"][sure])
    assert np.allclose(np.asarray(r["recovered_prob"])[sure], ref["prob"][sure], rtol=1e-5, atol=1e-7)
