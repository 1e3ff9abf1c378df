"""bench.py --timeline: the trace variant of the library reports every kernel of a call, in an order that makes sense."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.mark.gpu
def test_timeline_of_a_sampling_and_a_verification_call():
    run = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--timeline", "c1,c4"],
                         capture_output=True, text=True, timeout=900, cwd=ROOT)
    assert run.returncode == 0, run.stdout[-2000:] + run.stderr[-2000:]
    tl = json.loads(run.stdout.strip().splitlines()[-1])["timeline"]
    for name, expect in (("c1", 6), ("c4", 9)):
        k = tl[name]["kernels"]
        assert len(k) == expect, k                               # every kernel of the call reported
        assert all(0.0 <= a <= b < 1000.0 for a, b in k.values()), k
        s, m = k["sonic_stream_kernel"], k["sonic_merge_kernel"]
        assert s[0] == 0.0 and m[1] >= s[1]                      # the merge ends after the streaming kernel
        # the histogram path runs behind the streaming kernel, in order, and the cluster kernel ends the rows' work
        h, c, f, x = (k[n] for n in ("sonic_dense_stage2_kernel", "sonic_dense_collect_kernel", "sonic_dense_finish_kernel",
                                     "sonic_exact_kernel"))
        assert s[1] <= h[1] <= c[1] <= f[1] <= x[1] and m[1] <= x[1]
    assert "sonic_verify_combine_kernel" in tl["c4"]["kernels"]
