"""Child process of tests/test_gpu_wait_expiry.py: runs the test-only build of the library (short wait limit, one
withheld tile copy) in a process of its own and prints what it saw as one JSON line.  No wait here is unbounded, nothing
faults: the withheld copy is simply never issued, the kernel's waits give up after 4096 rounds and the call returns."""
import json
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2607_20475_b200 import build as _build

_build.LIB = _build.WAITTEST_LIB           # before the binding loads the library
from paper_2607_20475_b200 import binding, harness, workloads as wl  # noqa: E402
from tests.helpers import make_sample  # noqa: E402

WS_TEST_WITHHOLD = 100                      # header word of the test-only build


def main():
    assert os.path.exists(_build.WAITTEST_LIB), "test-only library missing (built by __graft_entry__.build())"
    binding.lib()
    V, B = 40000, 6
    rng = np.random.default_rng(77)
    x = rng.standard_normal((B, V)).astype(np.float32) * 2
    mode = [wl.GREEDY, wl.TOP_K | wl.TEMPERATURE, wl.TOP_P, wl.MIN_P | wl.TEMPERATURE, wl.TOP_K | wl.TOP_P, wl.TEMPERATURE]
    w = make_sample(x, mode, temperature=[1, .8, 1, 1.2, 1, .9], top_k=[0, 40, 0, 0, 300, 0], top_p=[1, 1, .9, 1, .8, 1],
                    min_p=[0, 0, 0, .05, 0, 0], seed=np.arange(B) + 5)
    dev = harness.DeviceSample(w)
    hdr = dev.ws[:512].view(torch.int32)
    out = {}
    dev.run()
    good = dev.results()
    out["good_tokens"] = good["token"].tolist()
    out["good_flags"] = good["flags"].tolist()
    out["error_word_before"] = int(hdr[0].item())
    tiles = (V + 8191) // 8192
    hdr[WS_TEST_WITHHOLD] = 2 * tiles + 1 + 1          # row 2, tile 1
    torch.cuda.synchronize()
    dev.run()
    r1 = dev.results()                                  # returns: every wait is bounded
    out["expired_tokens"] = r1["token"].tolist()
    out["expired_flags"] = r1["flags"].tolist()
    out["error_word_after"] = int(hdr[0].item())
    hdr[WS_TEST_WITHHOLD] = 0
    torch.cuda.synchronize()
    dev.run()                                           # same workspace, not initialised again: the error is sticky
    r2 = dev.results()
    out["sticky_flags"] = r2["flags"].tolist()
    out["sticky_tokens"] = r2["token"].tolist()
    binding.sonic_workspace_init(dev.ws)
    torch.cuda.synchronize()
    dev.run()
    r3 = dev.results()
    out["recovered_tokens"] = r3["token"].tolist()
    out["recovered_flags"] = r3["flags"].tolist()
    out["recovered_prob"] = [float(v) for v in r3["prob"]]
    out["error_word_recovered"] = int(hdr[0].item())
    print("RESULT " + json.dumps(out))


if __name__ == "__main__":
    main()
