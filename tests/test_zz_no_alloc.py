"""sonic_topk_static: the entry point for callers that must not allocate device memory
(a plugin under a fixed memory budget, a process whose pool was sized at start-up, a
serving loop in which cudaMalloc would stall the device).  It takes no workspace: its scratch is a fixed array inside the
library.  Checked here against sonic_topk, bit for bit, on two calls in a row with
different inputs, so that what the first call leaves in the shared array cannot leak
into the second; and against the CPU oracle's sorted top-k as well, so that the check does
not rest on the other entry point alone.  Collected last on purpose."""
import numpy as np
import pytest

from paper_2607_20475_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def test_static_scratch_topk_matches_workspace_topk_twice():
    import torch
    from paper_2607_20475_b200 import harness as binding

    binding.lib()
    B, V = binding.STATIC_MAX_ROWS, 70001
    for call, (regime, k) in enumerate((("normal", 64), ("zeros", 3000))):   # second call: all ties, exact path
        tw = wl.config5(regime, B=B, V=V)
        ref = binding.DeviceTopK(tw, k)
        ref.run()
        ref_vals, ref_idx = ref.results()
        out_vals = torch.full((B, k), -1.0, dtype=torch.float32, device="cuda")
        out_idx = torch.full((B, k), -7, dtype=torch.int32, device="cuda")
        binding.sonic_topk_static(ref.logits, tw.dtype, B, V, ref.logits.shape[1], k, out_vals, out_idx)
        torch.cuda.synchronize()
        assert np.array_equal(out_idx.cpu().numpy(), ref_idx), f"call {call}: indices differ"
        assert np.array_equal(out_vals.cpu().numpy().view(np.uint32), ref_vals.view(np.uint32)), f"call {call}"
        from oracle import oracle
        ov, oi = oracle.topk(tw.logits_f32(), k)
        assert np.array_equal(out_idx.cpu().numpy(), oi), f"call {call}: indices differ from the oracle's"
        assert np.array_equal(out_vals.cpu().numpy().view(np.uint32), ov.view(np.uint32)), f"call {call}: values differ from the oracle's"


def test_static_scratch_rejects_more_rows_than_it_holds():
    import torch
    from paper_2607_20475_b200 import harness as binding

    B, V, k = binding.STATIC_MAX_ROWS + 1, 4096, 4
    x = torch.zeros((B, V), dtype=torch.float32, device="cuda")
    ov = torch.zeros((B, k), dtype=torch.float32, device="cuda")
    oi = torch.zeros((B, k), dtype=torch.int32, device="cuda")
    with pytest.raises(binding.SonicError) as err:
        binding.sonic_topk_static(x, wl.DTYPE_F32, B, V, V, k, ov, oi)
    assert err.value.code == -2 and "SONIC_STATIC_MAX_ROWS" in str(err.value)
