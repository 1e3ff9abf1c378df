"""Host-side checks that need no GPU: the C-ABI library loads, exports every symbol the header
declares, sizes its workspace as documented and rejects bad arguments before touching CUDA."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from paper_2607_20475_b200 import binding, workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "sonic.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sonic_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = binding.lib()
    names = declared_symbols()
    assert {"sonic_sample", "sonic_verify", "sonic_topk", "sonic_workspace_bytes", "sonic_workspace_init",
            "sonic_last_error", "sonic_topk_static"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n


def test_struct_layout_matches_header_field_count():
    text = open(os.path.join(ROOT, "include", "sonic.h")).read()
    body = text[text.index("typedef struct sonic_sample_args {"):text.index("} sonic_sample_args;")]
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    fields = [f for f in re.findall(r"([A-Za-z_][A-Za-z_0-9]*)\s*(?:,|;)", body)]
    assert fields == [n for n, _ in binding.SampleArgs._fields_]
    assert C.sizeof(binding.SampleArgs) == 8 * 28 + 8      # 30 fields, natural alignment on LP64


def test_workspace_size_grows_with_rows_and_vocabulary():
    V = binding.MAX_VOCAB
    b1, b2, b64 = (binding.sonic_workspace_bytes(n, V) for n in (1, 2, 64))
    assert b1 < b2 < b64 and b64 < 64 * 1400 * 1024          # about 1.3 MB per row at the largest vocabulary
    assert b2 - b1 > 1024 * 1024
    assert binding.sonic_workspace_bytes(0, V) == b1
    small = binding.sonic_workspace_bytes(64, 32768)
    assert small < b64 // 3                                    # a V = 32768 caller does not pay for V = 262144
    sizes = [binding.sonic_workspace_bytes(64, v) for v in (1, 8192, 8193, 100000, 131072, 262144)]
    assert sizes == sorted(sizes) and sizes[0] == sizes[1] < sizes[2]


def test_bad_arguments_are_rejected_on_the_host():
    lib = binding.lib()
    a = binding.SampleArgs()
    assert lib.sonic_sample(C.byref(a), None, 0, None) == -1            # struct_size mismatch
    assert b"struct_size" in lib.sonic_last_error()
    a.struct_size = C.sizeof(binding.SampleArgs)
    a.B, a.V, a.dtype = 1, 1000, 0
    assert lib.sonic_sample(C.byref(a), None, 0, None) == -1            # NULL logits
    a.logits = 4096
    a.row_stride = 1001                                                 # not a multiple of 16 bytes
    assert lib.sonic_sample(C.byref(a), None, 0, None) == -2
    a.row_stride = 1000
    a.V = binding.MAX_VOCAB + 1
    assert lib.sonic_sample(C.byref(a), None, 0, None) == -2
    a.V = 1000
    a.dtype = 7
    assert lib.sonic_sample(C.byref(a), None, 0, None) == -2
    assert lib.sonic_topk(4096, 0, 2, 1000, 1000, 0, 4096, 4096, None, 0, None) == -2       # k < 1
    assert lib.sonic_topk(4096, 0, 2, 1000, 1000, 5000, 4096, 4096, None, 0, None) == -2    # k > V
    assert lib.sonic_topk_static(4096, 0, 9, 1000, 1000, 4, 4096, 4096, None) == -2         # more rows than the static scratch holds
    v = binding.VerifyArgs()
    v.struct_size = C.sizeof(binding.VerifyArgs)
    v.s.struct_size = C.sizeof(binding.SampleArgs)
    v.K = 16
    assert lib.sonic_verify(C.byref(v), None, 0, None) == -2
    assert lib.sonic_workspace_init(None, 1 << 20, None) == -1


def test_workload_generators_are_seeded_and_well_formed():
    a, b = wl.config2(B=6, V=3000), wl.config2(B=6, V=3000)
    assert np.array_equal(a.logits, b.logits) and np.array_equal(a.hist_ids, b.hist_ids)
    assert a.logits.dtype == np.uint16 and a.mode.dtype == np.uint32
    for r in range(6):
        ids = a.hist_ids[r, : a.hist_len[r]]
        assert len(np.unique(ids)) == len(ids) and a.hist_counts[r, : a.hist_len[r]].sum() == 512
        assert len(np.unique(a.bias_ids[r])) == 16
        assert bool(a.mode[r] & wl.GREEDY) == (r % 2 == 1)
    c = wl.config3(B=4, V=4000)
    allowed = np.unpackbits(c.bitmask.view(np.uint8), axis=1, bitorder="little")[:, :4000]
    raw_am = np.argmax(c.logits, axis=1)
    for r in range(4):
        assert allowed[r, raw_am[r]] == (r % 2 == 0)
        assert abs(int(allowed[r].sum()) - 80) <= 1
    v = wl.config4(B=4, K=2, V=2000)
    assert v.draft_probs.shape == (4, 2, 2000) and np.allclose(v.draft_probs.sum(axis=2), 1.0, atol=1e-5)
    assert np.all(v.draft_probs[np.arange(4)[:, None], np.arange(2)[None, :], v.draft_tokens] > 0)
    assert wl.bf16_bits_to_f32(wl.f32_to_bf16_bits(np.array([1.0, -2.5, 3.140625], np.float32))).tolist() == [1.0, -2.5, 3.140625]
