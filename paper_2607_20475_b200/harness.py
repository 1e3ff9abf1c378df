"""Seeded synthetic workloads held on the GPU, with their output buffers and argument structs: what the
tests, the smoke check and the benchmark use to call the library.  Not part of the binding proper
(paper_2607_20475_b200.binding, which only marshals arguments); nothing here computes any step of the path."""
from __future__ import annotations

import ctypes as C
from typing import Optional

import numpy as np
import torch

from . import workloads as wl
from .binding import (FLAG_BADPARAM, FLAG_DENSE, FLAG_FALLBACK, FLAG_NO_TOKEN, FLAG_TIMEOUT, MAX_TOPK, MAX_VOCAB,  # noqa: F401
                      STATIC_MAX_ROWS, SampleArgs, SonicError, VerifyArgs, _ptr, lib, lib_path, new_workspace,
                      sonic_sample, sonic_topk, sonic_topk_static, sonic_verify, sonic_workspace_bytes,
                      sonic_workspace_init)


def _dev(a: Optional[np.ndarray], device, pin=False):
    if a is None:
        return None
    if a.dtype == np.uint32:
        t = torch.from_numpy(np.ascontiguousarray(a).view(np.int32))
    elif a.dtype == np.uint64:
        t = torch.from_numpy(np.ascontiguousarray(a).view(np.int64))
    elif a.dtype == np.uint16:
        t = torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).view(torch.bfloat16)
    else:
        t = torch.from_numpy(np.ascontiguousarray(a))
    return t.to(device)


def _padded_logits(logits: np.ndarray, dtype: int) -> np.ndarray:
    """Pads rows to a 16-byte multiple; the padding holds a huge value the kernels must never read as data."""
    vec = 4 if dtype == wl.DTYPE_F32 else 8
    rows, V = logits.shape
    stride = (V + vec - 1) // vec * vec
    if stride == V:
        return logits
    out = np.empty((rows, stride), dtype=logits.dtype)
    out[:, :V] = logits
    out[:, V:] = np.float32(1e30) if dtype == wl.DTYPE_F32 else np.uint16(0x7F00)
    return out


class DeviceSample:
    """A SampleWorkload resident on the GPU with its outputs and argument struct."""

    def __init__(self, w: wl.SampleWorkload, device="cuda", ws: Optional[torch.Tensor] = None, rows: Optional[int] = None):
        self.w = w
        self.device = device
        rows = w.logits.shape[0] if rows is None else rows
        self.t = {}
        for name in ("mode", "bitmask", "temperature", "top_k", "top_p", "min_p", "rep_penalty",
                     "freq_penalty", "pres_penalty", "hist_ids", "hist_counts", "hist_len", "bias_ids", "bias_vals",
                     "bias_len", "seed", "offset"):
            self.t[name] = _dev(getattr(w, name), device)
        self.t["logits"] = _dev(_padded_logits(w.logits, w.dtype), device)
        B = w.B
        self.out_token = torch.full((B,), -7, dtype=torch.int32, device=device)
        self.out_prob = torch.zeros(B, dtype=torch.float32, device=device)
        self.out_flags = torch.zeros(B, dtype=torch.int32, device=device)
        self.out_support = torch.zeros(B, dtype=torch.int32, device=device)
        self.ws = new_workspace(rows, w.V, device) if ws is None else ws
        self.args = self._args()

    def _args(self) -> SampleArgs:
        w, t = self.w, self.t
        a = SampleArgs()
        a.struct_size = C.sizeof(SampleArgs)
        a.B, a.V = w.B, w.V
        a.logits = _ptr(t["logits"])
        a.dtype = w.dtype
        a.row_stride = self.t["logits"].shape[1]
        a.mode = _ptr(t["mode"])
        a.bitmask = _ptr(t["bitmask"])
        a.bitmask_stride = 0 if w.bitmask is None else w.bitmask.shape[-1]
        for name in ("temperature", "top_k", "top_p", "min_p", "rep_penalty", "freq_penalty", "pres_penalty",
                     "hist_ids", "hist_counts", "hist_len", "bias_ids", "bias_vals", "bias_len", "seed", "offset"):
            setattr(a, name, _ptr(t[name]))
        a.hist_stride = 0 if w.hist_ids is None else w.hist_ids.shape[1]
        a.bias_stride = 0 if w.bias_ids is None else w.bias_ids.shape[1]
        a.out_token = _ptr(self.out_token)
        a.out_prob = _ptr(self.out_prob)
        a.out_flags = _ptr(self.out_flags)
        a.out_support = _ptr(self.out_support)
        return a

    def run(self):
        sonic_sample(self.args, self.ws)

    def results(self):
        torch.cuda.synchronize()
        return dict(token=self.out_token.cpu().numpy(), prob=self.out_prob.cpu().numpy(),
                    flags=self.out_flags.cpu().numpy().view(np.uint32), support=self.out_support.cpu().numpy())


class DeviceVerify:
    """A VerifyWorkload resident on the GPU."""

    def __init__(self, vw: wl.VerifyWorkload, device="cuda", ws: Optional[torch.Tensor] = None):
        self.vw = vw
        B, K = vw.B, vw.K
        self.s = DeviceSample(vw.sample, device, ws=ws, rows=B * (K + 1))
        self.ws = self.s.ws
        self.draft_tokens = _dev(np.ascontiguousarray(vw.draft_tokens, np.int32), device)
        self.draft_probs = _dev(np.ascontiguousarray(vw.draft_probs, np.float32), device)
        self.out_tokens = torch.full((B, K + 1), -7, dtype=torch.int32, device=device)
        self.out_accept = torch.zeros(B, dtype=torch.int32, device=device)
        self.out_p_draft = torch.zeros((B, max(K, 1)), dtype=torch.float32, device=device)
        a = VerifyArgs()
        a.struct_size = C.sizeof(VerifyArgs)
        a.K = K
        a.s = self.s.args
        a.draft_tokens = _ptr(self.draft_tokens) if K > 0 else None
        a.draft_probs = _ptr(self.draft_probs) if K > 0 else None
        a.out_tokens = _ptr(self.out_tokens)
        a.out_accept_len = _ptr(self.out_accept)
        a.out_p_draft = _ptr(self.out_p_draft)
        self.args = a

    def run(self):
        sonic_verify(self.args, self.ws)

    def results(self):
        torch.cuda.synchronize()
        K = self.vw.K
        return dict(tokens=self.out_tokens.cpu().numpy(), accept_len=self.out_accept.cpu().numpy(),
                    p_draft=self.out_p_draft.cpu().numpy()[:, :K],
                    flags=self.s.out_flags.cpu().numpy().view(np.uint32))


class DeviceTopK:
    def __init__(self, tw: wl.TopKWorkload, k: int, device="cuda", ws: Optional[torch.Tensor] = None,
                 logits: Optional[torch.Tensor] = None):
        self.tw = tw
        self.k = k
        self.logits = _dev(_padded_logits(tw.logits, tw.dtype), device) if logits is None else logits   # (shared between holders of several k)
        self.out_vals = torch.zeros((tw.B, k), dtype=torch.float32, device=device)
        self.out_idx = torch.full((tw.B, k), -7, dtype=torch.int32, device=device)
        self.ws = new_workspace(tw.B, tw.V, device) if ws is None else ws

    def run(self):
        sonic_topk(self.logits, self.tw.dtype, self.tw.B, self.tw.V, self.logits.shape[1], self.k,
                   self.out_vals, self.out_idx, self.ws)

    def results(self):
        torch.cuda.synchronize()
        return self.out_vals.cpu().numpy(), self.out_idx.cpu().numpy()
