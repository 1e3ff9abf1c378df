"""Thin Python binding of the C-ABI library (include/sonic.h).

Argument marshalling only: torch supplies device memory and the current CUDA
stream; every step of the path runs in the library's kernels.  There is no CPU
fallback: if libsonic.so cannot be loaded the import of this module's functions
fails loudly.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import numpy as np
import torch

from . import build as _build
from . import workloads as wl

SONIC_OK = 0
FLAG_NO_TOKEN, FLAG_BADPARAM, FLAG_FALLBACK = 1, 2, 4
MAX_VOCAB = 262144
MAX_TOPK = 4096


class SampleArgs(C.Structure):
    _fields_ = [
        ("struct_size", C.c_uint32), ("B", C.c_int32), ("V", C.c_int32),
        ("logits", C.c_void_p), ("dtype", C.c_int32), ("row_stride", C.c_int64),
        ("mode", C.c_void_p), ("bitmask", C.c_void_p), ("bitmask_stride", C.c_int64),
        ("temperature", C.c_void_p), ("top_k", C.c_void_p), ("top_p", C.c_void_p), ("min_p", C.c_void_p),
        ("rep_penalty", C.c_void_p), ("freq_penalty", C.c_void_p), ("pres_penalty", C.c_void_p),
        ("hist_ids", C.c_void_p), ("hist_counts", C.c_void_p), ("hist_len", C.c_void_p), ("hist_stride", C.c_int32),
        ("bias_ids", C.c_void_p), ("bias_vals", C.c_void_p), ("bias_len", C.c_void_p), ("bias_stride", C.c_int32),
        ("seed", C.c_void_p), ("offset", C.c_void_p),
        ("out_token", C.c_void_p), ("out_prob", C.c_void_p), ("out_flags", C.c_void_p), ("out_support", C.c_void_p),
    ]


class VerifyArgs(C.Structure):
    _fields_ = [
        ("struct_size", C.c_uint32), ("K", C.c_int32), ("s", SampleArgs),
        ("draft_tokens", C.c_void_p), ("draft_probs", C.c_void_p),
        ("out_tokens", C.c_void_p), ("out_accept_len", C.c_void_p), ("out_p_draft", C.c_void_p),
    ]


_lib = None


def lib_path() -> str:
    return _build.LIB


def lib():
    """Loads libsonic.so (building it with nvcc first if it is missing)."""
    global _lib
    if _lib is None:
        path = _build.LIB
        if not os.path.exists(path):
            path = _build.build()
        L = C.CDLL(path)
        L.sonic_workspace_bytes.restype = C.c_size_t
        L.sonic_workspace_bytes.argtypes = [C.c_int]
        L.sonic_workspace_init.restype = C.c_int
        L.sonic_workspace_init.argtypes = [C.c_void_p, C.c_size_t, C.c_void_p]
        L.sonic_sample.restype = C.c_int
        L.sonic_sample.argtypes = [C.POINTER(SampleArgs), C.c_void_p, C.c_size_t, C.c_void_p]
        L.sonic_verify.restype = C.c_int
        L.sonic_verify.argtypes = [C.POINTER(VerifyArgs), C.c_void_p, C.c_size_t, C.c_void_p]
        L.sonic_topk.restype = C.c_int
        L.sonic_topk.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int64, C.c_int, C.c_void_p, C.c_void_p,
                                 C.c_void_p, C.c_size_t, C.c_void_p]
        L.sonic_topk_static.restype = C.c_int
        L.sonic_topk_static.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int64, C.c_int, C.c_void_p,
                                        C.c_void_p, C.c_void_p]
        L.sonic_last_error.restype = C.c_char_p
        _lib = L
    return _lib


class SonicError(RuntimeError):
    def __init__(self, code: int):
        super().__init__(f"sonic error {code}: {lib().sonic_last_error().decode()}")
        self.code = code


def _check(rc: int):
    if rc != SONIC_OK:
        raise SonicError(rc)


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else t.data_ptr()


def sonic_workspace_bytes(max_rows: int) -> int:
    return int(lib().sonic_workspace_bytes(int(max_rows)))


def sonic_workspace_init(ws: torch.Tensor):
    _check(lib().sonic_workspace_init(ws.data_ptr(), ws.numel() * ws.element_size(), _stream()))


def new_workspace(max_rows: int, device="cuda") -> torch.Tensor:
    """Allocates and initialises a workspace for calls over at most max_rows logit rows."""
    ws = torch.empty(sonic_workspace_bytes(max_rows), dtype=torch.uint8, device=device)
    sonic_workspace_init(ws)
    return ws


def sonic_sample(args: SampleArgs, ws: torch.Tensor):
    _check(lib().sonic_sample(C.byref(args), ws.data_ptr(), ws.numel(), _stream()))


def sonic_verify(args: VerifyArgs, ws: torch.Tensor):
    _check(lib().sonic_verify(C.byref(args), ws.data_ptr(), ws.numel(), _stream()))


def sonic_topk(logits: torch.Tensor, dtype: int, B: int, V: int, row_stride: int, k: int,
               out_vals: torch.Tensor, out_idx: torch.Tensor, ws: torch.Tensor):
    _check(lib().sonic_topk(logits.data_ptr(), dtype, B, V, row_stride, k, out_vals.data_ptr(), out_idx.data_ptr(),
                            ws.data_ptr(), ws.numel(), _stream()))


STATIC_MAX_ROWS = 8


def sonic_topk_static(logits: torch.Tensor, dtype: int, B: int, V: int, row_stride: int, k: int,
                      out_vals: torch.Tensor, out_idx: torch.Tensor):
    """sonic_topk for callers that cannot allocate: no workspace argument, at most STATIC_MAX_ROWS rows.
    The scratch is a fixed array inside the library; calls on one device must not overlap."""
    _check(lib().sonic_topk_static(logits.data_ptr(), dtype, B, V, row_stride, k, out_vals.data_ptr(),
                                   out_idx.data_ptr(), _stream()))


# --------------------------------------------------------------------------- device-side holders
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
        self.ws = new_workspace(rows, device) if ws is None else ws
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
    def __init__(self, tw: wl.TopKWorkload, k: int, device="cuda", ws: Optional[torch.Tensor] = None):
        self.tw = tw
        self.k = k
        self.logits = _dev(_padded_logits(tw.logits, tw.dtype), device)
        self.out_vals = torch.zeros((tw.B, k), dtype=torch.float32, device=device)
        self.out_idx = torch.full((tw.B, k), -7, dtype=torch.int32, device=device)
        self.ws = new_workspace(tw.B, device) if ws is None else ws

    def run(self):
        sonic_topk(self.logits, self.tw.dtype, self.tw.B, self.tw.V, self.logits.shape[1], self.k,
                   self.out_vals, self.out_idx, self.ws)

    def results(self):
        torch.cuda.synchronize()
        return self.out_vals.cpu().numpy(), self.out_idx.cpu().numpy()
