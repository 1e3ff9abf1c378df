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

import torch

from . import build as _build

SONIC_OK = 0
FLAG_NO_TOKEN, FLAG_BADPARAM, FLAG_FALLBACK, FLAG_DENSE, FLAG_TIMEOUT = 1, 2, 4, 8, 16
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
        L.sonic_workspace_bytes.argtypes = [C.c_int, C.c_int, C.c_int]
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


def sonic_workspace_bytes(max_rows: int, max_vocab: int = MAX_VOCAB, max_topk: int = MAX_TOPK) -> int:
    return int(lib().sonic_workspace_bytes(int(max_rows), int(max_vocab), int(max_topk)))


def sonic_workspace_init(ws: torch.Tensor):
    _check(lib().sonic_workspace_init(ws.data_ptr(), ws.numel() * ws.element_size(), _stream()))


def new_workspace(max_rows: int, max_vocab: int = MAX_VOCAB, device="cuda") -> torch.Tensor:
    """Allocates and initialises a workspace for calls over at most max_rows logit rows of at most max_vocab entries."""
    ws = torch.empty(sonic_workspace_bytes(max_rows, max_vocab), dtype=torch.uint8, device=device)
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
