"""ctypes binding of the CPU oracle (oracle/tslt_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the benchmark's
CPU-baseline leg.  The product package never imports this module, and this module never
imports the product package's CUDA binding.  Arrays are numpy (bf16 logits are passed as
uint16 bit patterns, or as torch CPU tensors which are viewed without copying).
"""
from __future__ import annotations

import ctypes
from typing import Optional

import numpy as np

from .build import build as _build

F32, BF16 = 0, 1
FLAG_SEL, FLAG_SMP, FLAG_ACC, FLAG_RES, FLAG_DEGEN, FLAG_EMPTY = 1, 2, 4, 8, 16, 32

_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        L = ctypes.CDLL(_build())
        c_i, c_ll, c_d, c_p = ctypes.c_int, ctypes.c_longlong, ctypes.c_double, ctypes.c_void_p
        L.tslt_oracle_sparsify.restype = c_i
        L.tslt_oracle_sparsify.argtypes = [c_p, c_i, c_i, c_i, c_ll, c_i, c_d, c_d, c_i, c_p,
                                           c_p, c_p, c_p, c_p, c_p, c_p, c_p, c_p]
        L.tslt_oracle_verify.restype = c_i
        L.tslt_oracle_verify.argtypes = [c_p, c_i, c_i, c_i, c_i, c_ll, c_i, c_p, c_p, c_p, c_p,
                                         c_d, c_d, c_p, c_p, c_p, c_p, c_p, c_p, c_p, c_p, c_p]
        L.tslt_oracle_tree_verify.restype = c_i
        L.tslt_oracle_tree_verify.argtypes = [c_p, c_i, c_i, c_i, c_i, c_ll, c_p, c_p, c_i, c_i,
                                              c_p, c_p, c_p, c_p, c_d, c_d, c_p, c_p, c_i,
                                              c_p, c_p, c_p, c_p, c_p, c_p]
        _lib = L
    return _lib


def as_logits(x):
    """Return (numpy array, dtype code).  Accepts numpy float32 / uint16 (bf16 bits) or a
    torch CPU tensor of float32 / bfloat16."""
    if not isinstance(x, np.ndarray):
        import torch
        assert x.device.type == "cpu"
        x = x.contiguous()
        if x.dtype == torch.bfloat16:
            x = x.view(torch.int16).numpy().view(np.uint16)
        else:
            x = x.numpy()
    if x.dtype == np.float32:
        return np.ascontiguousarray(x), F32
    if x.dtype == np.uint16:
        return np.ascontiguousarray(x), BF16
    raise TypeError("logits must be float32 or bf16 bit patterns (uint16)")


def _np(x, dtype):
    if x is None:
        return None
    if not isinstance(x, np.ndarray):
        x = x.numpy() if hasattr(x, "numpy") else np.asarray(x)
    return np.ascontiguousarray(x, dtype=dtype)


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def sparsify(logits, k: int, top_p: float, temperature: float, uniforms, *, row_stride=None,
             rows=None, want_dense: bool = False):
    """logits [rows, V]; uniforms [rows, num_samples].  Returns a dict of numpy arrays."""
    z, dt = as_logits(logits)
    V = z.shape[-1]
    if rows is None:
        rows = int(np.prod(z.shape[:-1]))
    if row_stride is None:
        row_stride = V
    u = _np(uniforms, np.float32).reshape(rows, -1)
    s = u.shape[1]
    out = dict(idx=np.empty((rows, k), np.int32), logit=np.empty((rows, k), np.float32),
               count=np.empty(rows, np.int32), token=np.empty((rows, s), np.int32),
               lse=np.empty(rows, np.float64), mass=np.empty(rows, np.float64),
               flags=np.empty(rows, np.int32))
    dense = np.empty((rows, V), np.float64) if want_dense else None
    rc = lib().tslt_oracle_sparsify(_ptr(z), dt, rows, V, row_stride, k, float(top_p),
                                    float(temperature), s, _ptr(u), _ptr(out["idx"]),
                                    _ptr(out["logit"]), _ptr(out["count"]), _ptr(out["token"]),
                                    _ptr(out["lse"]), _ptr(out["mass"]), _ptr(out["flags"]),
                                    _ptr(dense))
    if rc != 0:
        raise ValueError("tslt_oracle_sparsify failed with status %d" % rc)
    if want_dense:
        out["qtilde"] = dense
    return out


def verify(target_logits, draft_idx, draft_logit, draft_count, draft_token,
           draft_temperature: float, target_temperature: float, u_accept, u_sample, *,
           row_stride=None, want_dense: bool = False):
    """target_logits [B, gamma+1, V]; drafts [B, gamma, k]; returns a dict of numpy arrays."""
    z, dt = as_logits(target_logits)
    B, g1, V = z.shape
    gamma = g1 - 1
    if row_stride is None:
        row_stride = V
    di = _np(draft_idx, np.int32).reshape(B, gamma, -1)
    k = di.shape[2]
    dl = _np(draft_logit, np.float32).reshape(B, gamma, k)
    dc = _np(draft_count, np.int32).reshape(B, gamma)
    tk = _np(draft_token, np.int32).reshape(B, gamma)
    ua = _np(u_accept, np.float32).reshape(B, gamma)
    us = _np(u_sample, np.float32).reshape(B)
    out = dict(accepted_len=np.empty(B, np.int32), out_token=np.empty(B, np.int32),
               accept_prob=np.empty((B, gamma), np.float64),
               beta_hat=np.empty((B, gamma), np.float64),
               lse_p=np.empty((B, gamma + 1), np.float64), flags=np.empty(B, np.int32))
    dense = np.empty((B, V), np.float64) if want_dense else None
    rc = lib().tslt_oracle_verify(_ptr(z), dt, B, gamma, V, row_stride, k, _ptr(di), _ptr(dl),
                                  _ptr(dc), _ptr(tk), float(draft_temperature),
                                  float(target_temperature), _ptr(ua), _ptr(us),
                                  _ptr(out["accepted_len"]), _ptr(out["out_token"]),
                                  _ptr(out["accept_prob"]), _ptr(out["beta_hat"]),
                                  _ptr(out["lse_p"]), _ptr(out["flags"]), _ptr(dense))
    if rc != 0:
        raise ValueError("tslt_oracle_verify failed with status %d" % rc)
    if want_dense:
        out["final_pmf"] = dense
    return out


def tree_verify(target_logits, parent, node_draft_row, node_token, draft_idx, draft_logit,
                draft_count, draft_temperature: float, target_temperature: float, u_accept,
                u_sample, max_depth: int, *, row_stride=None, want_dense: bool = False):
    """target_logits [B, N, V]; drafts [B, M, k]; returns a dict of numpy arrays."""
    z, dt = as_logits(target_logits)
    B, N, V = z.shape
    if row_stride is None:
        row_stride = V
    par = _np(parent, np.int32).reshape(N)
    ndr = _np(node_draft_row, np.int32).reshape(N)
    M = int((ndr >= 0).sum())
    di = _np(draft_idx, np.int32).reshape(B, max(M, 1), -1) if M else np.zeros((B, 1, 1), np.int32)
    k = di.shape[2]
    dl = _np(draft_logit, np.float32).reshape(B, M, k) if M else np.zeros((B, 1, 1), np.float32)
    dc = _np(draft_count, np.int32).reshape(B, M) if M else np.zeros((B, 1), np.int32)
    tk = _np(node_token, np.int32).reshape(B, N)
    ua = _np(u_accept, np.float32).reshape(B, N)
    us = _np(u_sample, np.float32).reshape(B, N)
    out = dict(accepted_path=np.empty((B, max(max_depth, 1)), np.int32),
               accepted_len=np.empty(B, np.int32), out_token=np.empty(B, np.int32),
               accept_prob=np.empty((B, N), np.float64), flags=np.empty(B, np.int32))
    dense = np.empty((B, V), np.float64) if want_dense else None
    rc = lib().tslt_oracle_tree_verify(_ptr(z), dt, B, N, V, row_stride, _ptr(par), _ptr(ndr),
                                       M, k, _ptr(tk), _ptr(di), _ptr(dl), _ptr(dc),
                                       float(draft_temperature), float(target_temperature),
                                       _ptr(ua), _ptr(us), max_depth,
                                       _ptr(out["accepted_path"]), _ptr(out["accepted_len"]),
                                       _ptr(out["out_token"]), _ptr(out["accept_prob"]),
                                       _ptr(out["flags"]), _ptr(dense))
    if rc != 0:
        raise ValueError("tslt_oracle_tree_verify failed with status %d" % rc)
    out["accepted_path"] = out["accepted_path"][:, :max_depth]
    if want_dense:
        out["final_pmf"] = dense
    return out
