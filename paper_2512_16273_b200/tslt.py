"""Thin Python binding of libtslt (include/tslt.h): argument marshalling only.

Every step of the hot path runs in the CUDA kernels of libtslt.so; this module checks
shapes, hands raw device pointers and the current CUDA stream to the C ABI, and uses torch
only to own device memory.  There is no CPU fallback: importing the binding without the
built library, or calling it with CPU tensors, raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Dict, Optional, Sequence

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libtslt.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_DEVICE_STATUS = 0, -1, -2, -3, -4, -5
ERR_STATIC_SCRATCH = -6
STATIC_SCRATCH_BYTES = 8 << 20
F32, BF16 = 0, 1
MAX_K = 1024

EXPORTS = ["tslt_version", "tslt_status_string", "tslt_workspace_status", "tslt_set_ready_poll_limit",
           "tslt_sparsify_workspace_bytes", "tslt_sparsify", "tslt_sparsify_shard", "tslt_sparsify_merge",
           "tslt_verify_workspace_bytes", "tslt_verify", "tslt_verify_static",
           "tslt_tree_verify_workspace_bytes", "tslt_tree_verify",
           "tslt_tree_verify_walk_workspace_bytes", "tslt_tree_verify_walk",
           "tslt_payload_words", "tslt_pack_payload", "tslt_unpack_payload",
           "tslt_verify_packed", "tslt_tree_verify_packed",
           "tslt_diagnostics_workspace_bytes", "tslt_diagnostics"]

PROB_F32, PROB_BF16, PROB_F16 = 0, 1, 2


class TsltError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s failed: %s (status %d)" % (where, status_string(status), status))


_lib = None


def lib() -> ctypes.CDLL:
    """Load libtslt.so (built in-tree by paper_2512_16273_b200/build.py).  Raises if absent."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise ImportError("libtslt.so is not built: run `python -m paper_2512_16273_b200.build` "
                          "(nvcc, sm_100a).  There is no fallback path.")
    L = ctypes.CDLL(_LIB_PATH)
    i, ll, f, p, sz = ctypes.c_int, ctypes.c_longlong, ctypes.c_float, ctypes.c_void_p, ctypes.c_size_t
    psz = ctypes.POINTER(ctypes.c_size_t)
    L.tslt_version.restype = i
    L.tslt_version.argtypes = []
    L.tslt_status_string.restype = ctypes.c_char_p
    L.tslt_status_string.argtypes = [i]
    L.tslt_workspace_status.restype = i
    L.tslt_workspace_status.argtypes = [p, p, ctypes.POINTER(i)]
    L.tslt_set_ready_poll_limit.restype = i
    L.tslt_set_ready_poll_limit.argtypes = [i]
    L.tslt_sparsify_workspace_bytes.restype = i
    L.tslt_sparsify_workspace_bytes.argtypes = [i, i, i, i, psz]
    L.tslt_sparsify.restype = i
    L.tslt_sparsify.argtypes = [p, i, i, i, i, ll, i, f, f, i, p, p, p, p, p, p, p, p, sz, p]
    L.tslt_sparsify_shard.restype = i
    L.tslt_sparsify_shard.argtypes = [p, i, i, i, ll, i, f, p, p, p, p, p, sz, p]
    L.tslt_sparsify_merge.restype = i
    L.tslt_sparsify_merge.argtypes = [i, i, i, ctypes.POINTER(i), i, p, p, p, p, f, f, i, p, p, p, p, p, p, p, p, sz, p]
    L.tslt_verify_workspace_bytes.restype = i
    L.tslt_verify_workspace_bytes.argtypes = [i, i, i, i, psz]
    L.tslt_verify.restype = i
    L.tslt_verify.argtypes = [p, i, i, i, i, ll, i, p, p, p, p, f, f, p, p, p, p, p, p, p, p, sz, p]
    L.tslt_verify_static.restype = i
    L.tslt_verify_static.argtypes = [p, i, i, i, i, ll, i, p, p, p, p, f, f, p, p, p, p, p, p, p, p]
    L.tslt_tree_verify_workspace_bytes.restype = i
    L.tslt_tree_verify_workspace_bytes.argtypes = [i, i, i, i, psz]
    L.tslt_tree_verify.restype = i
    L.tslt_tree_verify.argtypes = [p, i, i, i, i, ll, p, p, i, i, p, p, p, p, f, f, p, p, i, p, p, p,
                                   p, sz, p]
    L.tslt_tree_verify_walk_workspace_bytes.restype = i
    L.tslt_tree_verify_walk_workspace_bytes.argtypes = [i, i, i, i, psz]
    L.tslt_tree_verify_walk.restype = i
    L.tslt_tree_verify_walk.argtypes = L.tslt_tree_verify.argtypes
    L.tslt_diagnostics_workspace_bytes.restype = i
    L.tslt_diagnostics_workspace_bytes.argtypes = [i, i, i, i, psz]
    L.tslt_diagnostics.restype = i
    L.tslt_diagnostics.argtypes = [p, p, i, i, i, ll, p, i, i, f, f, p, p, p, p, p, p, p, sz, p]
    L.tslt_verify_packed.restype = i
    L.tslt_verify_packed.argtypes = [p, i, i, i, i, ll, i, p, i, p, f, f, p, p, p, p, p, p, p, p, sz, p]
    L.tslt_tree_verify_packed.restype = i
    L.tslt_tree_verify_packed.argtypes = [i, p, i, i, i, i, ll, p, p, i, i, p, p, i, f, f, p, p, i, p, p, p, p, sz, p]
    L.tslt_payload_words.restype = i
    L.tslt_payload_words.argtypes = [i, i, i, ctypes.POINTER(i), ctypes.POINTER(i)]
    L.tslt_pack_payload.restype = i
    L.tslt_pack_payload.argtypes = [p, p, p, i, i, i, i, p, p, p]
    L.tslt_unpack_payload.restype = i
    L.tslt_unpack_payload.argtypes = [p, i, i, i, i, p, p, p, p, p]
    _lib = L
    return L


def version() -> int:
    return lib().tslt_version()


def status_string(status: int) -> str:
    return lib().tslt_status_string(int(status)).decode()


def _check(status: int, where: str) -> None:
    if status != OK:
        raise TsltError(status, where)


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TsltError(ERR_UNSUPPORTED, "dtype %s" % t.dtype)


def _cuda(t: Optional[torch.Tensor], name: str, dtype=None) -> Optional[torch.Tensor]:
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError("%s must be a CUDA tensor (libtslt has no CPU path)" % name)
    if dtype is not None and t.dtype != dtype:
        raise ValueError("%s must have dtype %s" % (name, dtype))
    if not t.is_contiguous():
        raise ValueError("%s must be contiguous" % name)
    return t


def _out(o: dict, name: str, dtype, numel: int, required: bool = True) -> None:
    """An output buffer the kernels will write: CUDA, contiguous, the right dtype and size."""
    t = o.get(name)
    if t is None:
        if required:
            raise ValueError("output %s is missing" % name)
        return
    _cuda(t, name, dtype)
    if t.numel() != numel:
        raise ValueError("output %s must have %d elements, has %d" % (name, numel, t.numel()))


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream() -> ctypes.c_void_p:
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _row_layout(logits: torch.Tensor):
    """(rows, V, row stride in elements) of a tensor [..., V] whose leading dimensions flatten
    to equally spaced rows (a contiguous tensor, or a [:, ..., :V] view of a padded one)."""
    if logits.dim() < 1 or (logits.shape[-1] > 1 and logits.stride(-1) != 1):
        raise ValueError("logits must be contiguous along the vocabulary")
    V = logits.shape[-1]
    rows = logits.numel() // V if V else 0
    if logits.dim() == 1:
        return rows, V, V
    stride = logits.stride(-2)
    for d in range(logits.dim() - 2):
        if logits.shape[d] > 1 and logits.stride(d) != logits.stride(d + 1) * logits.shape[d + 1]:
            raise ValueError("rows of logits must be equally spaced in memory")
    if rows <= 1 or logits.shape[-2] == 1:
        # a single row per block: take the spacing from the next dimension that has one
        stride = V
        for d in range(logits.dim() - 2, -1, -1):
            if logits.shape[d] > 1:
                stride = logits.stride(d)
                break
    return rows, V, max(int(stride), V)


_ws_cache: Dict[tuple, torch.Tensor] = {}


def workspace(nbytes: int, device) -> torch.Tensor:
    """A cached device buffer of at least nbytes (torch's allocator returns >= 512-byte aligned)."""
    key = (str(device), torch.cuda.current_stream(device).cuda_stream)
    ws = _ws_cache.get(key)
    if ws is None or ws.numel() < nbytes:
        ws = torch.empty(max(int(nbytes), 4096), dtype=torch.uint8, device=device)
        _ws_cache[key] = ws
    return ws


def sparsify_workspace_bytes(rows: int, V: int, k: int, num_samples: int) -> int:
    n = ctypes.c_size_t(0)
    _check(lib().tslt_sparsify_workspace_bytes(rows, V, k, num_samples, ctypes.byref(n)),
           "tslt_sparsify_workspace_bytes")
    return int(n.value)


def verify_workspace_bytes(B: int, gamma: int, V: int, k: int) -> int:
    n = ctypes.c_size_t(0)
    _check(lib().tslt_verify_workspace_bytes(B, gamma, V, k, ctypes.byref(n)), "tslt_verify_workspace_bytes")
    return int(n.value)


def tree_verify_workspace_bytes(B: int, N: int, V: int, k: int) -> int:
    n = ctypes.c_size_t(0)
    _check(lib().tslt_tree_verify_workspace_bytes(B, N, V, k, ctypes.byref(n)),
           "tslt_tree_verify_workspace_bytes")
    return int(n.value)


def workspace_status(ws: torch.Tensor) -> int:
    """Synchronous: device status word of a workspace (0 = every device-side wait completed)."""
    word = ctypes.c_int(0)
    rc = lib().tslt_workspace_status(_ptr(ws), _stream(), ctypes.byref(word))
    if rc not in (OK, ERR_DEVICE_STATUS):
        raise TsltError(rc, "tslt_workspace_status")
    return int(word.value)


STATUS_WAIT_FELL_BACK = 1
STATUS_BAD_RECORD = 2


def set_ready_poll_limit(polls: int) -> None:
    """Process-wide: polls a finish CTA of tslt_sparsify spends on its row's ready flags before it
    takes the fall-back (and sets STATUS_WAIT_FELL_BACK in the status word).  0: at once."""
    _check(lib().tslt_set_ready_poll_limit(int(polls)), "tslt_set_ready_poll_limit")


def sparsify(logits: torch.Tensor, k: int, top_p: float = 1.0, temperature: float = 1.0,
             uniforms: Optional[torch.Tensor] = None, *, want_stats: bool = True,
             out: Optional[dict] = None, ws: Optional[torch.Tensor] = None) -> dict:
    """tslt_sparsify on logits [..., V] (fp32 / bf16, CUDA).  uniforms [rows, num_samples] fp32.

    Returns dict(idx [rows,k] int32, logit [rows,k] fp32, count [rows] int32,
    token [rows,num_samples] int32, lse [rows] fp32, mass [rows] fp32, workspace)."""
    if not logits.is_cuda:
        raise ValueError("logits must be a CUDA tensor (libtslt has no CPU path)")
    rows, V, stride = _row_layout(logits)
    flat = logits
    dev = logits.device
    ns = 0
    if uniforms is not None:
        _cuda(uniforms, "uniforms", torch.float32)
        if rows and uniforms.numel() % rows:
            raise ValueError("uniforms must be [rows, num_samples]")
        ns = uniforms.numel() // rows if rows else 0
    o = out if out is not None else {}
    if "idx" not in o:
        o["idx"] = torch.empty(rows, k, dtype=torch.int32, device=dev)
        o["logit"] = torch.empty(rows, k, dtype=torch.float32, device=dev)
        o["count"] = torch.empty(rows, dtype=torch.int32, device=dev)
        o["token"] = torch.empty(rows, ns, dtype=torch.int32, device=dev)
        if want_stats:
            o["lse"] = torch.empty(rows, dtype=torch.float32, device=dev)
            o["mass"] = torch.empty(rows, dtype=torch.float32, device=dev)
    for name, dt, ne, req in (("idx", torch.int32, rows * k, True), ("logit", torch.float32, rows * k, True),
                              ("count", torch.int32, rows, True), ("token", torch.int32, rows * ns, True),
                              ("lse", torch.float32, rows, False), ("mass", torch.float32, rows, False)):
        _out(o, name, dt, ne, req)
    if ws is None:
        ws = workspace(sparsify_workspace_bytes(rows, V, k, ns), dev)
    rc = lib().tslt_sparsify(_ptr(flat), _dtype_code(logits), rows, 1, V, stride, k, top_p, temperature,
                             ns, _ptr(uniforms), _ptr(o["idx"]), _ptr(o["logit"]), _ptr(o["count"]),
                             _ptr(o["token"]), _ptr(o.get("lse")), _ptr(o.get("mass")), _ptr(ws),
                             ws.numel(), _stream())
    _check(rc, "tslt_sparsify")
    o["workspace"] = ws
    return o


MAX_SHARDS = 16


def sparsify_shard(logits_shard: torch.Tensor, k: int, temperature: float = 1.0, *, out: Optional[dict] = None,
                   ws: Optional[torch.Tensor] = None) -> dict:
    """tslt_sparsify_shard on one vocabulary shard [rows, V_shard] (a column slice of a wider tensor
    is fine if it starts on a 16-byte boundary).  Returns dict(idx, logit [rows, k], count [rows]
    int32, lse2 [rows] fp64, workspace); idx is local to the shard."""
    if not logits_shard.is_cuda:
        raise ValueError("logits must be a CUDA tensor (libtslt has no CPU path)")
    rows, V, stride = _row_layout(logits_shard)
    dev = logits_shard.device
    o = out if out is not None else {}
    if "idx" not in o:
        o["idx"] = torch.empty(rows, k, dtype=torch.int32, device=dev)
        o["logit"] = torch.empty(rows, k, dtype=torch.float32, device=dev)
        o["count"] = torch.empty(rows, dtype=torch.int32, device=dev)
        o["lse2"] = torch.empty(rows, dtype=torch.float64, device=dev)
    for name, dt, ne in (("idx", torch.int32, rows * k), ("logit", torch.float32, rows * k),
                         ("count", torch.int32, rows), ("lse2", torch.float64, rows)):
        _out(o, name, dt, ne)
    if ws is None:
        ws = workspace(sparsify_workspace_bytes(rows, V, k, 0), dev)
    rc = lib().tslt_sparsify_shard(_ptr(logits_shard), _dtype_code(logits_shard), rows, V, stride, k, temperature,
                                   _ptr(o["idx"]), _ptr(o["logit"]), _ptr(o["count"]), _ptr(o["lse2"]), _ptr(ws),
                                   ws.numel(), _stream())
    _check(rc, "tslt_sparsify_shard")
    o["workspace"] = ws
    return o


def sparsify_merge(part_idx: torch.Tensor, part_logit: torch.Tensor, part_count: torch.Tensor,
                   part_lse2: torch.Tensor, shard_offset: Sequence[int], dtype: torch.dtype, top_p: float = 1.0,
                   temperature: float = 1.0, uniforms: Optional[torch.Tensor] = None, *, want_stats: bool = True,
                   out: Optional[dict] = None, ws: Optional[torch.Tensor] = None) -> dict:
    """tslt_sparsify_merge: part_idx / part_logit [nshards, rows, k], part_count (int32) / part_lse2
    (fp64) [nshards, rows], as the shards wrote them; dtype = the logits' element type.  Returns what
    sparsify() returns for the whole-vocabulary rows."""
    _cuda(part_idx, "part_idx", torch.int32)
    _cuda(part_logit, "part_logit", torch.float32)
    _cuda(part_count, "part_count", torch.int32)
    _cuda(part_lse2, "part_lse2", torch.float64)
    if part_idx.dim() != 3 or part_idx.shape != part_logit.shape:
        raise ValueError("part_idx and part_logit must be [nshards, rows, k]")
    nshards, rows, k = part_idx.shape
    if tuple(part_count.shape) != (nshards, rows) or tuple(part_lse2.shape) != (nshards, rows):
        raise ValueError("part_count and part_lse2 must be [nshards, rows]")
    if len(shard_offset) != nshards:
        raise ValueError("one offset per shard")
    dev = part_idx.device
    ns = 0
    if uniforms is not None:
        _cuda(uniforms, "uniforms", torch.float32)
        if rows and uniforms.numel() % rows:
            raise ValueError("uniforms must be [rows, num_samples]")
        ns = uniforms.numel() // rows if rows else 0
    o = out if out is not None else {}
    if "idx" not in o:
        o["idx"] = torch.empty(rows, k, dtype=torch.int32, device=dev)
        o["logit"] = torch.empty(rows, k, dtype=torch.float32, device=dev)
        o["count"] = torch.empty(rows, dtype=torch.int32, device=dev)
        o["token"] = torch.empty(rows, ns, dtype=torch.int32, device=dev)
        if want_stats:
            o["lse"] = torch.empty(rows, dtype=torch.float32, device=dev)
            o["mass"] = torch.empty(rows, dtype=torch.float32, device=dev)
    for name, dt, ne, req in (("idx", torch.int32, rows * k, True), ("logit", torch.float32, rows * k, True),
                              ("count", torch.int32, rows, True), ("token", torch.int32, rows * ns, True),
                              ("lse", torch.float32, rows, False), ("mass", torch.float32, rows, False)):
        _out(o, name, dt, ne, req)
    if ws is None:
        ws = torch.empty(4096, dtype=torch.uint8, device=dev)
    code = F32 if dtype == torch.float32 else BF16 if dtype == torch.bfloat16 else None
    if code is None:
        raise TsltError(ERR_UNSUPPORTED, "dtype %s" % dtype)
    offs = (ctypes.c_int * nshards)(*[int(x) for x in shard_offset])
    rc = lib().tslt_sparsify_merge(code, rows, nshards, offs, k, _ptr(part_idx), _ptr(part_logit), _ptr(part_count),
                                   _ptr(part_lse2), top_p, temperature, ns, _ptr(uniforms), _ptr(o["idx"]),
                                   _ptr(o["logit"]), _ptr(o["count"]), _ptr(o["token"]), _ptr(o.get("lse")),
                                   _ptr(o.get("mass")), _ptr(ws), ws.numel(), _stream())
    _check(rc, "tslt_sparsify_merge")
    o["workspace"] = ws
    return o


def sparsify_sharded(logits: torch.Tensor, shard_bounds: Sequence[int], k: int, top_p: float = 1.0,
                     temperature: float = 1.0, uniforms: Optional[torch.Tensor] = None) -> dict:
    """The two-stage path on ONE device: logits [rows, V] are cut at shard_bounds (ascending token
    ids 0 = b_0 < b_1 < ... < b_n = V, each a multiple of 16 bytes' worth of elements), every slice
    goes through sparsify_shard with its own workspace, and sparsify_merge joins them.  On several
    devices each rank runs sparsify_shard on its slice and the parts are all-gathered before the
    merge; the kernels are the same."""
    if logits.dim() != 2:
        raise ValueError("logits must be [rows, V]")
    rows, V = logits.shape
    b = [int(x) for x in shard_bounds]
    if len(b) < 2 or b[0] != 0 or b[-1] != V or any(y <= x for x, y in zip(b, b[1:])):
        raise ValueError("shard_bounds must ascend from 0 to V")
    n = len(b) - 1
    dev = logits.device
    part = dict(idx=torch.empty(n, rows, k, dtype=torch.int32, device=dev),
                logit=torch.empty(n, rows, k, dtype=torch.float32, device=dev),
                count=torch.empty(n, rows, dtype=torch.int32, device=dev),
                lse2=torch.empty(n, rows, dtype=torch.float64, device=dev))
    spaces = []
    for s in range(n):
        sl = logits[:, b[s]:b[s + 1]]
        ws = torch.empty(max(sparsify_workspace_bytes(rows, b[s + 1] - b[s], k, 0), 4096), dtype=torch.uint8, device=dev)
        sparsify_shard(sl, k, temperature, out={name: part[name][s] for name in part}, ws=ws)
        spaces.append(ws)
    o = sparsify_merge(part["idx"], part["logit"], part["count"], part["lse2"], b[:-1], logits.dtype, top_p,
                       temperature, uniforms)
    o["parts"] = part
    o["shard_workspaces"] = spaces
    return o


def _check_verify_outputs(o: dict, B: int, gamma: int) -> None:
    for name, dt, ne, req in (("accepted_len", torch.int32, B, True), ("out_token", torch.int32, B, True),
                              ("accept_prob", torch.float32, B * gamma, False),
                              ("beta_hat", torch.float32, B * gamma, False),
                              ("lse_p", torch.float32, B * (gamma + 1), False)):
        _out(o, name, dt, ne, req)


def verify(target_logits: torch.Tensor, draft_idx: torch.Tensor, draft_logit: torch.Tensor,
           draft_count: torch.Tensor, draft_token: torch.Tensor, draft_temperature: float,
           target_temperature: float, u_accept: torch.Tensor, u_sample: torch.Tensor, *,
           want_diag: bool = True, out: Optional[dict] = None,
           ws: Optional[torch.Tensor] = None) -> dict:
    """tslt_verify.  target_logits [B, gamma+1, V]; drafts [B, gamma, k] as written by sparsify.

    Returns dict(accepted_len [B], out_token [B], and with want_diag accept_prob, beta_hat
    [B, gamma], lse_p [B, gamma+1], workspace)."""
    if not target_logits.is_cuda:
        raise ValueError("target_logits must be a CUDA tensor (libtslt has no CPU path)")
    if target_logits.dim() != 3:
        raise ValueError("target_logits must be [B, gamma+1, V]")
    B, g1, V = target_logits.shape
    _, _, stride = _row_layout(target_logits)
    gamma = g1 - 1
    k = draft_idx.shape[-1] if gamma > 0 else 1
    dev = target_logits.device
    _cuda(draft_idx, "draft_idx", torch.int32)
    _cuda(draft_logit, "draft_logit", torch.float32)
    _cuda(draft_count, "draft_count", torch.int32)
    _cuda(draft_token, "draft_token", torch.int32)
    _cuda(u_accept, "u_accept", torch.float32)
    _cuda(u_sample, "u_sample", torch.float32)
    if draft_idx.numel() != B * gamma * k or draft_logit.numel() != B * gamma * k or \
            draft_count.numel() != B * gamma or draft_token.numel() != B * gamma or \
            u_accept.numel() != B * gamma or u_sample.numel() != B:
        raise ValueError("draft / uniform shapes do not match target_logits")
    o = out if out is not None else {}
    if "accepted_len" not in o:
        o["accepted_len"] = torch.empty(B, dtype=torch.int32, device=dev)
        o["out_token"] = torch.empty(B, dtype=torch.int32, device=dev)
        if want_diag:
            o["accept_prob"] = torch.empty(B, gamma, dtype=torch.float32, device=dev)
            o["beta_hat"] = torch.empty(B, gamma, dtype=torch.float32, device=dev)
            o["lse_p"] = torch.empty(B, gamma + 1, dtype=torch.float32, device=dev)
    _check_verify_outputs(o, B, gamma)
    if ws is None:
        ws = workspace(verify_workspace_bytes(B, gamma, V, k), dev)
    rc = lib().tslt_verify(_ptr(target_logits), _dtype_code(target_logits), B, gamma, V, stride, k,
                           _ptr(draft_idx), _ptr(draft_logit), _ptr(draft_count), _ptr(draft_token),
                           draft_temperature, target_temperature, _ptr(u_accept), _ptr(u_sample),
                           _ptr(o["accepted_len"]), _ptr(o["out_token"]), _ptr(o.get("accept_prob")),
                           _ptr(o.get("beta_hat")), _ptr(o.get("lse_p")), _ptr(ws), ws.numel(), _stream())
    _check(rc, "tslt_verify")
    o["workspace"] = ws
    return o


def verify_static(target_logits: torch.Tensor, draft_idx: torch.Tensor, draft_logit: torch.Tensor,
                  draft_count: torch.Tensor, draft_token: torch.Tensor, draft_temperature: float,
                  target_temperature: float, u_accept: torch.Tensor, u_sample: torch.Tensor, out: dict) -> dict:
    """tslt_verify_static: tslt_verify for callers that may not allocate device memory.  The scratch
    is an 8 MiB array built into the library (shared by all calls on the device, so calls must not
    overlap), and this wrapper allocates nothing either: `out` must already hold the output tensors
    accepted_len [B] and out_token [B] (int32) and may hold accept_prob, beta_hat [B, gamma] and
    lse_p [B, gamma+1] (fp32).  Raises TsltError(ERR_STATIC_SCRATCH) when the problem needs more
    scratch than the array holds."""
    if not target_logits.is_cuda or target_logits.dim() != 3:
        raise ValueError("target_logits must be a CUDA tensor [B, gamma+1, V]")
    B, g1, V = target_logits.shape
    _, _, stride = _row_layout(target_logits)
    gamma = g1 - 1
    k = draft_idx.shape[-1] if gamma > 0 else 1
    for name, t, dt in (("draft_idx", draft_idx, torch.int32), ("draft_logit", draft_logit, torch.float32),
                        ("draft_count", draft_count, torch.int32), ("draft_token", draft_token, torch.int32),
                        ("u_accept", u_accept, torch.float32), ("u_sample", u_sample, torch.float32),
                        ("accepted_len", out["accepted_len"], torch.int32), ("out_token", out["out_token"], torch.int32)):
        _cuda(t, name, dt)
    if draft_idx.numel() != B * gamma * k or draft_logit.numel() != B * gamma * k or \
            draft_count.numel() != B * gamma or draft_token.numel() != B * gamma or \
            u_accept.numel() != B * gamma or u_sample.numel() != B or \
            out["accepted_len"].numel() != B or out["out_token"].numel() != B:
        raise ValueError("draft / uniform / output shapes do not match target_logits")
    _check_verify_outputs(out, B, gamma)
    rc = lib().tslt_verify_static(_ptr(target_logits), _dtype_code(target_logits), B, gamma, V, stride, k,
                                  _ptr(draft_idx), _ptr(draft_logit), _ptr(draft_count), _ptr(draft_token),
                                  draft_temperature, target_temperature, _ptr(u_accept), _ptr(u_sample),
                                  _ptr(out["accepted_len"]), _ptr(out["out_token"]), _ptr(out.get("accept_prob")),
                                  _ptr(out.get("beta_hat")), _ptr(out.get("lse_p")), _stream())
    _check(rc, "tslt_verify_static")
    return out


def tree_verify_walk_workspace_bytes(B: int, N: int, V: int, k: int) -> int:
    n = ctypes.c_size_t(0)
    _check(lib().tslt_tree_verify_walk_workspace_bytes(B, N, V, k, ctypes.byref(n)),
           "tslt_tree_verify_walk_workspace_bytes")
    return int(n.value)


def tree_verify(target_logits: torch.Tensor, parent: Sequence[int], node_draft_row: Sequence[int],
                node_token: torch.Tensor, draft_idx: torch.Tensor, draft_logit: torch.Tensor,
                draft_count: torch.Tensor, draft_temperature: float, target_temperature: float,
                u_accept: torch.Tensor, u_sample: torch.Tensor, max_depth: int, *,
                out: Optional[dict] = None, ws: Optional[torch.Tensor] = None, walk: bool = False) -> dict:
    """tslt_tree_verify (walk=False: every node's row is streamed) or tslt_tree_verify_walk (walk=True:
    only the rows on each sequence's path).  target_logits [B, N, V]; parent / node_draft_row are host
    sequences [N]; drafts [B, M, k].  Returns dict(accepted_path [B, max_depth], accepted_len [B],
    out_token [B])."""
    if not target_logits.is_cuda:
        raise ValueError("target_logits must be a CUDA tensor (libtslt has no CPU path)")
    if target_logits.dim() != 3:
        raise ValueError("target_logits must be [B, N, V]")
    B, N, V = target_logits.shape
    _, _, stride = _row_layout(target_logits)
    par = np.ascontiguousarray(np.asarray(parent, dtype=np.int32))
    ndr = np.ascontiguousarray(np.asarray(node_draft_row, dtype=np.int32))
    if par.shape != (N,) or ndr.shape != (N,):
        raise ValueError("parent and node_draft_row must have N entries")
    M = int((ndr >= 0).sum())
    k = draft_idx.shape[-1] if M > 0 else 1
    dev = target_logits.device
    for name, t, dt in (("node_token", node_token, torch.int32), ("draft_idx", draft_idx, torch.int32),
                        ("draft_logit", draft_logit, torch.float32), ("draft_count", draft_count, torch.int32),
                        ("u_accept", u_accept, torch.float32), ("u_sample", u_sample, torch.float32)):
        _cuda(t, name, dt)
    if node_token.numel() != B * N or u_accept.numel() != B * N or u_sample.numel() != B * N or \
            draft_idx.numel() != B * M * k or draft_logit.numel() != B * M * k or draft_count.numel() != B * M:
        raise ValueError("tree tensors do not match target_logits / the tree shape")
    o = out if out is not None else {}
    if "accepted_len" not in o:
        o["accepted_path"] = torch.empty(B, max_depth, dtype=torch.int32, device=dev)
        o["accepted_len"] = torch.empty(B, dtype=torch.int32, device=dev)
        o["out_token"] = torch.empty(B, dtype=torch.int32, device=dev)
    for name, dt, ne in (("accepted_path", torch.int32, B * max_depth), ("accepted_len", torch.int32, B),
                         ("out_token", torch.int32, B)):
        _out(o, name, dt, ne)
    if ws is None:
        ws = workspace((tree_verify_walk_workspace_bytes if walk else tree_verify_workspace_bytes)(B, N, V, k), dev)
    entry = lib().tslt_tree_verify_walk if walk else lib().tslt_tree_verify
    rc = entry(_ptr(target_logits), _dtype_code(target_logits), B, N, V, stride,
                                par.ctypes.data_as(ctypes.c_void_p), ndr.ctypes.data_as(ctypes.c_void_p),
                                M, k, _ptr(node_token), _ptr(draft_idx), _ptr(draft_logit), _ptr(draft_count),
                                draft_temperature, target_temperature, _ptr(u_accept), _ptr(u_sample),
                                max_depth, _ptr(o["accepted_path"]), _ptr(o["accepted_len"]),
                                _ptr(o["out_token"]), _ptr(ws), ws.numel(), _stream())
    _check(rc, "tslt_tree_verify_walk" if walk else "tslt_tree_verify")
    o["workspace"] = ws
    return o


def verify_packed(target_logits: torch.Tensor, payload: torch.Tensor, prob_format: int, k: int,
                  draft_token: torch.Tensor, draft_temperature: float, target_temperature: float,
                  u_accept: torch.Tensor, u_sample: torch.Tensor, *, want_diag: bool = True,
                  out: Optional[dict] = None, ws: Optional[torch.Tensor] = None) -> dict:
    """tslt_verify_packed: tslt_verify on the uplink records themselves.  payload [B*gamma, words] int32
    as pack_payload writes it (words = payload_words(k, V, prob_format)[0]).  Returns what verify() returns."""
    if not target_logits.is_cuda:
        raise ValueError("target_logits must be a CUDA tensor (libtslt has no CPU path)")
    if target_logits.dim() != 3:
        raise ValueError("target_logits must be [B, gamma+1, V]")
    B, g1, V = target_logits.shape
    _, _, stride = _row_layout(target_logits)
    gamma = g1 - 1
    dev = target_logits.device
    words, _ = payload_words(k, V, prob_format)
    _cuda(payload, "payload", torch.int32)
    _cuda(draft_token, "draft_token", torch.int32)
    _cuda(u_accept, "u_accept", torch.float32)
    _cuda(u_sample, "u_sample", torch.float32)
    if payload.numel() != B * gamma * words or draft_token.numel() != B * gamma or \
            u_accept.numel() != B * gamma or u_sample.numel() != B:
        raise ValueError("payload / token / uniform shapes do not match target_logits")
    o = out if out is not None else {}
    if "accepted_len" not in o:
        o["accepted_len"] = torch.empty(B, dtype=torch.int32, device=dev)
        o["out_token"] = torch.empty(B, dtype=torch.int32, device=dev)
        if want_diag:
            o["accept_prob"] = torch.empty(B, gamma, dtype=torch.float32, device=dev)
            o["beta_hat"] = torch.empty(B, gamma, dtype=torch.float32, device=dev)
            o["lse_p"] = torch.empty(B, gamma + 1, dtype=torch.float32, device=dev)
    _check_verify_outputs(o, B, gamma)
    if ws is None:
        ws = workspace(verify_workspace_bytes(B, gamma, V, k), dev)
    rc = lib().tslt_verify_packed(_ptr(target_logits), _dtype_code(target_logits), B, gamma, V, stride, k,
                                  _ptr(payload), prob_format, _ptr(draft_token), draft_temperature, target_temperature,
                                  _ptr(u_accept), _ptr(u_sample), _ptr(o["accepted_len"]), _ptr(o["out_token"]),
                                  _ptr(o.get("accept_prob")), _ptr(o.get("beta_hat")), _ptr(o.get("lse_p")), _ptr(ws),
                                  ws.numel(), _stream())
    _check(rc, "tslt_verify_packed")
    o["workspace"] = ws
    return o


def tree_verify_packed(target_logits: torch.Tensor, parent: Sequence[int], node_draft_row: Sequence[int],
                       node_token: torch.Tensor, payload: torch.Tensor, prob_format: int, k: int,
                       draft_temperature: float, target_temperature: float, u_accept: torch.Tensor,
                       u_sample: torch.Tensor, max_depth: int, *, out: Optional[dict] = None,
                       ws: Optional[torch.Tensor] = None, walk: bool = False) -> dict:
    """tslt_tree_verify_packed: tree_verify() with the drafts as uplink records, payload [B*M, words]."""
    if not target_logits.is_cuda:
        raise ValueError("target_logits must be a CUDA tensor (libtslt has no CPU path)")
    if target_logits.dim() != 3:
        raise ValueError("target_logits must be [B, N, V]")
    B, N, V = target_logits.shape
    _, _, stride = _row_layout(target_logits)
    par = np.ascontiguousarray(np.asarray(parent, dtype=np.int32))
    ndr = np.ascontiguousarray(np.asarray(node_draft_row, dtype=np.int32))
    if par.shape != (N,) or ndr.shape != (N,):
        raise ValueError("parent and node_draft_row must have N entries")
    M = int((ndr >= 0).sum())
    dev = target_logits.device
    words, _ = payload_words(k, V, prob_format)
    for name, t, dt in (("node_token", node_token, torch.int32), ("payload", payload, torch.int32),
                        ("u_accept", u_accept, torch.float32), ("u_sample", u_sample, torch.float32)):
        _cuda(t, name, dt)
    if node_token.numel() != B * N or u_accept.numel() != B * N or u_sample.numel() != B * N or \
            payload.numel() != B * M * words:
        raise ValueError("tree tensors do not match target_logits / the tree shape")
    o = out if out is not None else {}
    if "accepted_len" not in o:
        o["accepted_path"] = torch.empty(B, max_depth, dtype=torch.int32, device=dev)
        o["accepted_len"] = torch.empty(B, dtype=torch.int32, device=dev)
        o["out_token"] = torch.empty(B, dtype=torch.int32, device=dev)
    for name, dt, ne in (("accepted_path", torch.int32, B * max_depth), ("accepted_len", torch.int32, B),
                         ("out_token", torch.int32, B)):
        _out(o, name, dt, ne)
    if ws is None:
        ws = workspace((tree_verify_walk_workspace_bytes if walk else tree_verify_workspace_bytes)(B, N, V, k), dev)
    rc = lib().tslt_tree_verify_packed(1 if walk else 0, _ptr(target_logits), _dtype_code(target_logits), B, N, V, stride,
                                       par.ctypes.data_as(ctypes.c_void_p), ndr.ctypes.data_as(ctypes.c_void_p), M, k,
                                       _ptr(node_token), _ptr(payload), prob_format, draft_temperature,
                                       target_temperature, _ptr(u_accept), _ptr(u_sample), max_depth,
                                       _ptr(o["accepted_path"]), _ptr(o["accepted_len"]), _ptr(o["out_token"]), _ptr(ws),
                                       ws.numel(), _stream())
    _check(rc, "tslt_tree_verify_packed")
    o["workspace"] = ws
    return o


def payload_words(k: int, V: int, prob_format: int):
    """(32-bit words per row record, bits per entry) of the uplink payload."""
    w, b = ctypes.c_int(0), ctypes.c_int(0)
    _check(lib().tslt_payload_words(k, V, prob_format, ctypes.byref(w), ctypes.byref(b)), "tslt_payload_words")
    return int(w.value), int(b.value)


def pack_payload(idx: torch.Tensor, logit: torch.Tensor, count: torch.Tensor, V: int, prob_format: int) -> dict:
    """tslt_pack_payload on the output of sparsify: idx / logit [rows, k], count [rows].
    Returns dict(payload [rows, words] int32 (bit patterns), bits [rows] int64)."""
    _cuda(idx, "idx", torch.int32); _cuda(logit, "logit", torch.float32); _cuda(count, "count", torch.int32)
    k = idx.shape[-1]
    rows = count.numel()
    if idx.numel() != rows * k or logit.numel() != rows * k:
        raise ValueError("idx / logit / count shapes do not match")
    words, _ = payload_words(k, V, prob_format)
    payload = torch.empty(rows, words, dtype=torch.int32, device=idx.device)
    bits = torch.empty(rows, dtype=torch.int64, device=idx.device)
    _check(lib().tslt_pack_payload(_ptr(idx), _ptr(logit), _ptr(count), rows, k, V, prob_format, _ptr(payload),
                                   _ptr(bits), _stream()), "tslt_pack_payload")
    return {"payload": payload, "bits": bits}


def unpack_payload(payload: torch.Tensor, k: int, V: int, prob_format: int, *, out: Optional[dict] = None) -> dict:
    """tslt_unpack_payload: records [rows, words] -> dict(idx, logit [rows, k], count [rows], flag [1])
    in the form verify / tree_verify take.  `out` reuses buffers of an earlier call (its flag is sticky)."""
    _cuda(payload, "payload", torch.int32)
    words, _ = payload_words(k, V, prob_format)
    if payload.dim() != 2 or payload.shape[1] != words:
        raise ValueError("payload must be [rows, %d] for this k, V and format" % words)
    rows = payload.shape[0]
    dev = payload.device
    o = out if out is not None else {
        "idx": torch.empty(rows, k, dtype=torch.int32, device=dev),
        "logit": torch.empty(rows, k, dtype=torch.float32, device=dev),
        "count": torch.empty(rows, dtype=torch.int32, device=dev),
        "flag": torch.zeros(1, dtype=torch.int32, device=dev)}
    for name, dt, ne in (("idx", torch.int32, rows * k), ("logit", torch.float32, rows * k), ("count", torch.int32, rows),
                         ("flag", torch.int32, 1)):
        _out(o, name, dt, ne)
    _check(lib().tslt_unpack_payload(_ptr(payload), rows, k, V, prob_format, _ptr(o["idx"]), _ptr(o["logit"]),
                                     _ptr(o["count"]), _ptr(o["flag"]), _stream()), "tslt_unpack_payload")
    return o


def diagnostics(draft_logits: torch.Tensor, target_logits: torch.Tensor, k_list: Sequence[int], num_candidates: int,
                draft_temperature: float = 1.0, target_temperature: float = 1.0) -> dict:
    """tslt_diagnostics on paired rows [rows, V]: dict(beta_j, z_j [rows, c], theta [rows], rho, theta_hat
    [rows, n_k], beta_hat_j [rows, n_k, c]), all fp32."""
    if not draft_logits.is_cuda or not target_logits.is_cuda:
        raise ValueError("logits must be CUDA tensors (libtslt has no CPU path)")
    if draft_logits.shape != target_logits.shape or draft_logits.dtype != target_logits.dtype:
        raise ValueError("draft and target logits must have the same shape and dtype")
    rows, V, stride = _row_layout(draft_logits)
    rows2, _, stride2 = _row_layout(target_logits)
    if stride != stride2 or rows != rows2:
        raise ValueError("draft and target logits must have the same row layout")
    ks = np.ascontiguousarray(np.asarray(list(k_list), dtype=np.int32))
    nk, c, dev = int(ks.size), int(num_candidates), draft_logits.device
    o = {"beta_j": torch.empty(rows, c, device=dev), "z_j": torch.empty(rows, c, device=dev),
         "theta": torch.empty(rows, device=dev), "rho": torch.empty(rows, nk, device=dev),
         "beta_hat_j": torch.empty(rows, nk, c, device=dev), "theta_hat": torch.empty(rows, nk, device=dev)}
    n = ctypes.c_size_t(0)
    _check(lib().tslt_diagnostics_workspace_bytes(rows, V, int(ks.max()) if nk else 1, c, ctypes.byref(n)),
           "tslt_diagnostics_workspace_bytes")
    ws = torch.empty(max(int(n.value), 256), dtype=torch.uint8, device=dev)
    rc = lib().tslt_diagnostics(_ptr(draft_logits), _ptr(target_logits), _dtype_code(draft_logits), rows, V, stride,
                                ks.ctypes.data_as(ctypes.c_void_p), nk, c, draft_temperature, target_temperature,
                                _ptr(o["beta_j"]), _ptr(o["z_j"]), _ptr(o["theta"]), _ptr(o["rho"]), _ptr(o["beta_hat_j"]),
                                _ptr(o["theta_hat"]), _ptr(ws), ws.numel(), _stream())
    _check(rc, "tslt_diagnostics")
    o["workspace"] = ws
    return o
