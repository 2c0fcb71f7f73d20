"""tslt_sparsify over a vocabulary that is split across ranks (tensor-parallel output projection): the
one place on this path with an exchange step.

Every rank holds the same rows and its own slice [vocab_start, vocab_start + V_local) of the vocabulary.
Each runs tslt_sparsify_shard on its slice; the parts (k pairs, a count and a log-normaliser per row:
8 k + 12 bytes) are all-gathered; tslt_sparsify_merge then gives, on every rank, exactly what
tslt_sparsify gives on the whole rows.  No logits cross the link.  The collective is torch.distributed's
all_gather (NCCL over NVLink for CUDA tensors); the compute steps are the library's kernels.

The two compute steps can be replaced (shard_fn, merge_fn): the CPU test of this module's plumbing
(rank order, offsets, layout of the gathered parts) runs it under gloo with stand-ins, since the
kernels themselves need a GPU.
"""
from __future__ import annotations

from typing import Callable, Optional

import torch
import torch.distributed as dist


def _default_shard(local_logits, k, temperature):
    from . import tslt
    o = tslt.sparsify_shard(local_logits, k, temperature)
    return {n: o[n] for n in ("idx", "logit", "count", "lse2")}


def _default_merge(parts, offsets, dtype, top_p, temperature, uniforms):
    from . import tslt
    return tslt.sparsify_merge(parts["idx"], parts["logit"], parts["count"], parts["lse2"], offsets, dtype, top_p,
                               temperature, uniforms)


def sparsify_vocab_parallel(local_logits: torch.Tensor, vocab_start: int, k: int, top_p: float = 1.0,
                            temperature: float = 1.0, uniforms: Optional[torch.Tensor] = None, *, group=None,
                            shard_fn: Callable = _default_shard, merge_fn: Callable = _default_merge) -> dict:
    """local_logits [rows, V_local]: this rank's slice, starting at token id vocab_start.  Slices must
    not overlap and must ascend with the rank (rank r's slice ends where rank r + 1's begins, or
    before).  uniforms [rows, num_samples] must be the same on every rank.  Returns what sparsify()
    returns for the whole rows, on every rank."""
    if not dist.is_initialized():
        raise RuntimeError("torch.distributed is not initialised")
    world = dist.get_world_size(group)
    if world > 16:
        raise ValueError("at most 16 vocabulary shards")
    part = shard_fn(local_logits, k, temperature)
    rows = local_logits.shape[0]
    gathered = {}
    for name, t in part.items():
        t = t.contiguous()
        bufs = [torch.empty_like(t) for _ in range(world)]
        dist.all_gather(bufs, t, group=group)
        gathered[name] = torch.stack(bufs, 0)  # [world, rows, ...] in rank order = vocabulary order
    span = torch.tensor([int(vocab_start), int(vocab_start) + int(local_logits.shape[1])], dtype=torch.int64,
                        device=local_logits.device)
    spans = [torch.empty_like(span) for _ in range(world)]
    dist.all_gather(spans, span, group=group)
    spans = [tuple(int(x) for x in s.tolist()) for s in spans]
    for (a0, a1), (b0, _) in zip(spans, spans[1:]):
        if b0 < a1:
            raise ValueError("vocabulary slices must ascend with the rank and must not overlap: %s" % (spans,))
    assert gathered["idx"].shape[:2] == (world, rows)
    return merge_fn(gathered, [s[0] for s in spans], local_logits.dtype, top_p, temperature, uniforms)
