"""Seeded synthetic inputs for the TSLT hot path.

This module serves both the CUDA path and the CPU oracle and therefore holds none of
the method's arithmetic: it only draws logits, uniforms and tree shapes.  Everything is
a pure function of (seed, tensor id, shape), built from torch ops that run on either
device, so a test can draw on the CPU and copy to the GPU while a full-size benchmark
draws directly in HBM and copies sampled rows back for the oracle.

Recipe (stands in for the draft / target language-model logits of the paper's
experiments, Section 5, whose weights and prompts are not available):

* draft logits  z_q = g + b,  g ~ N(0,1) per entry,  b_v = -1.1 * ln(rank_v) with the
  ranks 1..V randomly permuted per row (a Zipf(1.1) bias);
* target logits z_p = z_q (unrounded fp32) + N(0, sigma_t^2); rows that verify nothing
  (the bonus row, tree leaves) are fresh draws of the draft law;
* both are then rounded to the storage dtype (bf16: round-to-nearest-even);
* uniforms are fp32 U[0,1), one per sampling or acceptance decision.
"""
from __future__ import annotations

from typing import List, Sequence, Tuple

import torch

ZIPF_EXPONENT = 1.1

# Tensor ids mixed into the seed so that every tensor of a workload is an independent stream.
TID_DRAFT = 1
TID_TARGET_NOISE = 2
TID_TARGET_FRESH = 3
TID_U_DRAFT = 4
TID_U_ACCEPT = 5
TID_U_SAMPLE = 6


def _gen(seed: int, tensor_id: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed((int(seed) * 1_000_003 + int(tensor_id) * 7_919 + 12_345) & 0x7FFF_FFFF_FFFF)
    return g


def _zipf_rows(rows: int, V: int, gen: torch.Generator, device, chunk_rows: int = 64) -> torch.Tensor:
    """[rows, V] fp32: N(0,1) noise plus a per-row randomly permuted Zipf bias."""
    out = torch.empty(rows, V, dtype=torch.float32, device=device)
    for r0 in range(0, rows, chunk_rows):
        r1 = min(rows, r0 + chunk_rows)
        n = r1 - r0
        rank = torch.rand(n, V, generator=gen, device=device).argsort(dim=-1)
        bias = (rank + 1).to(torch.float32).log_().mul_(-ZIPF_EXPONENT)
        del rank
        g = torch.randn(n, V, generator=gen, device=device, dtype=torch.float32)
        out[r0:r1] = g.add_(bias)
    return out


def uniforms(shape: Sequence[int], seed: int, tensor_id: int, device="cpu") -> torch.Tensor:
    """fp32 U[0,1) of the given shape (torch.rand never returns 1.0)."""
    return torch.rand(*shape, generator=_gen(seed, tensor_id, device), device=device,
                      dtype=torch.float32)


def draft_rows(rows: int, V: int, dtype: torch.dtype, seed: int, device="cpu") -> torch.Tensor:
    """Draft logits [rows, V] alone (the rows sequence_logits would draw as its draft)."""
    return _zipf_rows(rows, V, _gen(seed, TID_DRAFT, device), device).to(dtype).contiguous()


def sequence_logits(B: int, gamma: int, V: int, dtype: torch.dtype, sigma_t: float,
                    seed: int, device="cpu") -> Tuple[torch.Tensor, torch.Tensor]:
    """Draft logits [B, gamma, V] and target logits [B, gamma+1, V] for single-candidate TSLT.

    Target row j (j < gamma) is draft row j plus N(0, sigma_t^2); row gamma is a fresh draw.
    """
    zq32 = _zipf_rows(B * gamma, V, _gen(seed, TID_DRAFT, device), device).view(B, gamma, V)
    zp = torch.empty(B, gamma + 1, V, dtype=dtype, device=device)
    gn = _gen(seed, TID_TARGET_NOISE, device)
    for b in range(B):
        noise = torch.randn(gamma, V, generator=gn, device=device, dtype=torch.float32)
        zp[b, :gamma] = (zq32[b] + noise.mul_(sigma_t)).to(dtype)
    fresh = _zipf_rows(B, V, _gen(seed, TID_TARGET_FRESH, device), device)
    zp[:, gamma] = fresh.to(dtype)
    del fresh
    zq = zq32.to(dtype)
    return zq.contiguous(), zp.contiguous()


def complete_tree(expansion: Sequence[int]) -> Tuple[List[int], List[int], int, int]:
    """Parent array of a complete token tree with expansion configuration <k_1..k_L>.

    Nodes are numbered in breadth-first order, node 0 being the root (the prefix); the
    children of a node are consecutive and ascending.  Returns (parent, node_draft_row, M,
    depth): node_draft_row[n] is the index of node n among the internal nodes (those that
    carry a draft distribution) or -1 for a leaf; M is the number of internal nodes.
    """
    parent = [-1]
    level = [0]
    for k in expansion:
        nxt = []
        for p in level:
            for _ in range(int(k)):
                parent.append(p)
                nxt.append(len(parent) - 1)
        level = nxt
    N = len(parent)
    has_child = [False] * N
    for c in range(1, N):
        has_child[parent[c]] = True
    node_draft_row, M = [], 0
    for n in range(N):
        if has_child[n]:
            node_draft_row.append(M)
            M += 1
        else:
            node_draft_row.append(-1)
    return parent, node_draft_row, M, len(expansion)


def tree_logits(B: int, parent: Sequence[int], node_draft_row: Sequence[int], V: int,
                dtype: torch.dtype, sigma_t: float, seed: int, device="cpu"
                ) -> Tuple[torch.Tensor, torch.Tensor]:
    """Draft logits [B, M, V] (internal nodes) and target logits [B, N, V] (all nodes).

    The target row of an internal node is its draft row plus N(0, sigma_t^2); the target
    row of a leaf is a fresh draw of the draft law.
    """
    N = len(parent)
    M = sum(1 for r in node_draft_row if r >= 0)
    zq32 = _zipf_rows(B * M, V, _gen(seed, TID_DRAFT, device), device).view(B, M, V)
    zp = torch.empty(B, N, V, dtype=dtype, device=device)
    gn = _gen(seed, TID_TARGET_NOISE, device)
    gf = _gen(seed, TID_TARGET_FRESH, device)
    internal = [n for n in range(N) if node_draft_row[n] >= 0]
    leaves = [n for n in range(N) if node_draft_row[n] < 0]
    for b in range(B):
        noise = torch.randn(M, V, generator=gn, device=device, dtype=torch.float32)
        rows = (zq32[b] + noise.mul_(sigma_t)).to(dtype)
        for n in internal:
            zp[b, n] = rows[node_draft_row[n]]
        if leaves:
            fresh = _zipf_rows(len(leaves), V, gf, device).to(dtype)
            for i, n in enumerate(leaves):
                zp[b, n] = fresh[i]
    return zq32.to(dtype).contiguous(), zp.contiguous()


# The workloads named by the benchmark definition (index = config number).
CONFIGS = [
    dict(name="cfg0_sc_B1_g4_V32000_f32_k64", kind="sequence", B=1, gamma=4, V=32000,
         dtype="f32", k=64, top_p=1.0, temperature=1.0, sigma_t=0.5),
    dict(name="cfg1_sc_B8_g8_V32000_bf16_p0.9", kind="sequence", B=8, gamma=8, V=32000,
         dtype="bf16", k=256, top_p=0.9, temperature=0.8, sigma_t=0.5),
    dict(name="cfg2_sc_B32_g5_V128256_bf16_k128", kind="sequence", B=32, gamma=5, V=128256,
         dtype="bf16", k=128, top_p=1.0, temperature=1.0, sigma_t=0.3),
    dict(name="cfg3_tree_B16_333_V151936_bf16_k64", kind="tree", B=16, expansion=(3, 3, 3),
         V=151936, dtype="bf16", k=64, top_p=1.0, temperature=1.0, sigma_t=0.5),
    dict(name="cfg4_sweep_B256_g8_V256000_bf16", kind="sequence", B=256, gamma=8, V=256000,
         dtype="bf16", k=64, top_p=1.0, temperature=1.0, sigma_t=0.5,
         sweep=[(16, 1.0), (64, 1.0), (256, 1.0), (1024, 1.0), (1024, 0.95)]),
]


def torch_dtype(name: str) -> torch.dtype:
    return {"f32": torch.float32, "bf16": torch.bfloat16}[name]
