"""CPU oracle of the uplink payload: the sparse (token index, logit) pairs of a row written with
b_idx bits per index and b_prob bits per value.

TEST INFRASTRUCTURE ONLY: imported by tests/ (and nothing in the product package).  Plain numpy and
Python loops, one bit at a time where that is the clearest statement.

What the paper fixes (Section 2.2, the equations for D_up and D_V): a transmitted distribution
costs (number of entries) * (b_prob + b_idx) bits, b_prob = 32 for full precision or 16 for half
precision, b_idx = ceil(log2 |V|) for binary-coded indices.  Section 3 (Solution 1) fixes what is
sent: the selected logits and their token ids.  The paper fixes no wire layout; the layout below is
this library's (stated in the header of the C ABI as well):

  a row's record is `words` 32-bit little-endian words; word 0 is the number of entries n; the
  entries follow as one bit stream, entry e in bits [e*w, (e+1)*w) of the stream, w = b_idx +
  b_prob, bit i of the stream being bit (i mod 32) of word 1 + i // 32; inside an entry the low
  b_idx bits are the index and the next b_prob bits the value's bit pattern (fp32, bf16 or IEEE
  half, rounded to nearest even from the fp32 logit).  Bits past the last entry are zero.
"""
from __future__ import annotations

import math

import numpy as np

PROB_F32, PROB_BF16, PROB_F16 = 0, 1, 2


def index_bits(V: int) -> int:
    """b_idx = ceil(log2 |V|) (Section 2.2), by counting: the smallest b with 2**b >= V."""
    b = 0
    while (1 << b) < V:
        b += 1
    return b


def prob_bits(fmt: int) -> int:
    return 32 if fmt == PROB_F32 else 16


def entry_bits(V: int, fmt: int) -> int:
    return index_bits(V) + prob_bits(fmt)


def words_per_row(k: int, V: int, fmt: int) -> int:
    return 1 + (k * entry_bits(V, fmt) + 31) // 32


def payload_bits(count, V: int, fmt: int):
    """D for one transmitted row: n * (b_prob + b_idx) (the paper's D_V with |V| replaced by the
    n retained entries; the record's count word is not part of the paper's formula)."""
    return np.asarray(count, dtype=np.int64) * entry_bits(V, fmt)


def round_value(x: np.ndarray, fmt: int) -> np.ndarray:
    """fp32 logits as the receiver sees them after the wire format (fp32 array)."""
    x = np.asarray(x, dtype=np.float32)
    if fmt == PROB_F32:
        return x.copy()
    if fmt == PROB_F16:
        with np.errstate(over="ignore"):
            return x.astype(np.float16).astype(np.float32)
    return _bf16_bits_to_f32(_f32_to_bf16_bits(x))


def _f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round to nearest, ties to even, on the upper 16 bits; inf stays inf."""
    u = np.asarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    out = np.empty(u.shape, dtype=np.uint16)
    flat_u, flat_o = u.reshape(-1), out.reshape(-1)
    for i in range(flat_u.size):
        v = int(flat_u[i])
        exp_all_ones = (v & 0x7F800000) == 0x7F800000
        if exp_all_ones:  # inf or NaN: truncate (keep NaN a NaN)
            hi = v >> 16
            if (v & 0x007FFFFF) and not (hi & 0x7F):
                hi |= 1
        else:
            low, hi = v & 0xFFFF, v >> 16
            if low > 0x8000 or (low == 0x8000 and (hi & 1)):
                hi += 1
        flat_o[i] = hi & 0xFFFF
    return out


def _bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.asarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def value_pattern(x: float, fmt: int) -> int:
    """Bit pattern of one value on the wire."""
    a = np.array([x], dtype=np.float32)
    if fmt == PROB_F32:
        return int(a.view(np.uint32)[0])
    if fmt == PROB_F16:
        with np.errstate(over="ignore"):
            return int(a.astype(np.float16).view(np.uint16)[0])
    return int(_f32_to_bf16_bits(a)[0])


def pattern_value(p: int, fmt: int) -> float:
    if fmt == PROB_F32:
        return float(np.array([p], dtype=np.uint32).view(np.float32)[0])
    if fmt == PROB_F16:
        return float(np.array([p], dtype=np.uint16).view(np.float16).astype(np.float32)[0])
    return float(_bf16_bits_to_f32(np.array([p], dtype=np.uint16))[0])


def pack(idx: np.ndarray, logit: np.ndarray, count: np.ndarray, V: int, fmt: int) -> np.ndarray:
    """[rows, k] int32 indices / fp32 logits / [rows] counts -> [rows, words] uint32 records."""
    idx = np.asarray(idx)
    logit = np.asarray(logit, dtype=np.float32)
    rows, k = idx.shape
    bi, bp = index_bits(V), prob_bits(fmt)
    W = words_per_row(k, V, fmt)
    out = np.zeros((rows, W), dtype=np.uint32)
    for r in range(rows):
        n = int(count[r])
        words = [0] * W
        words[0] = n
        pos = 0
        for e in range(n):
            entry = int(idx[r, e]) | (value_pattern(float(logit[r, e]), fmt) << bi)
            for b in range(bi + bp):  # one bit at a time
                if (entry >> b) & 1:
                    words[1 + pos // 32] |= 1 << (pos % 32)
                pos += 1
        out[r] = np.array(words, dtype=np.uint64).astype(np.uint32)
    return out


def unpack(payload: np.ndarray, k: int, V: int, fmt: int):
    """[rows, words] uint32 -> (idx [rows, k] int32 padded with -1, logit [rows, k] fp32 padded
    with -inf, count [rows] int32)."""
    payload = np.asarray(payload, dtype=np.uint32)
    rows = payload.shape[0]
    bi, bp = index_bits(V), prob_bits(fmt)
    idx = np.full((rows, k), -1, dtype=np.int32)
    logit = np.full((rows, k), -np.inf, dtype=np.float32)
    count = np.zeros(rows, dtype=np.int32)
    for r in range(rows):
        n = int(payload[r, 0])
        count[r] = n
        pos = 0
        for e in range(n):
            entry = 0
            for b in range(bi + bp):
                bit = (int(payload[r, 1 + pos // 32]) >> (pos % 32)) & 1
                entry |= bit << b
                pos += 1
            idx[r, e] = entry & ((1 << bi) - 1)
            logit[r, e] = pattern_value(entry >> bi, fmt)
    return idx, logit, count


def full_distribution_bits(V: int, fmt: int, with_index: bool = True) -> int:
    """D_V of Section 2.2 for an untruncated distribution: |V| * (b_prob + b_idx); a dense vector
    needs no indices (with_index False), which is the figure the paper's experiments quote."""
    return V * (prob_bits(fmt) + (index_bits(V) if with_index else 0))


def log2_ceil_closed_form(V: int) -> int:
    """ceil(log2 V) through floating point, for the pin against index_bits."""
    return int(math.ceil(math.log2(V))) if V > 1 else 0
