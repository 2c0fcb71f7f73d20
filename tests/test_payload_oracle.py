"""Pins for the payload oracle (oracle/payload.py): bit widths and sizes against the paper's
formula and printed figure (Section 2.2, Section 5), the layout against a hand-worked record and
against an independent big-integer construction, the 16-bit roundings against torch's."""
import os

import numpy as np
import pytest
import torch

from oracle import payload as P

HERE = os.path.dirname(os.path.abspath(__file__))


def golden(name):
    vals = {}
    with open(os.path.join(HERE, "golden", name)) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if "=" in line:
                k, v = line.split("=", 1)
                vals[k.strip()] = v.strip()
    return vals


def test_index_bits_is_ceil_log2():
    g = golden("paper_values.txt")
    assert P.index_bits(32000) == int(g["index_bits_V32000"]) == 15
    for V, want in ((2, 1), (3, 2), (4, 2), (5, 3), (32768, 15), (32769, 16), (128256, 17), (151936, 18), (256000, 18)):
        assert P.index_bits(V) == want == (V - 1).bit_length() == P.log2_ceil_closed_form(V)
    assert P.index_bits(1) == 0


def test_sizes_follow_the_papers_formula():
    g = golden("paper_values.txt")
    # Section 5: 32K vocabulary at FP16 is "0.5 Mbit" per distribution (a dense vector, no indices)
    dense = P.full_distribution_bits(32000, P.PROB_F16, with_index=False)
    assert dense == int(g["payload_bits_full_V32000_fp16_prob_only"])
    assert abs(dense - 0.5e6) / 0.5e6 < 0.03
    # Section 2.2: D_V = |V| (b_prob + b_idx)
    assert P.full_distribution_bits(32000, P.PROB_F16) == 32000 * 31
    assert P.full_distribution_bits(32000, P.PROB_F32) == 32000 * 47
    # truncated: the retained entries in place of |V|
    assert int(P.payload_bits(320, 32000, P.PROB_F16)) == int(g["tslt_payload_bits_V32000_K320_fp16"])
    assert int(P.payload_bits(32, 32000, P.PROB_BF16)) == int(g["tslt_payload_bits_V32000_K32_fp16"])
    assert list(P.payload_bits(np.array([0, 1, 64]), 256000, P.PROB_F32)) == [0, 50, 3200]
    assert P.words_per_row(64, 256000, P.PROB_BF16) == 1 + (64 * 34 + 31) // 32
    assert P.words_per_row(1, 2, P.PROB_BF16) == 2


def test_hand_worked_record():
    g = golden("payload_example.txt")
    V, k = int(g["V"]), int(g["k"])
    idx = np.full((1, k), -1, np.int32)
    logit = np.full((1, k), -np.inf, np.float32)
    ii = [int(x) for x in g["idx"].split(",")]
    ll = [float(x) for x in g["logit"].split(",")]
    idx[0, :len(ii)] = ii
    logit[0, :len(ll)] = ll
    want = [int(x, 16) for x in g["words"].split(",")]
    got = P.pack(idx, logit, np.array([len(ii)], np.int32), V, P.PROB_BF16)
    assert got.shape == (1, len(want))
    assert [int(x) for x in got[0]] == want
    i2, l2, c2 = P.unpack(np.array([want], dtype=np.uint32), k, V, P.PROB_BF16)
    assert c2[0] == len(ii) and list(i2[0]) == ii + [-1] and list(l2[0][:2]) == ll and l2[0][2] == -np.inf


def big_integer_record(idx, logit_patterns, bi, bp, words):
    """The same record built as one big integer: sum of entry_e << (e * w), cut into words."""
    stream = 0
    for e, (i, pat) in enumerate(zip(idx, logit_patterns)):
        stream |= (i | (pat << bi)) << (e * (bi + bp))
    out = [len(idx)]
    for w in range(words - 1):
        out.append((stream >> (32 * w)) & 0xFFFFFFFF)
    return out


@pytest.mark.parametrize("fmt", [P.PROB_F32, P.PROB_BF16, P.PROB_F16])
@pytest.mark.parametrize("V", [2, 1000, 32000, 256000])
def test_layout_against_big_integer_and_round_trip(V, fmt):
    rng = np.random.default_rng(V + fmt)
    k, rows = 37, 6
    idx = np.full((rows, k), -1, np.int32)
    logit = np.full((rows, k), -np.inf, np.float32)
    count = np.array([0, 1, 5, 36, 37, 17], np.int32)
    for r in range(rows):
        n = int(count[r])
        idx[r, :n] = np.sort(rng.choice(V, size=min(n, V), replace=False))[:n] if n <= V else np.arange(n) % V
        logit[r, :n] = (rng.standard_normal(n) * 6).astype(np.float32)
    if rows > 3:
        logit[3, 0] = -np.inf
        logit[3, 1] = 65520.0 if fmt == P.PROB_F16 else 3.0e38  # rounds to inf in half precision
    rec = P.pack(idx, logit, count, V, fmt)
    W = P.words_per_row(k, V, fmt)
    assert rec.shape == (rows, W)
    bi, bp = P.index_bits(V), P.prob_bits(fmt)
    for r in range(rows):
        n = int(count[r])
        pats = [P.value_pattern(float(x), fmt) for x in logit[r, :n]]
        assert [int(x) for x in rec[r]] == big_integer_record([int(x) for x in idx[r, :n]], pats, bi, bp, W)
    i2, l2, c2 = P.unpack(rec, k, V, fmt)
    assert (c2 == count).all() and (i2 == idx).all()
    want = np.where(np.arange(k)[None, :] < count[:, None], P.round_value(logit, fmt), -np.inf).astype(np.float32)
    assert l2.tobytes() == want.tobytes()


def test_roundings_match_torch():
    rng = np.random.default_rng(7)
    x = np.concatenate([
        (rng.standard_normal(4000) * 10).astype(np.float32),
        np.array([0.0, -0.0, 1.0, -1.0, np.inf, -np.inf, 1e-40, -1e-40, 3.3895314e38, 65504.0, 65519.9, 65520.0, 1e-8],
                 np.float32),
        # exact ties of the bf16 rounding: low half = 0x8000 with even and odd upper halves
        np.array([0x3F808000, 0x3F818000, 0xC0008000, 0xC0018000, 0x7F7F8000], np.uint32).view(np.float32),
        # exact ties of the half rounding (13 dropped bits = 0x1000)
        np.array([0x3F801000, 0x3F803000, 0xBF801000], np.uint32).view(np.float32)])
    t = torch.from_numpy(x)
    assert P.round_value(x, P.PROB_BF16).tobytes() == t.to(torch.bfloat16).to(torch.float32).numpy().tobytes()
    assert P.round_value(x, P.PROB_F16).tobytes() == t.to(torch.float16).to(torch.float32).numpy().tobytes()
    assert P.round_value(x, P.PROB_F32).tobytes() == x.tobytes()
    # bf16 payload of logits that came from bf16 storage is lossless
    z = t.to(torch.bfloat16).to(torch.float32).numpy()
    assert P.round_value(z, P.PROB_BF16).tobytes() == z.tobytes()
