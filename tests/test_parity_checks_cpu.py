"""The parity bar itself, exercised on the CPU: the comparison helpers accept the oracle's own
outputs, accept a token on the other side of a flagged boundary, and reject everything else
(a wrong token on an unflagged row, an invalid token on a flagged one, an accepted length that
no uniform within the band explains).  The mistakes are planted in copies of the ORACLE's
outputs; no GPU is involved."""
import numpy as np
import pytest
import torch

import oracle
from paper_2512_16273_b200 import synth
from parity_utils import (BAND, compare_sparsify, compare_tree, compare_verify, token_is_valid, verify_inputs)


def test_token_validity_band():
    w = np.array([0.1, 0.0, 0.4, 0.5])
    assert token_is_valid(w, 0.05, 0) and not token_is_valid(w, 0.05, 2)
    assert not token_is_valid(w, 0.3, 1)                      # zero mass is never valid
    assert token_is_valid(w, 0.1 + 0.5 * BAND, 0) and token_is_valid(w, 0.1 - 0.5 * BAND, 2)
    assert not token_is_valid(w, 0.1 + 3 * BAND, 0)
    assert token_is_valid(w, 1.5, 3)                          # u >= 1 is clamped, the last item takes it


def small_round(seed=3, B=4, gamma=3, V=300, k=16, top_p=1.0, T=0.9):
    zq, zp = synth.sequence_logits(B, gamma, V, torch.float32, 0.5, seed, "cpu")
    ud = synth.uniforms((B * gamma, 2), seed, synth.TID_U_DRAFT)
    ua = synth.uniforms((B, gamma), seed, synth.TID_U_ACCEPT)
    us = synth.uniforms((B,), seed, synth.TID_U_SAMPLE)
    ref_s = oracle.sparsify(zq.reshape(-1, V), k, top_p, T, ud.numpy())
    tok = ref_s["token"][:, 0].reshape(B, gamma)
    inp = verify_inputs(zp, ref_s, B, gamma, k, tok, T, T, ua, us)
    ref_v = oracle.verify(zp, inp["idx"], inp["logit"], inp["count"], inp["token"], T, T, inp["ua"], inp["us"])
    return zq.reshape(-1, V), ud, ref_s, inp, ref_v, T


def as_gpu(ref, names):
    return {n: torch.from_numpy(np.array(ref[n], copy=True).astype(np.float32 if ref[n].dtype == np.float64 else ref[n].dtype))
            for n in names}


def test_sparsify_compare_accepts_oracle_and_rejects_planted_mistakes():
    z, ud, ref_s, _, _, T = small_round()
    names = ("idx", "logit", "count", "token", "lse", "mass")
    compare_sparsify(as_gpu(ref_s, names), ref_s, logits=z, uniforms=ud, T=T)
    bad = as_gpu(ref_s, names); bad["token"][1, 0] = bad["idx"][1, 0] if bad["token"][1, 0] != bad["idx"][1, 0] else bad["idx"][1, 1]
    with pytest.raises(AssertionError):
        compare_sparsify(bad, ref_s, logits=z, uniforms=ud, T=T)
    bad = as_gpu(ref_s, names); bad["idx"][2, 3] += 1
    with pytest.raises(AssertionError):
        compare_sparsify(bad, ref_s, logits=z, uniforms=ud, T=T)
    bad = as_gpu(ref_s, names); bad["mass"][0] *= 1.0 + 1e-4
    with pytest.raises(AssertionError):
        compare_sparsify(bad, ref_s, logits=z, uniforms=ud, T=T)


def test_sparsify_flagged_sample_accepts_only_the_neighbour():
    """A uniform placed on a CDF step: the oracle flags the row; the token on the other side of the
    step passes, any other token does not."""
    z, ud, ref_s, _, _, T = small_round()
    r, n = 0, int(ref_s["count"][0])
    y = ref_s["logit"][r, :n].astype(np.float64) / T
    cdf = np.cumsum(np.exp(y - y.max())); cdf /= cdf[-1]
    u2 = ud.numpy().copy(); u2[r, 0] = np.float32(cdf[4])
    ref2 = oracle.sparsify(z, ref_s["idx"].shape[1], 1.0, T, u2)
    assert ref2["flags"][r] & oracle.FLAG_SMP
    names = ("idx", "logit", "count", "token", "lse", "mass")
    g = as_gpu(ref2, names)
    other = ref2["idx"][r, 4] if ref2["token"][r, 0] == ref2["idx"][r, 5] else ref2["idx"][r, 5]
    g["token"][r, 0] = int(other)
    compare_sparsify(g, ref2, logits=z, uniforms=u2, T=T)
    g["token"][r, 0] = int(ref2["idx"][r, 9])
    with pytest.raises(AssertionError):
        compare_sparsify(g, ref2, logits=z, uniforms=u2, T=T)


def test_sparsify_cut_moved_by_one_is_checked_against_the_order():
    z, ud, _, _, _, T = small_round()
    k = 16
    # top_p placed exactly on a cumulative mass of row 0
    full = oracle.sparsify(z[:1], k, 1.0, T, ud.numpy()[:1])
    zz = z[0].double().numpy()
    order = np.lexsort((np.arange(len(zz)), -zz))
    q = np.exp(zz / T - full["lse"][0])
    top_p = float(np.cumsum(q[order])[5])
    ref = oracle.sparsify(z[:1], k, top_p, T, ud.numpy()[:1])
    assert ref["flags"][0] & oracle.FLAG_SEL
    n = int(ref["count"][0])
    alt = oracle.sparsify(z[:1], n + 1 if n == 6 else n - 1, 1.0, T, ud.numpy()[:1])  # the cut one entry away
    names = ("idx", "logit", "count", "token", "lse", "mass")
    g = as_gpu(alt, names)
    pad = k - g["idx"].shape[1]
    g["idx"] = torch.cat([g["idx"], torch.full((1, pad), -1, dtype=torch.int32)], 1)
    g["logit"] = torch.cat([g["logit"], torch.full((1, pad), -np.inf)], 1)
    compare_sparsify(g, ref, logits=z[:1], uniforms=ud.numpy()[:1], T=T)
    g["idx"][0, 0] += 1
    with pytest.raises(AssertionError):
        compare_sparsify(g, ref, logits=z[:1], uniforms=ud.numpy()[:1], T=T)


def test_verify_compare_accepts_oracle_and_rejects_planted_mistakes():
    _, _, _, inp, ref_v, _ = small_round()
    names = ("accepted_len", "out_token", "accept_prob", "beta_hat", "lse_p")
    compare_verify(as_gpu(ref_v, names), ref_v, inputs=inp)
    b = int(np.nonzero((ref_v["flags"] == 0))[0][0])
    bad = as_gpu(ref_v, names); bad["out_token"][b] += 1
    with pytest.raises(AssertionError):
        compare_verify(bad, ref_v, inputs=inp)
    bad = as_gpu(ref_v, names); bad["accepted_len"][b] = (int(bad["accepted_len"][b]) + 1) % 4
    with pytest.raises(AssertionError):
        compare_verify(bad, ref_v, inputs=inp)


def test_verify_flagged_acceptance_other_branch_is_validated():
    """A uniform placed on an acceptance probability: the other stop position is accepted only with a
    token that is valid for THAT position's residual."""
    _, _, _, inp, ref_v, _ = small_round()
    b = 0
    ap = ref_v["accept_prob"][b]
    j = 0
    inp2 = dict(inp); ua = inp["ua"].copy(); ua[b, :] = 0.0; ua[b, j] = np.float32(ap[j]) if ap[j] < 1 else np.float32(0.999999)
    if ap[j] >= 1.0:
        pytest.skip("position always accepted for this seed")
    inp2["ua"] = ua
    ref2 = oracle.verify(inp["zp"], inp["idx"], inp["logit"], inp["count"], inp["token"], inp["Tq"], inp["Tp"], ua, inp["us"])
    assert ref2["flags"][b] & oracle.FLAG_ACC
    names = ("accepted_len", "out_token", "accept_prob", "beta_hat", "lse_p")
    # the other branch, computed by the oracle with the uniform pushed across
    ua3 = ua.copy(); ua3[b, j] = 0.0 if ref2["accepted_len"][b] == j else 0.9999999
    ref3 = oracle.verify(inp["zp"], inp["idx"], inp["logit"], inp["count"], inp["token"], inp["Tq"], inp["Tp"], ua3, inp["us"])
    assert ref3["accepted_len"][b] != ref2["accepted_len"][b]
    g = as_gpu(ref2, names); g["accepted_len"][b] = int(ref3["accepted_len"][b]); g["out_token"][b] = int(ref3["out_token"][b])
    compare_verify(g, ref2, inputs=inp2)
    g["out_token"][b] = int(ref3["out_token"][b]) + 1
    with pytest.raises(AssertionError):
        compare_verify(g, ref2, inputs=inp2)
    # a stop position no uniform within the band explains
    g = as_gpu(ref2, names); g["accepted_len"][b] = 3 if ref2["accepted_len"][b] < 2 else 0
    with pytest.raises(AssertionError):
        compare_verify(g, ref2, inputs=inp2)


def test_tree_compare_accepts_oracle_and_rejects_planted_mistakes():
    B, V, k, T = 3, 200, 8, 1.0
    parent, ndr, M, depth = synth.complete_tree((2, 2))
    N = len(parent)
    zq, zp = synth.tree_logits(B, parent, ndr, V, torch.float32, 0.5, 2, "cpu")
    ud = synth.uniforms((B * M, 2), 2, synth.TID_U_DRAFT)
    ref_s = oracle.sparsify(zq.reshape(B * M, V), k, 1.0, T, ud.numpy())
    toks = np.zeros((B, N), np.int32)
    for n in range(N):
        if ndr[n] >= 0:
            ch = [c for c in range(N) if parent[c] == n]
            for b in range(B):
                toks[b, ch] = ref_s["token"][b * M + ndr[n], :len(ch)]
    ua = synth.uniforms((B, N), 2, synth.TID_U_ACCEPT).numpy()
    us = synth.uniforms((B, N), 2, synth.TID_U_SAMPLE).numpy()
    inp = dict(zp=zp, parent=parent, ndr=ndr, toks=toks, idx=ref_s["idx"].reshape(B, M, k),
               logit=ref_s["logit"].reshape(B, M, k), count=ref_s["count"].reshape(B, M), Tq=T, Tp=T, ua=ua, us=us, depth=depth)
    ref = oracle.tree_verify(zp, parent, ndr, toks, inp["idx"], inp["logit"], inp["count"], T, T, ua, us, depth)
    names = ("accepted_path", "accepted_len", "out_token")
    compare_tree(as_gpu(ref, names), ref, inputs=inp)
    bad = as_gpu(ref, names); bad["out_token"][0] += 1
    with pytest.raises(AssertionError):
        compare_tree(bad, ref, inputs=inp)
    bad = as_gpu(ref, names)
    bad["accepted_len"][1] = 1 if ref["accepted_len"][1] != 1 else 0
    bad["accepted_path"][1] = torch.tensor([1, -1] if ref["accepted_len"][1] != 1 else [-1, -1], dtype=torch.int32)
    with pytest.raises(AssertionError):
        compare_tree(bad, ref, inputs=inp)
