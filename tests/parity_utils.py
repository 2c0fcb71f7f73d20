"""Helpers shared by the GPU parity tests: run the CUDA path and the CPU oracle on the same
seeded inputs and compare element by element.

Bar (written here, used everywhere): integer outputs (indices, counts, tokens, accepted
lengths, paths) bit-exact except where the oracle flags a decision within 1e-6 of a
boundary; fp32 outputs (logsumexp, retained mass, acceptance probabilities) within 1e-5
relative (plus 1e-6 absolute for probabilities that can be tiny).
"""
import numpy as np
import torch

import oracle
from paper_2512_16273_b200 import tslt

RTOL = 1e-5
ATOL_PROB = 1e-6


def to_np(t):
    return t.detach().cpu().numpy()


def close(a, b, rtol=RTOL, atol=0.0):
    a = np.asarray(a, np.float64)
    b = np.asarray(b, np.float64)
    both_inf = np.isinf(a) & np.isinf(b) & (np.sign(a) == np.sign(b))
    with np.errstate(invalid="ignore"):  # inf - inf where both are infinite: covered by both_inf
        ok = both_inf | (np.abs(a - b) <= atol + rtol * np.abs(b))
    return ok


def compare_sparsify(gpu: dict, ref: dict, what=""):
    """Returns (number of flagged rows, number of rows).  Asserts on any unflagged mismatch."""
    idx, logit, count, token = (to_np(gpu[k]) for k in ("idx", "logit", "count", "token"))
    fl = ref["flags"]
    sel = (fl & oracle.FLAG_SEL) != 0
    smp = (fl & oracle.FLAG_SMP) != 0
    rows = len(fl)
    for r in range(rows):
        if sel[r]:
            # the cut may move by one position when a cumulative mass sits on top_p
            assert abs(int(count[r]) - int(ref["count"][r])) <= 1, (what, r)
            continue
        assert count[r] == ref["count"][r], (what, "count", r, count[r], ref["count"][r])
        assert np.array_equal(idx[r], ref["idx"][r]), (what, "idx", r)
        assert np.array_equal(logit[r], ref["logit"][r]), (what, "logit", r)
        if not smp[r]:
            assert np.array_equal(token[r], ref["token"][r]), (what, "token", r, token[r], ref["token"][r])
        else:
            assert np.isin(token[r], idx[r]).all(), (what, "token not in set", r)
    if "lse" in gpu:
        ok = close(to_np(gpu["lse"]), ref["lse"])
        assert ok.all(), (what, "lse", np.nonzero(~ok)[0][:5])
        m_ok = close(to_np(gpu["mass"]), ref["mass"], atol=ATOL_PROB) | sel
        assert m_ok.all(), (what, "mass", np.nonzero(~m_ok)[0][:5])
    return int((sel | smp).sum()), rows


def compare_verify(gpu: dict, ref: dict, what=""):
    fl = ref["flags"]
    acc = (fl & oracle.FLAG_ACC) != 0
    res = (fl & (oracle.FLAG_RES | oracle.FLAG_DEGEN)) != 0
    al, tok = to_np(gpu["accepted_len"]), to_np(gpu["out_token"])
    bad_len = (al != ref["accepted_len"]) & ~acc
    assert not bad_len.any(), (what, "accepted_len", np.nonzero(bad_len)[0][:5], al[bad_len][:5],
                               ref["accepted_len"][bad_len][:5])
    bad_tok = (tok != ref["out_token"]) & ~(acc | res)
    assert not bad_tok.any(), (what, "out_token", np.nonzero(bad_tok)[0][:5], tok[bad_tok][:5],
                               ref["out_token"][bad_tok][:5])
    if "accept_prob" in gpu:
        for key in ("accept_prob", "beta_hat"):
            ok = close(to_np(gpu[key]), ref[key], atol=ATOL_PROB)
            assert ok.all(), (what, key, np.argwhere(~ok)[:5], to_np(gpu[key])[~ok][:5], ref[key][~ok][:5])
        ok = close(to_np(gpu["lse_p"]), ref["lse_p"])
        assert ok.all(), (what, "lse_p", np.argwhere(~ok)[:5])
    return int((acc | res).sum()), len(fl)


def compare_tree(gpu: dict, ref: dict, what=""):
    fl = ref["flags"]
    acc = (fl & oracle.FLAG_ACC) != 0
    res = (fl & (oracle.FLAG_RES | oracle.FLAG_DEGEN)) != 0
    al, tok, path = to_np(gpu["accepted_len"]), to_np(gpu["out_token"]), to_np(gpu["accepted_path"])
    bad = (al != ref["accepted_len"]) & ~acc
    assert not bad.any(), (what, "accepted_len", np.nonzero(bad)[0][:5])
    badp = (path != ref["accepted_path"]).any(axis=1) & ~acc
    assert not badp.any(), (what, "accepted_path", np.nonzero(badp)[0][:5])
    badt = (tok != ref["out_token"]) & ~(acc | res)
    assert not badt.any(), (what, "out_token", np.nonzero(badt)[0][:5], tok[badt][:5], ref["out_token"][badt][:5])
    return int((acc | res).sum()), len(fl)


def to_gpu_rows(t_cpu):
    """Copy [..., V] logits to the GPU with rows padded to a multiple of 16 bytes (the ABI's
    alignment rule), returned as a [..., :V] view."""
    V = t_cpu.shape[-1]
    per = 16 // t_cpu.element_size()
    Vp = (V + per - 1) // per * per
    if Vp == V:
        return t_cpu.cuda()
    buf = torch.zeros(*t_cpu.shape[:-1], Vp, dtype=t_cpu.dtype, device="cuda")
    buf[..., :V] = t_cpu.cuda()
    return buf[..., :V]


def run_sequence_case(zq_cpu, zp_cpu, k, top_p, T, seed, num_samples=1, what=""):
    """Full single-candidate round on both sides from CPU tensors zq [B,g,V], zp [B,g+1,V].

    The verifier of both sides consumes the ORACLE's sparse drafts, so each entry point is
    compared on identical inputs."""
    from paper_2512_16273_b200 import synth
    B, gamma, V = zq_cpu.shape
    rows = B * gamma
    ud = synth.uniforms((rows, num_samples), seed, synth.TID_U_DRAFT)
    ua = synth.uniforms((B, gamma), seed, synth.TID_U_ACCEPT)
    us = synth.uniforms((B,), seed, synth.TID_U_SAMPLE)
    ref_s = oracle.sparsify(zq_cpu.reshape(rows, V), k, top_p, T, ud.numpy())
    gpu_s = tslt.sparsify(to_gpu_rows(zq_cpu), k, top_p, T, ud.cuda())
    torch.cuda.synchronize()
    assert tslt.workspace_status(gpu_s["workspace"]) == 0
    f1 = compare_sparsify(gpu_s, ref_s, what + " sparsify")
    tok = ref_s["token"][:, 0].reshape(B, gamma)
    ref_v = oracle.verify(zp_cpu, ref_s["idx"].reshape(B, gamma, k), ref_s["logit"].reshape(B, gamma, k),
                          ref_s["count"].reshape(B, gamma), tok, T, T, ua.numpy(), us.numpy())
    gpu_v = tslt.verify(to_gpu_rows(zp_cpu), torch.from_numpy(ref_s["idx"]).cuda().view(B, gamma, k),
                        torch.from_numpy(ref_s["logit"]).cuda().view(B, gamma, k),
                        torch.from_numpy(ref_s["count"]).cuda().view(B, gamma),
                        torch.from_numpy(np.ascontiguousarray(tok)).cuda(), T, T, ua.cuda(), us.cuda())
    torch.cuda.synchronize()
    assert tslt.workspace_status(gpu_v["workspace"]) == 0
    f2 = compare_verify(gpu_v, ref_v, what + " verify")
    return f1, f2, ref_s, ref_v
