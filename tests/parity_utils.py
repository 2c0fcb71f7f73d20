"""Helpers shared by the GPU parity tests: run the CUDA path and the CPU oracle on the same
seeded inputs and compare element by element.

Bar (written here, used everywhere): integer outputs (indices, counts, tokens, accepted
lengths, paths) bit-exact; fp32 outputs (logsumexp, retained mass, acceptance probabilities)
within 1e-5 relative (plus 1e-6 absolute for probabilities that can be tiny).

Where the oracle flags a decision that sits within 1e-6 of a boundary (a uniform next to a CDF
step or to an acceptance probability, a cumulative mass next to top_p), a finite-precision
implementation may land on the other side of it.  Such a row is not waved through: the GPU's
value is checked for VALIDITY against what the oracle returns for that row:
  * a sampled token t must have positive mass and CDF(t-1) - 1e-6 <= u <= CDF(t) + 1e-6 under
    the oracle's own distribution for the decision that was taken;
  * an accepted length / tree path that differs from the oracle's must be reachable by moving
    only uniforms that sit within 1e-6 of their acceptance probability, and the token must then
    be valid for THAT stop position (the oracle is run again with those decisions forced);
  * a top-p cut that differs must differ by one entry, and the set must be the oracle's order
    (logit descending, index ascending) cut at that length.
No branch of a compare_* function returns without having checked the GPU's value.
"""
import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import torch

import oracle
from paper_2512_16273_b200 import tslt

RTOL = 1e-5
ATOL_PROB = 1e-6
# logsumexp is a logarithm: its ABSOLUTE error is the relative error of the normaliser it stands for,
# so 1e-5 relative on the normaliser allows 1e-5 absolute on lse.  A tenth of that is asked for, next
# to the 1e-5 relative bound (which alone would demand 2e-8 absolute of an lse that happens to be 2e-3).
ATOL_LSE = 1e-6
BAND = 1e-6
ONE_M = float(np.nextafter(np.float32(1), np.float32(0)))


def to_np(t):
    return t.detach().cpu().numpy() if isinstance(t, torch.Tensor) else np.asarray(t)


def close(a, b, rtol=RTOL, atol=0.0):
    a = np.asarray(a, np.float64)
    b = np.asarray(b, np.float64)
    both_inf = np.isinf(a) & np.isinf(b) & (np.sign(a) == np.sign(b))
    with np.errstate(invalid="ignore"):  # inf - inf where both are infinite: covered by both_inf
        ok = both_inf | (np.abs(a - b) <= atol + rtol * np.abs(b))
    return ok


def clamp_u(u):
    u = float(u)
    if not u >= 0.0:
        return 0.0
    return ONE_M if u >= 1.0 else u


def token_is_valid(weights, u, pos):
    """Inverse-CDF validity of position `pos` for uniform u over non-negative weights: positive
    mass there, and u within 1e-6 of the interval [CDF(pos-1), CDF(pos)) (normalised)."""
    w = np.asarray(weights, np.float64)
    tot = w.sum()
    if not (0 <= pos < len(w)) or not tot > 0.0 or not w[pos] > 0.0:
        return False
    cum = np.cumsum(w) / tot
    lower = cum[pos - 1] if pos > 0 else 0.0
    u = clamp_u(u)
    # the last positive item also takes whatever rounding leaves above the total
    upper = 1.0 if not (w[pos + 1:] > 0.0).any() else cum[pos]
    return lower - BAND <= u <= upper + BAND


def logits_as_f64(z):
    """[..., V] torch CPU tensor (fp32 / bf16) or numpy float array -> float64 numpy (exact)."""
    if isinstance(z, torch.Tensor):
        return z.to(torch.float64).numpy()
    return np.asarray(z, np.float64)


def order_desc(z_row):
    """Indices of the finite entries in the order (logit descending, index ascending)."""
    z = np.asarray(z_row, np.float64)
    fin = np.nonzero(np.isfinite(z))[0]
    return fin[np.lexsort((fin, -z[fin]))]


def compare_sparsify(gpu: dict, ref: dict, what="", logits=None, uniforms=None, T=None):
    """Returns (number of flagged rows, number of rows).  Asserts on any mismatch; flagged rows
    are checked for validity, which needs `logits` [rows, V], `uniforms` [rows, s] and T."""
    idx, logit, count, token = (to_np(gpu[k]) for k in ("idx", "logit", "count", "token"))
    fl = ref["flags"]
    sel = (fl & oracle.FLAG_SEL) != 0
    smp = (fl & oracle.FLAG_SMP) != 0
    rows = len(fl)
    k = idx.shape[1]
    token = token.reshape(rows, -1)
    gmass = to_np(gpu["mass"]) if "mass" in gpu else None
    if (sel | smp).any():
        assert logits is not None and uniforms is not None and T is not None, \
            (what, "flagged rows need the inputs to be checked")
        uniforms = to_np(uniforms).reshape(rows, -1)
    for r in range(rows):
        n_ref = int(ref["count"][r])
        if sel[r]:
            # the cut may move by one position when a cumulative mass sits on top_p; the set is
            # then the oracle's order cut one entry earlier or later
            n = int(count[r])
            assert abs(n - n_ref) <= 1 and 1 <= n <= k, (what, "count", r, n, n_ref)
            z = logits_as_f64(logits[r])
            want = np.sort(order_desc(z)[:n])
            assert np.array_equal(idx[r, :n], want) and (idx[r, n:] == -1).all(), (what, "idx (cut moved)", r)
            assert np.array_equal(logit[r, :n], z[want].astype(np.float32)), (what, "logit (cut moved)", r)
            assert np.isneginf(logit[r, n:]).all(), (what, "logit padding", r)
            y = z[want] / T
            w = np.exp(y - y.max())
            for s in range(token.shape[1]):
                pos = np.searchsorted(want, token[r, s])
                assert pos < n and want[pos] == token[r, s] and token_is_valid(w, uniforms[r, s], pos), \
                    (what, "token (cut moved)", r, s, token[r, s])
            if gmass is not None:
                m = np.exp(y - float(ref["lse"][r])).sum()
                assert close(gmass[r], m, atol=ATOL_PROB), (what, "mass (cut moved)", r, gmass[r], m)
            continue
        assert count[r] == n_ref, (what, "count", r, count[r], n_ref)
        assert np.array_equal(idx[r], ref["idx"][r]), (what, "idx", r)
        assert logit[r].tobytes() == ref["logit"][r].tobytes(), (what, "logit", r)
        if not smp[r]:
            assert np.array_equal(token[r], ref["token"][r].reshape(-1)), (what, "token", r, token[r], ref["token"][r])
        else:
            y = ref["logit"][r, :n_ref].astype(np.float64) / T
            w = np.exp(y - y.max())
            for s in range(token.shape[1]):
                if token[r, s] == ref["token"][r].reshape(-1)[s]:
                    continue
                pos = np.searchsorted(ref["idx"][r, :n_ref], token[r, s])
                assert pos < n_ref and ref["idx"][r, pos] == token[r, s] and token_is_valid(w, uniforms[r, s], pos), \
                    (what, "token (flagged)", r, s, token[r, s], ref["token"][r])
    if "lse" in gpu:
        ok = close(to_np(gpu["lse"]), ref["lse"], atol=ATOL_LSE)
        assert ok.all(), (what, "lse", np.nonzero(~ok)[0][:5], to_np(gpu["lse"])[~ok][:5], ref["lse"][~ok][:5])
        m_ok = close(gmass, ref["mass"], atol=ATOL_PROB) | sel  # (rows whose cut moved were checked above)
        assert m_ok.all(), (what, "mass", np.nonzero(~m_ok)[0][:5], gmass[~m_ok][:5], ref["mass"][~m_ok][:5])
    return int((sel | smp).sum()), rows


def _verify_one(inp, b, ua_row):
    """The oracle on sequence b alone with the given acceptance uniforms, dense pmf wanted."""
    return oracle.verify(inp["zp"][b:b + 1], inp["idx"][b:b + 1], inp["logit"][b:b + 1], inp["count"][b:b + 1],
                         inp["token"][b:b + 1], inp["Tq"], inp["Tp"], np.asarray(ua_row, np.float32)[None],
                         inp["us"][b:b + 1], want_dense=True)


def compare_verify(gpu: dict, ref: dict, what="", inputs=None):
    """inputs: dict(zp [B, g+1, V] CPU logits, idx, logit, count, token (numpy, [B, g, ...]), Tq, Tp,
    ua [B, g], us [B]) as given to the oracle; needed only when some sequence is flagged or differs."""
    fl = ref["flags"]
    B = len(fl)
    acc = (fl & oracle.FLAG_ACC) != 0
    res = (fl & (oracle.FLAG_RES | oracle.FLAG_DEGEN)) != 0
    al, tok = to_np(gpu["accepted_len"]), to_np(gpu["out_token"])
    gamma = ref["accept_prob"].shape[1]
    for b in range(B):
        same_len = al[b] == ref["accepted_len"][b]
        if same_len and tok[b] == ref["out_token"][b]:
            continue
        assert acc[b] or (same_len and res[b]), \
            (what, "unflagged mismatch", b, al[b], ref["accepted_len"][b], tok[b], ref["out_token"][b], fl[b])
        assert inputs is not None, (what, "flagged sequences need the inputs to be checked")
        a = int(al[b])
        assert 0 <= a <= gamma, (what, "accepted_len out of range", b, a)
        ua = np.array([clamp_u(u) for u in to_np(inputs["ua"])[b]], np.float64)
        ap = ref["accept_prob"][b]
        forced = ua.astype(np.float32).copy()
        if not same_len:
            # every decision of the GPU's run must be compatible with the oracle's acceptance
            # probabilities to within the band; then force exactly those decisions
            for j in range(a):
                assert ua[j] < ap[j] + BAND, (what, "accepted beyond the band", b, j, ua[j], ap[j])
                forced[j] = 0.0
            if a < gamma:
                assert ua[a] >= ap[a] - BAND, (what, "rejected beyond the band", b, a, ua[a], ap[a])
                forced[a] = ONE_M
        o2 = _verify_one(inputs, b, forced)
        assert o2["accepted_len"][0] == a, (what, "stop position not reachable", b, a, o2["accepted_len"][0])
        assert token_is_valid(o2["final_pmf"][0], to_np(inputs["us"])[b], int(tok[b])), \
            (what, "out_token invalid for its stop position", b, a, tok[b], o2["out_token"][0])
    if "accept_prob" in gpu:
        for key in ("accept_prob", "beta_hat"):
            ok = close(to_np(gpu[key]), ref[key], atol=ATOL_PROB)
            assert ok.all(), (what, key, np.argwhere(~ok)[:5], to_np(gpu[key])[~ok][:5], ref[key][~ok][:5])
        ok = close(to_np(gpu["lse_p"]), ref["lse_p"], atol=ATOL_LSE)
        assert ok.all(), (what, "lse_p", np.argwhere(~ok)[:5])
    return int((acc | res).sum()), B


def compare_tree(gpu: dict, ref: dict, what="", inputs=None):
    """inputs: dict(zp [B, N, V], parent, ndr, toks [B, N], idx, logit, count ([B, M, ...]), Tq, Tp,
    ua [B, N], us [B, N], depth)."""
    fl = ref["flags"]
    B = len(fl)
    acc = (fl & oracle.FLAG_ACC) != 0
    res = (fl & (oracle.FLAG_RES | oracle.FLAG_DEGEN)) != 0
    al, tok, path = to_np(gpu["accepted_len"]), to_np(gpu["out_token"]), to_np(gpu["accepted_path"])
    for b in range(B):
        same_path = al[b] == ref["accepted_len"][b] and np.array_equal(path[b], ref["accepted_path"][b])
        if same_path and tok[b] == ref["out_token"][b]:
            continue
        assert acc[b] or (same_path and res[b]), \
            (what, "unflagged mismatch", b, al[b], ref["accepted_len"][b], path[b], ref["accepted_path"][b],
             tok[b], ref["out_token"][b], fl[b])
        assert inputs is not None, (what, "flagged sequences need the inputs to be checked")
        parent = list(inputs["parent"])
        N = len(parent)
        n_acc = int(al[b])
        gp = [int(x) for x in path[b, :n_acc]]
        assert all(x == -1 for x in path[b, n_acc:]), (what, "path padding", b)
        ua0 = np.array([clamp_u(u) for u in to_np(inputs["ua"])[b]], np.float64)
        forced = ua0.astype(np.float32).copy()
        node, decisions = 0, []  # (child, accepted?)
        for step in range(n_acc + 1):
            children = [c for c in range(N) if parent[c] == node]
            nxt = gp[step] if step < n_acc else None
            if nxt is not None:
                assert nxt in children, (what, "path leaves the tree", b, gp)
            for c in children:
                if c == nxt:
                    decisions.append((c, True))
                    forced[c] = 0.0
                    break
                decisions.append((c, False))
                forced[c] = ONE_M
            if nxt is None:
                break
            node = nxt
        sl = slice(b, b + 1)
        o2 = oracle.tree_verify(inputs["zp"][sl], inputs["parent"], inputs["ndr"], inputs["toks"][sl], inputs["idx"][sl],
                                inputs["logit"][sl], inputs["count"][sl], inputs["Tq"], inputs["Tp"], forced[None],
                                to_np(inputs["us"])[sl], inputs["depth"], want_dense=True)
        assert o2["accepted_len"][0] == n_acc and list(o2["accepted_path"][0, :n_acc]) == gp, \
            (what, "path not reachable", b, gp, o2["accepted_path"][0])
        for c, took in decisions:  # each decision within the band of the oracle's probability for it
            ap = o2["accept_prob"][0, c]
            if took:
                assert ua0[c] < ap + BAND, (what, "accepted beyond the band", b, c, ua0[c], ap)
            else:
                assert ua0[c] >= ap - BAND, (what, "rejected beyond the band", b, c, ua0[c], ap)
        stop = gp[-1] if gp else 0
        assert token_is_valid(o2["final_pmf"][0], to_np(inputs["us"])[b, stop], int(tok[b])), \
            (what, "out_token invalid for its stop node", b, stop, tok[b], o2["out_token"][0])
    return int((acc | res).sum()), B


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


# ---- the oracle over the host cores (ctypes releases the GIL) -------------------------------------
def _cores():
    return max(1, len(os.sched_getaffinity(0)))


def oracle_sparsify_parallel(z_rows, k, top_p, T, u):
    """oracle.sparsify on [rows, V] CPU logits, one row per task over the host cores."""
    zn, _ = oracle.as_logits(z_rows)
    u = np.ascontiguousarray(to_np(u), np.float32).reshape(zn.shape[0], -1)
    oracle.lib()
    with ThreadPoolExecutor(max_workers=_cores()) as ex:
        parts = list(ex.map(lambda r: oracle.sparsify(zn[r:r + 1], k, top_p, T, u[r:r + 1]), range(zn.shape[0])))
    return {key: np.concatenate([p[key] for p in parts]) for key in parts[0]}


def oracle_verify_parallel(zp, di, dl, dc, tk, Tq, Tp, ua, us):
    zn, _ = oracle.as_logits(zp)
    B = zn.shape[0]
    oracle.lib()
    with ThreadPoolExecutor(max_workers=_cores()) as ex:
        parts = list(ex.map(lambda b: oracle.verify(zn[b:b + 1], di[b:b + 1], dl[b:b + 1], dc[b:b + 1], tk[b:b + 1],
                                                    Tq, Tp, ua[b:b + 1], us[b:b + 1]), range(B)))
    return {key: np.concatenate([p[key] for p in parts]) for key in parts[0]}


def oracle_tree_parallel(zp, parent, ndr, toks, di, dl, dc, Tq, Tp, ua, us, depth):
    zn, _ = oracle.as_logits(zp)
    B = zn.shape[0]
    oracle.lib()
    with ThreadPoolExecutor(max_workers=_cores()) as ex:
        parts = list(ex.map(lambda b: oracle.tree_verify(zn[b:b + 1], parent, ndr, toks[b:b + 1], di[b:b + 1],
                                                         dl[b:b + 1], dc[b:b + 1], Tq, Tp, ua[b:b + 1], us[b:b + 1], depth),
                            range(B)))
    return {key: np.concatenate([p[key] for p in parts]) for key in parts[0]}


def verify_inputs(zp_cpu, ref_s, B, gamma, k, tok, Tq, Tp, ua, us):
    return dict(zp=zp_cpu, idx=np.ascontiguousarray(ref_s["idx"]).reshape(B, gamma, k),
                logit=np.ascontiguousarray(ref_s["logit"]).reshape(B, gamma, k),
                count=np.ascontiguousarray(ref_s["count"]).reshape(B, gamma), token=np.ascontiguousarray(tok, np.int32),
                Tq=Tq, Tp=Tp, ua=np.ascontiguousarray(to_np(ua), np.float32), us=np.ascontiguousarray(to_np(us), np.float32))


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
    f1 = compare_sparsify(gpu_s, ref_s, what + " sparsify", logits=zq_cpu.reshape(rows, V), uniforms=ud, T=T)
    tok = ref_s["token"][:, 0].reshape(B, gamma)
    inp = verify_inputs(zp_cpu, ref_s, B, gamma, k, tok, T, T, ua, us)
    ref_v = oracle.verify(zp_cpu, inp["idx"], inp["logit"], inp["count"], inp["token"], T, T, inp["ua"], inp["us"])
    gpu_v = tslt.verify(to_gpu_rows(zp_cpu), torch.from_numpy(inp["idx"]).cuda(), torch.from_numpy(inp["logit"]).cuda(),
                        torch.from_numpy(inp["count"]).cuda(), torch.from_numpy(inp["token"]).cuda(), T, T,
                        ua.cuda(), us.cuda())
    torch.cuda.synchronize()
    assert tslt.workspace_status(gpu_v["workspace"]) == 0
    f2 = compare_verify(gpu_v, ref_v, what + " verify", inputs=inp)
    return f1, f2, ref_s, ref_v
