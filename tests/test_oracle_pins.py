"""Pins for the CPU oracle: it is checked against what the paper and the mathematics fix,
never against itself or the CUDA path.

* losslessness of single-candidate verification (Section 3.2: the output law equals the
  target's whatever the draft distribution is) by exhaustive enumeration on V = 8..16;
* the same for multi-candidate verification (Section 4.2) over all candidate tuples;
* acceptance rate beta = sum min(q, p) = 1 - TV (the acceptance-rate lemma of Section 3.2),
  also by Monte Carlo through the oracle's own sampling code;
* Theorem 1: TV(q^, q) = sigma exactly and |beta^ - beta| <= sigma; Lemma 2;
* residual normaliser Z = 1 - beta^ (appendix, proof of the recursive TV lemma);
* multi-candidate acceptance beta^(j) = sum min(q, p^(j)) and total acceptance theta
  (Section 4.3);
* reductions to library routines (scipy softmax / logsumexp, torch.topk, argmax);
* hand-built rows for tie-break, padding, ordering, top-p crossing and cap binding;
* inverse-CDF conventions at u = 0 and u -> 1.
"""
import itertools
import math
import os

import numpy as np
import pytest
import scipy.special
import torch

import oracle
from paper_2512_16273_b200 import synth


def softmax64(z, T=1.0):
    return scipy.special.softmax(np.asarray(z, np.float64) / T, axis=-1)


def tiny_case(seed, V, spread=2.0):
    rng = np.random.default_rng(seed)
    zq = (rng.normal(size=V) * spread).astype(np.float32)
    zp = (zq + rng.normal(size=V) * 0.8).astype(np.float32)
    return zq, zp


def sparsify_row(zq, k, top_p, T, u=0.5, dense=True):
    o = oracle.sparsify(zq[None, :], k, top_p, T, np.array([[u]], np.float32), want_dense=dense)
    return o


def verify_one(zp_rows, sp, token, T_q, T_p, u_acc, u_smp, dense=True):
    """gamma = 1 verification of `token` against the payload of a single sparsify row."""
    return oracle.verify(zp_rows[None, :, :], sp["idx"][None], sp["logit"][None], sp["count"][None],
                         np.array([[token]], np.int32), T_q, T_p,
                         np.array([[u_acc]], np.float32), np.array([u_smp], np.float32),
                         want_dense=dense)


CASES = [
    # (seed, V, k, top_p, T_q, T_p)
    (1, 8, 3, 1.0, 1.0, 1.0),
    (2, 8, 8, 1.0, 1.0, 1.0),
    (3, 12, 5, 0.8, 0.7, 0.7),
    (4, 16, 4, 1.0, 1.3, 0.9),
    (5, 16, 16, 0.6, 1.0, 1.0),
    (6, 9, 1, 1.0, 1.0, 1.0),
]


@pytest.mark.parametrize("seed,V,k,top_p,Tq,Tp", CASES)
def test_single_candidate_lossless_enumeration(seed, V, k, top_p, Tq, Tp):
    """Sum over drafted tokens of q~(x) [a(x) 1{y=x}] + (1 - beta^) res(y) = p(y) for all y."""
    zq, zp = tiny_case(seed, V)
    zp_rows = np.stack([zp, zp])  # row 0 verifies, row 1 is the bonus row
    sp = sparsify_row(zq, k, top_p, Tq)
    qt = sp["qtilde"][0]
    p = softmax64(zp, Tp)
    assert abs(qt.sum() - 1.0) < 1e-12
    law = np.zeros(V)
    beta = 0.0
    res = None
    for x in np.nonzero(qt)[0]:
        # u_accept just below 1 forces a rejection whenever a(x) < 1, exposing the residual pmf
        o = verify_one(zp_rows, sp, int(x), Tq, Tp, np.nextafter(np.float32(1), np.float32(0)), 0.5)
        a = o["accept_prob"][0, 0]
        law[x] += qt[x] * a
        beta += qt[x] * a
        if o["accepted_len"][0] == 0:
            r = o["final_pmf"][0]
            if res is None:
                res = r
            else:
                assert np.allclose(res, r, atol=1e-15)
            assert r[x] == 0.0  # a rejected token has p(x) < q~(x): no residual mass
            assert abs(r.sum() - 1.0) < 1e-12
        assert abs(o["beta_hat"][0, 0] - np.minimum(p, qt).sum()) < 1e-12
    assert abs(beta - np.minimum(p, qt).sum()) < 1e-12  # acceptance-rate lemma
    if res is not None:
        law += (1.0 - beta) * res
    else:
        assert abs(beta - 1.0) < 1e-12
    assert np.allclose(law, p, atol=1e-12), (law, p)


@pytest.mark.parametrize("seed,V,k,top_p,Tq,Tp", CASES[:4])
def test_single_candidate_lossless_uniform_lattice(seed, V, k, top_p, Tq, Tp):
    """Drive the oracle's sampling code with lattices of uniforms; the three decisions use
    independent uniforms, so the joint law factorises into three 1-D lattices."""
    G = 4096
    zq, zp = tiny_case(seed, V)
    zp_rows = np.stack([zp, zp])
    p = softmax64(zp, Tp)
    grid = ((np.arange(G) + 0.5) / G).astype(np.float32)
    # (1) drafted token law from the u_draft lattice
    o = oracle.sparsify(np.repeat(zq[None], G, 0), k, top_p, Tq, grid[:, None])
    q_emp = np.bincount(o["token"][:, 0], minlength=V) / G
    sp1 = sparsify_row(zq, k, top_p, Tq)
    assert np.abs(q_emp - sp1["qtilde"][0]).max() <= 1.0 / G + 1e-12
    law = np.zeros(V)
    rej_mass = 0.0
    res_emp = None
    B = G
    tgt = np.repeat(zp_rows[None], B, 0)
    di = np.repeat(sp1["idx"][None], B, 0)
    dl = np.repeat(sp1["logit"][None], B, 0)
    dc = np.repeat(sp1["count"][None], B, 0)
    for x in np.nonzero(q_emp)[0]:
        # (2) acceptance from the u_accept lattice, (3) residual from the u_sample lattice
        o = oracle.verify(tgt, di, dl, dc, np.full((B, 1), x, np.int32), Tq, Tp, grid[:, None],
                          grid)
        acc = (o["accepted_len"] == 1)
        law[x] += q_emp[x] * acc.mean()
        rej_mass += q_emp[x] * (1 - acc.mean())
        if (~acc).any():
            # all lattice points of u_sample among the rejected ones: take the residual law from
            # a run where every point rejects
            o2 = oracle.verify(tgt, di, dl, dc, np.full((B, 1), x, np.int32), Tq, Tp,
                               np.full((B, 1), np.nextafter(np.float32(1), np.float32(0))), grid)
            assert (o2["accepted_len"] == 0).all()
            res_emp = np.bincount(o2["out_token"], minlength=V) / G
    if res_emp is not None:
        law += rej_mass * res_emp
    # each of the three lattices resolves its law to 1/G per step of its CDF
    assert np.abs(law - p).max() < 3.0 * V / G, (law, p)


def test_bonus_token_law_is_target():
    """All accepted (gamma = 2, z_p == z_q, k = V): the extra token is drawn from P_{gamma+1}."""
    V, G = 10, 4096
    rng = np.random.default_rng(7)
    zq = rng.normal(size=(2, V)).astype(np.float32) * 2
    zb = rng.normal(size=V).astype(np.float32) * 2
    tgt = np.concatenate([zq, zb[None]], 0)
    sp = oracle.sparsify(zq, V, 1.0, 1.0, np.full((2, 1), 0.3, np.float32))
    grid = ((np.arange(G) + 0.5) / G).astype(np.float32)
    o = oracle.verify(np.repeat(tgt[None], G, 0), np.repeat(sp["idx"][None], G, 0),
                      np.repeat(sp["logit"][None], G, 0), np.repeat(sp["count"][None], G, 0),
                      np.repeat(sp["token"].reshape(1, 2), G, 0), 1.0, 1.0,
                      np.tile(grid[:, None], (1, 2)), grid)
    assert (o["accepted_len"] == 2).all()  # identical distributions: ratio = 1, always accepted
    emp = np.bincount(o["out_token"], minlength=V) / G
    assert np.abs(emp - softmax64(zb)).max() <= 1.0 / G + 1e-12


@pytest.mark.parametrize("seed,V,k,top_p,T", [(11, 16, 5, 1.0, 1.0), (12, 16, 16, 0.7, 0.8),
                                                (13, 12, 3, 1.0, 1.5), (14, 300, 40, 0.9, 1.0)])
def test_theorem1_truncation_identities(seed, V, k, top_p, T):
    """TV(q^, q) = sigma exactly, |beta^ - beta| <= sigma, Lemma 2, Z = 1 - beta^."""
    zq, zp = tiny_case(seed, V)
    sp = sparsify_row(zq, k, top_p, T)
    q = softmax64(zq, T)
    p = softmax64(zp, T)
    qt = sp["qtilde"][0]
    n = sp["count"][0]
    S = sp["idx"][0, :n]
    rho = q[S].sum()
    sigma = 1.0 - rho
    assert abs(sp["mass"][0] - rho) < 1e-12
    assert abs(sp["lse"][0] - scipy.special.logsumexp(zq.astype(np.float64) / T)) < 1e-12
    assert np.allclose(qt[S], q[S] / rho, rtol=1e-12)          # renormalisation on the kept set
    assert qt.sum() == pytest.approx(1.0, abs=1e-12)
    assert (np.delete(qt, S) == 0).all()                         # zero elsewhere
    tv_qq = 0.5 * np.abs(qt - q).sum()
    assert abs(tv_qq - sigma) < 1e-12                            # Theorem 1, second claim
    beta = np.minimum(q, p).sum()
    beta_hat = np.minimum(qt, p).sum()
    assert abs(beta_hat - beta) <= sigma + 1e-12                 # Theorem 1, first claim
    tv = lambda a, b: 0.5 * np.abs(a - b).sum()
    assert abs(tv(qt, p) - tv(q, p)) <= tv(qt, q) + 1e-12        # Lemma 2
    zp_rows = np.stack([zp, zp])
    x = int(S[0])
    o = verify_one(zp_rows, sp, x, T, T, 0.5, 0.5)
    assert abs(o["beta_hat"][0, 0] - beta_hat) < 1e-12
    assert abs(o["beta_hat"][0, 0] - (1 - tv(qt, p))) < 1e-12    # beta^ = 1 - TV(q^, p)
    assert abs(o["lse_p"][0, 0] - scipy.special.logsumexp(zp.astype(np.float64) / T)) < 1e-12
    # the unnormalised residual sums to Z = 1 - beta^
    Z = np.maximum(p - qt, 0).sum()
    assert abs(Z - (1 - beta_hat)) < 1e-12
    if Z > 1e-9:
        o = verify_one(zp_rows, sp, x, T, T, np.nextafter(np.float32(1), np.float32(0)), 0.5)
        if o["accepted_len"][0] == 0:
            assert np.allclose(o["final_pmf"][0], np.maximum(p - qt, 0) / Z, atol=1e-13)


def test_acceptance_monte_carlo():
    """Empirical acceptance through the oracle's sampling code matches sum min(p, q~)."""
    V, k, n = 16, 6, 1_000_000
    zq, zp = tiny_case(21, V)
    zp_rows = np.stack([zp, zp])
    ud = synth.uniforms((n, 1), 5, synth.TID_U_DRAFT).numpy()
    ua = synth.uniforms((n, 1), 5, synth.TID_U_ACCEPT).numpy()
    us = synth.uniforms((n,), 5, synth.TID_U_SAMPLE).numpy()
    # row_stride = 0 replays the same row for every sample
    sp = oracle.sparsify(zq[None], k, 1.0, 1.0, ud, row_stride=0, rows=n)
    assert (sp["count"] == k).all()
    tgt = np.broadcast_to(zp_rows[None], (n, 2, V))
    o = oracle.verify(np.ascontiguousarray(tgt), sp["idx"], sp["logit"], sp["count"], sp["token"],
                      1.0, 1.0, ua, us)
    sp1 = sparsify_row(zq, k, 1.0, 1.0)
    p = softmax64(zp)
    beta_hat = np.minimum(p, sp1["qtilde"][0]).sum()
    acc = (o["accepted_len"] == 1).mean()
    sd = math.sqrt(beta_hat * (1 - beta_hat) / n)
    assert abs(acc - beta_hat) < 4 * sd, (acc, beta_hat, sd)
    # and the emitted token (accepted draft or correction) follows p
    emitted = np.where(o["accepted_len"] == 1, sp["token"][:, 0], o["out_token"])
    emp = np.bincount(emitted, minlength=V) / n
    assert np.abs(emp - p).max() < 5 * math.sqrt(0.25 / n)


def test_library_reductions():
    rng = np.random.default_rng(31)
    V = 257
    z = rng.normal(size=(5, V)).astype(np.float32) * 3
    T = 0.9
    u = rng.random((5, 1), dtype=np.float32)
    # k = V, top_p = 1: q~ is the softmax, lse is logsumexp
    o = oracle.sparsify(z, V, 1.0, T, u, want_dense=True)
    assert np.allclose(o["qtilde"], softmax64(z, T), rtol=1e-12, atol=0)
    assert np.allclose(o["lse"], scipy.special.logsumexp(z.astype(np.float64) / T, axis=1), rtol=1e-13)
    assert (o["count"] == V).all() and np.allclose(o["mass"], 1.0, atol=1e-12)
    assert (o["idx"] == np.arange(V)[None]).all() and (o["logit"] == z).all()
    # distinct fp32 values: the index set is torch.topk's
    k = 17
    o = oracle.sparsify(z, k, 1.0, T, u)
    tk = torch.topk(torch.from_numpy(z), k, dim=1).indices.numpy()
    for r in range(5):
        assert len(np.unique(z[r])) == V
        assert sorted(tk[r].tolist()) == o["idx"][r].tolist()
        assert (o["logit"][r] == z[r, o["idx"][r]]).all()
    # k = 1: the token is the (lowest-index) argmax and acceptance probability is min(1, p(argmax))
    o = oracle.sparsify(z, 1, 1.0, T, u)
    assert (o["token"][:, 0] == z.argmax(1)).all() and (o["idx"][:, 0] == z.argmax(1)).all()
    zp = (z + rng.normal(size=z.shape)).astype(np.float32)
    tgt = np.stack([zp, zp], 1)  # [5, 2, V], gamma = 1
    v = oracle.verify(tgt, o["idx"][:, None], o["logit"][:, None], o["count"][:, None], o["token"],
                      T, T, rng.random((5, 1), dtype=np.float32), rng.random(5, dtype=np.float32))
    p = softmax64(zp, T)
    assert np.allclose(v["accept_prob"][:, 0], p[np.arange(5), z.argmax(1)], rtol=1e-12)
    # z_p == z_q with k = V: everything is accepted whatever the uniforms
    gamma = 4
    zq = rng.normal(size=(gamma, V)).astype(np.float32)
    sp = oracle.sparsify(zq, V, 1.0, 1.0, rng.random((gamma, 1), dtype=np.float32))
    tgt = np.concatenate([zq, zq[:1]], 0)[None]
    v = oracle.verify(tgt, sp["idx"][None], sp["logit"][None], sp["count"][None],
                      sp["token"].reshape(1, gamma), 1.0, 1.0,
                      np.full((1, gamma), np.nextafter(np.float32(1), np.float32(0))),
                      np.array([0.5], np.float32))
    assert v["accepted_len"][0] == gamma
    assert np.allclose(v["accept_prob"], 1.0) and np.allclose(v["beta_hat"], 1.0, atol=1e-12)


def test_bf16_inputs_upcast_exactly():
    rng = np.random.default_rng(33)
    zt = torch.from_numpy(rng.normal(size=(3, 64)).astype(np.float32) * 4).to(torch.bfloat16)
    u = rng.random((3, 2), dtype=np.float32)
    a = oracle.sparsify(zt, 8, 0.9, 0.8, u)
    b = oracle.sparsify(zt.float(), 8, 0.9, 0.8, u)
    for key in a:
        assert np.array_equal(a[key], b[key]), key


def brute_topk(z, k):
    order = sorted(range(len(z)), key=lambda i: (-float(z[i]), i))
    return sorted(order[:k])


def test_tie_break_padding_and_order():
    # heavy ties: lower index wins; output ascending; padding -1 / -inf
    z = np.array([1.0, 3.0, 3.0, 2.0, 3.0, 2.0, 1.0, 2.0, -np.inf, 3.0], np.float32)
    for k in range(1, 10):
        o = oracle.sparsify(z[None], k, 1.0, 1.0, np.array([[0.0]], np.float32))
        n = o["count"][0]
        assert n == k
        assert o["idx"][0, :n].tolist() == brute_topk(z[:8].tolist() + [-1e30] + [3.0], k)
        assert (o["logit"][0, :n] == z[o["idx"][0, :n]]).all()
    # -inf is never selected: k larger than the finite count
    o = oracle.sparsify(z[None], 10, 1.0, 1.0, np.array([[0.0]], np.float32))
    assert o["count"][0] == 9 and o["idx"][0, 9] == -1 and np.isneginf(o["logit"][0, 9])
    assert 8 not in o["idx"][0, :9]
    # -0.0 and +0.0 tie (compare as floats): the lower index wins
    z2 = np.array([0.0, -0.0, -1.0, -0.0], np.float32)
    o = oracle.sparsify(z2[None], 2, 1.0, 1.0, np.array([[0.0]], np.float32))
    assert o["idx"][0].tolist() == [0, 1]
    # all entries non-finite
    z3 = np.full(6, -np.inf, np.float32)
    o = oracle.sparsify(z3[None], 3, 1.0, 1.0, np.array([[0.5]], np.float32))
    assert o["count"][0] == 0 and o["token"][0, 0] == -1 and o["flags"][0] & oracle.FLAG_EMPTY


def test_top_p_crossing_and_cap():
    # probabilities 0.4, 0.3, 0.2, 0.1 placed at scattered indices
    probs = np.array([0.1, 0.4, 0.2, 0.3])
    z = np.log(probs).astype(np.float32)
    u = np.array([[0.0]], np.float32)

    def n_for(top_p, k=4):
        return oracle.sparsify(z[None], k, top_p, 1.0, u)

    assert n_for(0.35)["idx"][0].tolist() == [1, -1, -1, -1]          # 0.4 >= 0.35
    assert n_for(0.45)["idx"][0].tolist() == [1, 3, -1, -1]           # crossing token is kept
    assert n_for(0.75)["idx"][0].tolist() == [1, 2, 3, -1]            # 0.7 < 0.75 <= 0.9
    assert n_for(0.95)["count"][0] == 4
    assert n_for(0.95, k=2)["idx"][0].tolist() == [1, 3]               # cap binds before crossing
    assert n_for(1.0, k=3)["idx"][0].tolist() == [1, 2, 3]             # pure top-k
    # mass is the cumulative full-softmax probability of the kept set
    assert n_for(0.45)["mass"][0] == pytest.approx(0.7, abs=1e-6)
    # boundary flag: top_p within 1e-6 of a cumulative next to the cut, not otherwise
    c2 = float(softmax64(z)[[1, 3]].sum())
    assert n_for(c2 + 5e-7)["flags"][0] & oracle.FLAG_SEL
    assert n_for(c2 - 5e-7)["flags"][0] & oracle.FLAG_SEL
    assert not (n_for(c2 + 1e-4)["flags"][0] & oracle.FLAG_SEL)
    # crossing inside a tie group: equal logits are taken in index order
    z4 = np.log(np.array([0.25, 0.25, 0.25, 0.25])).astype(np.float32)
    o = oracle.sparsify(z4[None], 4, 0.6, 1.0, u)
    assert o["idx"][0].tolist() == [0, 1, 2, -1]
    # temperature moves the cut: the kept set shrinks as T falls
    zt = np.array([2.0, 1.0, 0.0, -1.0, -2.0, 0.5], np.float32)
    counts = [oracle.sparsify(zt[None], 6, 0.8, T, u)["count"][0] for T in (2.0, 1.0, 0.5, 0.25)]
    assert counts == sorted(counts, reverse=True) and counts[0] > counts[-1]
    for T in (2.0, 1.0, 0.5):
        q = softmax64(zt, T)
        order = sorted(range(6), key=lambda i: (-zt[i], i))
        c = np.cumsum(q[order])
        n_star = int(np.argmax(c >= 0.8)) + 1
        assert oracle.sparsify(zt[None], 6, 0.8, T, u)["count"][0] == n_star


def test_inverse_cdf_conventions():
    V = 8
    probs = np.array([0.0, 0.2, 0.0, 0.3, 0.1, 0.0, 0.4, 0.0])
    with np.errstate(divide="ignore"):
        z = np.log(probs).astype(np.float32)  # zeros become -inf: never selected, probability 0
    one_m = np.nextafter(np.float32(1), np.float32(0))

    def tok(u):
        return oracle.sparsify(z[None], V, 1.0, 1.0, np.array([[u]], np.float32))["token"][0, 0]

    assert tok(0.0) == 1            # u = 0: first item with positive mass
    assert tok(one_m) == 6          # u just below 1: last item with positive mass
    assert tok(1.0) == 6 and tok(7.0) == 6   # u >= 1 is clamped below 1
    # step function by brute force: first index whose cumulative exceeds u
    c = np.cumsum(softmax64(z))
    for u in np.linspace(0.001, 0.999, 400, dtype=np.float32):
        expect = int(np.argmax(c > float(u)))
        assert tok(u) == expect
    # the same convention for the verifier's bonus row
    tgt = np.stack([z, z])[None]
    sp = oracle.sparsify(z[None], V, 1.0, 1.0, np.array([[0.5]], np.float32))
    for u, expect in [(0.0, 1), (one_m, 6), (0.19, 1), (0.21, 3)]:
        o = oracle.verify(tgt, sp["idx"][None], sp["logit"][None], sp["count"][None],
                          sp["token"].reshape(1, 1), 1.0, 1.0, np.array([[0.0]], np.float32),
                          np.array([u], np.float32))
        assert o["accepted_len"][0] == 1 and o["out_token"][0] == expect
    # near-boundary flag for sampling
    cq = float(np.cumsum(softmax64(z))[1])
    near = oracle.sparsify(z[None], V, 1.0, 1.0, np.array([[np.float32(cq) + np.float32(3e-7)]], np.float32))
    far = oracle.sparsify(z[None], V, 1.0, 1.0, np.array([[np.float32(cq) + np.float32(1e-3)]], np.float32))
    assert near["flags"][0] & oracle.FLAG_SMP and not (far["flags"][0] & oracle.FLAG_SMP)


def test_verify_strict_compare_and_rejection_position():
    """r < min(1, p/q~) is strict; positions after the first rejection are ignored."""
    V = 4
    q = np.array([0.5, 0.5, 0.0, 0.0])
    p = np.array([0.25, 0.25, 0.25, 0.25])
    with np.errstate(divide="ignore"):
        zq = np.log(q).astype(np.float32)
    zp = np.log(p).astype(np.float32)
    gamma = 3
    sp = oracle.sparsify(np.repeat(zq[None], gamma, 0), 2, 1.0, 1.0, np.zeros((gamma, 1), np.float32))
    assert sp["idx"][0].tolist() == [0, 1]
    tgt = np.repeat(zp[None], gamma + 1, 0)[None]
    toks = np.zeros((1, gamma), np.int32)

    def run(ua, us=0.0):
        return oracle.verify(tgt, sp["idx"][None], sp["logit"][None], sp["count"][None], toks, 1.0,
                             1.0, np.array([ua], np.float32), np.array([us], np.float32),
                             want_dense=True)

    o = run([0.4, 0.4, 0.4])
    assert np.allclose(o["accept_prob"], 0.5) and o["accepted_len"][0] == 3
    o = run([0.4, 0.5, 0.0])  # r == ratio is a rejection; the later 0.0 is never looked at
    assert o["accepted_len"][0] == 1
    # residual: max(0, p - q~) = [0, 0, .25, .25] -> tokens 2, 3 with equal mass
    assert np.allclose(o["final_pmf"][0], [0, 0, 0.5, 0.5])
    assert run([0.4, 0.5, 0.0], us=0.49)["out_token"][0] == 2
    assert run([0.4, 0.5, 0.0], us=0.51)["out_token"][0] == 3
    assert run([0.9, 0.0, 0.0])["accepted_len"][0] == 0
    # a token with p = 0 is never accepted, a ratio >= 1 always is
    zp2 = zp.copy(); zp2[0] = -np.inf
    tgt2 = np.repeat(zp2[None], gamma + 1, 0)[None]
    o = oracle.verify(tgt2, sp["idx"][None], sp["logit"][None], sp["count"][None], toks, 1.0, 1.0,
                      np.zeros((1, gamma), np.float32), np.array([0.0], np.float32))
    assert o["accepted_len"][0] == 0 and o["accept_prob"][0, 0] == 0.0
    # boundary flag on the acceptance test
    o = run([0.5 - 3e-7, 0.9, 0.9])
    assert o["flags"][0] & oracle.FLAG_ACC
    assert not (run([0.4, 0.9, 0.9])["flags"][0] & oracle.FLAG_ACC)


# --------------------------------------------------------------------------------------
# multi-candidate / tree
# --------------------------------------------------------------------------------------

def mc_reference(p, q, xs):
    """Algorithm 5 written out with numpy: acceptance chain and final residual for candidates xs."""
    p = p.copy()
    accs = []
    for x in xs:
        a = min(1.0, p[x] / q[x]) if q[x] > 0 else (1.0 if p[x] > 0 else 0.0)
        accs.append(a)
        r = np.maximum(p - q, 0)
        if r.sum() > 0:
            p = r / r.sum()
    return accs, p


@pytest.mark.parametrize("seed,V,K,k", [(41, 8, 4, 3), (42, 10, 3, 2), (43, 8, 8, 2)])
def test_multi_candidate_lossless_enumeration(seed, V, K, k):
    """Over all K^k candidate tuples (drawn iid from q~), the law of the first emitted token is p."""
    zq, zp = tiny_case(seed, V)
    sp = sparsify_row(zq, K, 1.0, 1.0)
    qt = sp["qtilde"][0]
    S = sp["idx"][0, :sp["count"][0]]
    p = softmax64(zp)
    parent, ndr, M, depth = synth.complete_tree([k])
    N = len(parent)
    rng = np.random.default_rng(seed)
    leaf_rows = rng.normal(size=(N - 1, V)).astype(np.float32)
    tgt = np.concatenate([zp[None], leaf_rows], 0)[None]
    one_m = np.nextafter(np.float32(1), np.float32(0))
    law = np.zeros(V)
    theta = 0.0
    for xs in itertools.product(S.tolist(), repeat=k):
        w = float(np.prod(qt[list(xs)]))
        toks = np.array([[0] + list(xs)], np.int32)
        # u_accept just below 1 rejects every candidate whose acceptance probability is < 1, so
        # the oracle reports the whole chain a_1..a_k (or stops at an a_i = 1, after which the
        # remaining candidates carry no weight)
        o = oracle.tree_verify(tgt, parent, ndr, toks, sp["idx"][None], sp["logit"][None],
                               sp["count"][None], 1.0, 1.0, np.full((1, N), one_m, np.float32),
                               np.full((1, N), 0.5, np.float32), depth, want_dense=True)
        ref_acc, ref_final = mc_reference(p, qt, xs)
        surv = 1.0
        for i, x in enumerate(xs):
            a = o["accept_prob"][0, 1 + i]
            assert a == pytest.approx(ref_acc[i], abs=1e-12)
            law[x] += w * surv * a
            theta += w * surv * a
            surv *= (1 - a)
            if a >= 1.0:
                break
        if surv > 0:
            assert o["accepted_len"][0] == 0
            assert np.allclose(o["final_pmf"][0], ref_final, atol=1e-12)
            law += w * surv * o["final_pmf"][0]
    assert np.allclose(law, p, atol=1e-12), (law, p)
    # total acceptance theta = beta1 + sum beta_i prod (1 - beta_j) with beta^(j) = sum min(q, p^(j))
    # holds per tuple chain in expectation only for k = 1; check k-independent first term instead
    beta1 = np.minimum(qt, p).sum()
    first = sum(float(qt[x]) * min(1.0, p[x] / qt[x]) for x in S)
    assert first == pytest.approx(beta1, abs=1e-12)
    assert theta >= beta1 - 1e-12


def test_multi_candidate_acceptance_monte_carlo():
    """Empirical per-candidate and total acceptance vs beta^(j) = sum min(q~, p^(j)) and theta
    with p^(j) the j-fold residual (valid as written when rejected candidates leave p^(j)
    dependent only on j, i.e. computed from the same q~ each time)."""
    V, K, k, n = 12, 5, 3, 400_000
    zq, zp = tiny_case(51, V)
    sp1 = sparsify_row(zq, K, 1.0, 1.0)
    qt = sp1["qtilde"][0]
    p = softmax64(zp)
    betas, pj = [], p.copy()
    for _ in range(k):
        betas.append(np.minimum(qt, pj).sum())
        r = np.maximum(pj - qt, 0)
        pj = r / r.sum()
    theta = betas[0] + sum(betas[i] * np.prod([1 - b for b in betas[:i]]) for i in range(1, k))
    parent, ndr, M, depth = synth.complete_tree([k])
    N = len(parent)
    ud = synth.uniforms((n, k), 9, synth.TID_U_DRAFT).numpy()
    sp = oracle.sparsify(zq[None], K, 1.0, 1.0, ud, row_stride=0, rows=n)
    toks = np.concatenate([np.zeros((n, 1), np.int32), sp["token"]], 1)
    rng = np.random.default_rng(3)
    leaf = rng.normal(size=(N - 1, V)).astype(np.float32)
    tgt = np.ascontiguousarray(np.broadcast_to(np.concatenate([zp[None], leaf], 0)[None], (n, N, V)))
    ua = synth.uniforms((n, N), 9, synth.TID_U_ACCEPT).numpy()
    us = synth.uniforms((n, N), 9, synth.TID_U_SAMPLE).numpy()
    o = oracle.tree_verify(tgt, parent, ndr, toks, sp["idx"][:, None], sp["logit"][:, None],
                           sp["count"][:, None], 1.0, 1.0, ua, us, depth)
    acc_any = (o["accepted_len"] == 1).mean()
    sd = math.sqrt(theta * (1 - theta) / n)
    assert abs(acc_any - theta) < 4 * sd, (acc_any, theta)
    first = (o["accepted_path"][:, 0] == 1).mean()
    assert abs(first - betas[0]) < 4 * math.sqrt(betas[0] * (1 - betas[0]) / n)
    # law of the first emitted token is p
    emitted = np.where(o["accepted_len"] == 1,
                       toks[np.arange(n), np.maximum(o["accepted_path"][:, 0], 0)], o["out_token"])
    # when a child is accepted the final out_token is the leaf's bonus token, the emitted first
    # token is the child's own token
    emp = np.bincount(emitted, minlength=V) / n
    assert np.abs(emp - p).max() < 5 * math.sqrt(0.25 / n)


def test_two_level_tree_walk_and_leaf_bonus():
    """Depth-2 tree, V = 8: the walk follows accepted children, stops at the first node whose
    children are all rejected, and a reached leaf emits a bonus token from its own target row."""
    V, K = 8, 4
    parent, ndr, M, depth = synth.complete_tree([2, 2])
    N = len(parent)
    assert parent == [-1, 0, 0, 1, 1, 2, 2] and ndr == [0, 1, 2, -1, -1, -1, -1] and M == 3
    rng = np.random.default_rng(61)
    zq = (rng.normal(size=(M, V)) * 2).astype(np.float32)
    zp = (rng.normal(size=(N, V)) * 2).astype(np.float32)
    sp = oracle.sparsify(zq, K, 1.0, 1.0, rng.random((M, 2), dtype=np.float32))
    toks = np.zeros((1, N), np.int32)
    for n in range(N):
        if ndr[n] >= 0:
            ch = [c for c in range(N) if parent[c] == n]
            toks[0, ch] = sp["token"][ndr[n]]
    P = softmax64(zp)

    def run(ua, us):
        return oracle.tree_verify(zp[None], parent, ndr, toks, sp["idx"][None], sp["logit"][None],
                                  sp["count"][None], 1.0, 1.0, np.asarray(ua, np.float32)[None],
                                  np.asarray(us, np.float32)[None], depth, want_dense=True)

    zero, one_m = 0.0, float(np.nextafter(np.float32(1), np.float32(0)))
    # accept-everything uniforms (u = 0 accepts whenever p(x) > 0): path 0 -> 1 -> 3, leaf bonus ~ P_3
    o = run([zero] * N, [0.5] * N)
    assert o["accepted_path"][0].tolist() == [1, 3] and o["accepted_len"][0] == 2
    assert np.allclose(o["final_pmf"][0], P[3], atol=1e-14)
    assert o["out_token"][0] == int(np.argmax(np.cumsum(P[3]) > 0.5))
    # the sampling uniform is the stop node's own entry of u_sample
    us = [0.999] * N; us[3] = 0.0
    assert run([zero] * N, us)["out_token"][0] == 0
    us = [0.0] * N; us[3] = 0.999
    assert run([zero] * N, us)["out_token"][0] == int(np.argmax(np.cumsum(P[3]) > np.float32(0.999)))
    # reject child 1 at the root, accept child 2, then reject both of its children
    ua = [zero] * N
    ua[1] = one_m; ua[5] = one_m; ua[6] = one_m
    o = run(ua, [0.5] * N)
    accs, _ = mc_reference(P[0], oracle_dense(sp, 0, V), [toks[0, 1], toks[0, 2]])
    if accs[0] < 1 and accs[1] > 0:
        assert o["accepted_path"][0, 0] == 2
        accs2, fin2 = mc_reference(P[2], oracle_dense(sp, 2, V), [toks[0, 5], toks[0, 6]])
        if accs2[0] < 1 and accs2[1] < 1:
            assert o["accepted_len"][0] == 1 and o["accepted_path"][0, 1] == -1
            assert np.allclose(o["final_pmf"][0], fin2, atol=1e-13)
            # the uniform used for the final token is the stop node's own
            us = [0.5] * N; us[2] = 0.0
            first_pos = int(np.argmax(fin2 > 0))
            assert run(ua, us)["out_token"][0] == first_pos
    # conditional law: given the prefix accepted so far, emitted-token law at a node is that node's p
    for node in (0, 1, 2):
        qd = oracle_dense(sp, ndr[node], V)
        ch = [c for c in range(N) if parent[c] == node]
        S = np.nonzero(qd)[0]
        law = np.zeros(V)
        for xs in itertools.product(S.tolist(), repeat=len(ch)):
            accs, fin = mc_reference(P[node], qd, xs)
            w, surv = float(np.prod(qd[list(xs)])), 1.0
            for x, a in zip(xs, accs):
                law[x] += w * surv * a
                surv *= 1 - a
            law += w * surv * fin
        assert np.allclose(law, P[node], atol=1e-12)


def oracle_dense(sp, row, V):
    d = np.zeros(V)
    n = sp["count"][row]
    l = sp["logit"][row, :n].astype(np.float64)
    w = np.exp(l - l.max())
    d[sp["idx"][row, :n]] = w / w.sum()
    return d


def test_duplicate_candidates_still_update_residual():
    """Children are drawn with replacement (Section 4.2): a repeated, already rejected token has
    zero residual mass, is rejected again, and the update is applied again."""
    V = 6
    q = np.array([0.7, 0.3, 0, 0, 0, 0.0])
    p = np.array([0.1, 0.2, 0.3, 0.2, 0.1, 0.1])
    with np.errstate(divide="ignore"):
        zq = np.log(q).astype(np.float32)
    zp = np.log(p).astype(np.float32)
    parent, ndr, M, depth = synth.complete_tree([3])
    N = len(parent)
    sp = oracle.sparsify(zq[None], 2, 1.0, 1.0, np.zeros((1, 1), np.float32))
    toks = np.array([[0, 0, 0, 1]], np.int32)  # candidate 0 twice, then 1
    tgt = np.concatenate([zp[None], np.zeros((3, V), np.float32)], 0)[None]
    one_m = np.nextafter(np.float32(1), np.float32(0))
    o = oracle.tree_verify(tgt, parent, ndr, toks, sp["idx"][None], sp["logit"][None],
                           sp["count"][None], 1.0, 1.0, np.full((1, N), one_m, np.float32),
                           np.full((1, N), 0.5, np.float32), depth, want_dense=True)
    qt = oracle_dense(sp, 0, V)
    accs, fin = mc_reference(softmax64(zp), qt, [0, 0, 1])
    assert accs[1] == 0.0  # the duplicate has no residual mass left
    assert np.allclose(o["accept_prob"][0, 1:], accs, atol=1e-12)
    assert np.allclose(o["final_pmf"][0], fin, atol=1e-12)
    assert o["accepted_len"][0] == 0


def test_golden_paper_values():
    """Closed-form quantities the paper states (tests/golden/paper_values.txt)."""
    vals = {}
    with open(os.path.join(os.path.dirname(__file__), "golden", "paper_values.txt")) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                key, v = [s.strip() for s in line.split("=")]
                vals[key] = v
    assert math.ceil(math.log2(32000)) == int(vals["index_bits_V32000"])
    assert 32000 * 16 == int(vals["payload_bits_full_V32000_fp16_prob_only"])
    for exp, key in (((2, 2, 2), "num_distributions_expansion_2_2_2"),
                     ((3, 3, 3), "num_distributions_expansion_3_3_3")):
        parent, ndr, M, depth = synth.complete_tree(exp)
        assert M == int(vals[key])
    parent, ndr, M, depth = synth.complete_tree((2, 2, 2))
    widths, level = [], [0]
    while level:
        widths.append(len(level))
        level = [c for c in range(len(parent)) if parent[c] in level]
    assert widths == [int(x) for x in vals["layer_widths_expansion_2_2_2"].split(",")]


def test_argument_errors():
    z = np.zeros((1, 8), np.float32)
    u = np.zeros((1, 1), np.float32)
    for k, top_p, T in [(0, 1.0, 1.0), (9, 1.0, 1.0), (2, 0.0, 1.0), (2, 1.0, 0.0)]:
        with pytest.raises(ValueError):
            oracle.sparsify(z, k, top_p, T, u)


def test_degenerate_residual_falls_back_to_the_target():
    """The one branch exact arithmetic never reaches from a well-formed round: the residual mass is
    zero.  Built by hand: the target equals the truncated draft on S (p = q~ there, -inf elsewhere)
    and the drafted token lies outside S, so it is rejected whatever the uniform (p(x) = 0) and
    max(0, p - q~) vanishes everywhere.  The oracle must flag DEGEN and sample the unmodified p by
    the usual inverse CDF (brute force below)."""
    V, k = 8, 3
    S = np.array([1, 3, 5], np.int32)
    lg = np.array([0.5, 1.25, -0.75], np.float32)          # exactly representable: p == q~ bit for bit
    zp = np.full((1, 2, V), -np.inf, np.float32)
    zp[0, 0, S] = lg
    zp[0, 1] = np.arange(V, dtype=np.float32)               # bonus row, unused
    idx, logit, count = S[None, None, :], lg[None, None, :], np.array([[k]], np.int32)
    p = softmax64(lg)
    cdf = np.cumsum(p)
    for u in (0.0, 0.3, float(cdf[0]) + 1e-3, 0.999):
        o = oracle.verify(zp, idx, logit, count, np.array([[0]], np.int32), 1.0, 1.0,
                          np.array([[0.0]], np.float32), np.array([u], np.float32), want_dense=True)
        assert o["accepted_len"][0] == 0 and o["accept_prob"][0, 0] == 0.0
        assert o["flags"][0] & oracle.FLAG_DEGEN
        assert o["out_token"][0] == S[int(np.searchsorted(cdf, u, side="right"))]
        assert np.allclose(o["final_pmf"][0, S], p, atol=1e-15) and o["final_pmf"][0].sum() == pytest.approx(1.0)
    # the same payload with a token inside S is an ordinary round: accepted with probability 1, no flag
    o = oracle.verify(zp, idx, logit, count, np.array([[3]], np.int32), 1.0, 1.0,
                      np.array([[0.5]], np.float32), np.array([0.5], np.float32))
    assert o["accepted_len"][0] == 1 and not (o["flags"][0] & oracle.FLAG_DEGEN)


def test_truncation_of_a_row_from_its_vocabulary_shards():
    """What the sharded two-stage form rests on, checked on the oracle alone: the k best tokens of a row
    (logit descending, index ascending) are among the k best of their own shards, and the row's
    normaliser is the sum of the shards' (Section 3.1's truncation equation needs nothing else of the
    row).  Shards are ragged; one holds fewer than k finite logits, one holds ties that straddle the cut."""
    rng = np.random.default_rng(12)
    V, k, T = 3000, 40, 0.8
    z = rng.normal(size=(3, V)).astype(np.float32) * 2.0
    z[0, 1000:1990] = -np.inf            # a shard with 10 finite logits
    z[1, 2100:2160] = z[1].max() + 1.0   # 60 ties at the top, all in the last shard: the cut falls among them
    bounds = [0, 7, 1000, 2000, V]
    u = np.zeros((3, 1), np.float32)
    whole = oracle.sparsify(z, k, 1.0, T, u)
    cand_idx, cand_logit, lses = [], [], []
    for a, b in zip(bounds, bounds[1:]):
        part = oracle.sparsify(np.ascontiguousarray(z[:, a:b]), min(k, b - a), 1.0, T, u)
        cand_idx.append(np.where(part["idx"] >= 0, part["idx"] + a, -1))
        cand_logit.append(part["logit"])
        lses.append(part["lse"])
    ci, cl = np.concatenate(cand_idx, 1), np.concatenate(cand_logit, 1)
    for r in range(3):
        keep = ci[r] >= 0
        order = np.lexsort((ci[r][keep], -cl[r][keep].astype(np.float64)))[:k]
        merged = np.sort(ci[r][keep][order])
        n = int(whole["count"][r])
        assert np.array_equal(merged[:n], whole["idx"][r, :n]) and len(merged) == n
    lse = scipy.special.logsumexp(np.stack(lses, 1), axis=1)
    assert np.allclose(lse, whole["lse"], rtol=1e-12, atol=1e-12)
