"""Pins for oracle/diagnostics.py: held against what the paper and the mathematics fix, not against
itself or the CUDA path.
* the acceptance-rate lemma of Section 3.2: beta = 1 - TV(q, p), with TV written out here;
* Theorem 1: TV(q^, q) = sigma exactly and |beta^ - beta| <= sigma;
* Theorem 2's inequality for every candidate j, with Z^(s) as the residual normalisers;
* theta: Monte Carlo through the C oracle's multi-candidate verification (a one-level tree of c
  children drafted iid from q^): the frequency of "some child accepted" is theta^;
* closed forms: K = V gives rho = 1 and beta^ = beta; identical models give beta = 1;
* the mass curve is non-decreasing in K, and rho(K) is the sum of the K largest q (numpy sort).
"""
import numpy as np
import pytest
import torch

import oracle
from oracle import diagnostics as D
from paper_2512_16273_b200 import synth


def rows(seed, n=3, V=400):
    zq, zp = synth.sequence_logits(1, n, V, torch.float32, 0.5, seed, "cpu")
    return zq[0].numpy(), zp[0, :n].numpy()


def test_lemma_beta_is_one_minus_tv_and_theorem1():
    zq, zp = rows(1)
    ks = [1, 4, 32, 100, 400]
    d = D.diagnostics(zq, zp, ks, 3, 0.9, 1.1)
    for r in range(len(zq)):
        q, p = D.softmax64(zq[r], 0.9), D.softmax64(zp[r], 1.1)
        assert d["beta"][r] == pytest.approx(1.0 - 0.5 * np.abs(q - p).sum(), abs=1e-13)
        srt = np.sort(q)[::-1]
        for i, K in enumerate(ks):
            rho = d["rho"][r, i]
            assert rho == pytest.approx(srt[:K].sum(), rel=1e-13)          # the K largest q, by numpy's sort
            sigma = 1.0 - rho
            S = D.order_desc(zq[r])[:K]
            qh = np.zeros_like(q); qh[S] = q[S] / rho
            assert 0.5 * np.abs(qh - q).sum() == pytest.approx(sigma, abs=1e-13)   # Theorem 1: TV(Q^, Q) = sigma
            assert abs(d["beta_hat_j"][r, i, 0] - d["beta"][r]) <= sigma + 1e-13   # Theorem 1: |beta^ - beta| <= sigma
        assert (np.diff(d["rho"][r]) >= -1e-15).all()
        assert d["rho"][r, -1] == pytest.approx(1.0, abs=1e-13)
        assert d["beta_hat_j"][r, -1] == pytest.approx(d["beta_j"][r], abs=1e-13)  # K = V: nothing truncated
        assert d["theta_hat"][r, -1] == pytest.approx(d["theta"][r], abs=1e-13)


def test_theorem2_inequality_and_z_identity():
    zq, zp = rows(2, n=4, V=300)
    ks = [2, 8, 50, 150]
    c = 4
    d = D.diagnostics(zq, zp, ks, c)
    for r in range(len(zq)):
        # Z^(j+1) = 1 - beta^(j): what a rejection leaves (appendix, proof of the recursive TV lemma)
        assert d["z_j"][r] == pytest.approx(1.0 - d["beta_j"][r], abs=1e-13)
        for i, K in enumerate(ks):
            sigma = 1.0 - d["rho"][r, i]
            for j in range(1, c + 1):
                lhs = abs(d["beta_hat_j"][r, i, j - 1] - d["beta_j"][r, j - 1])
                assert lhs <= D.theorem2_bound(d["z_j"][r], sigma, j) + 1e-12, (r, K, j)


def test_identical_models():
    zq, _ = rows(3)
    d = D.diagnostics(zq, zq, [5, 400], 2)
    assert d["beta"] == pytest.approx(np.ones(len(zq)), abs=1e-13)
    assert d["theta"] == pytest.approx(np.ones(len(zq)), abs=1e-13)
    # truncated draft against the untruncated target: beta^ = sum min(q/rho, q) = rho
    assert d["beta_hat_j"][:, 0, 0] == pytest.approx(d["rho"][:, 0], abs=1e-13)


def test_theta_hat_by_monte_carlo_through_the_c_oracle():
    """theta^ is the probability that one of c candidates drawn iid from q^ is accepted by the
    sequential multi-candidate test.  Counted here with the C oracle's tree verification."""
    V, K, c, n = 64, 6, 3, 60000
    zq, zp = rows(7, n=1, V=V)
    want = D.diagnostics(zq, zp, [K], c)["theta_hat"][0, 0]
    rng = np.random.default_rng(0)
    sp = oracle.sparsify(zq.astype(np.float32), K, 1.0, 1.0, rng.random((1, c * n), dtype=np.float32))
    toks = sp["token"][0].reshape(n, c)
    parent, ndr = [-1] + [0] * c, [0] + [-1] * c
    N = c + 1
    zt = np.zeros((n, N, V), np.float32)
    zt[:, 0] = zp[0]
    node_token = np.zeros((n, N), np.int32); node_token[:, 1:] = toks
    o = oracle.tree_verify(zt, parent, ndr, node_token, np.tile(sp["idx"], (n, 1, 1)), np.tile(sp["logit"], (n, 1, 1)),
                           np.tile(sp["count"], (n, 1)), 1.0, 1.0, rng.random((n, N), dtype=np.float32),
                           rng.random((n, N), dtype=np.float32), 1)
    got = (o["accepted_len"] >= 1).mean()
    assert abs(got - want) < 4.0 * np.sqrt(want * (1 - want) / n) + 1e-4, (got, want)
