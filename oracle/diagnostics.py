"""Plain numpy oracle of the truncation diagnostics (TEST INFRASTRUCTURE ONLY; the product path
never imports this file, and this file imports nothing of the product).

What it computes, per pair of rows (draft logits z_q, target logits z_p), straight from the
definitions, dense over the whole vocabulary, in fp64:

  q = softmax(z_q / T_q), p = softmax(z_p / T_p)
  for every K of a list: V' = the first K tokens in the order (q descending, index ascending)
      rho(K)   = sum_{V'} q                      retained mass (Section 5's top-K mass curve; Theorem 1)
      sigma(K) = 1 - rho(K)                      truncated mass
      q^_K     = q / rho on V', 0 elsewhere      the truncation equation of Section 3.1 (cases the right way round)
      beta^(j) = sum_v min(q, p^(j)),  p^(1) = p,  p^(j+1) = norm(max(0, p^(j) - q))
                                                 acceptance rate of the j-th candidate (Section 4.3), and the
                                                 same with q^_K in place of q: beta_hat^(j)(K)
      Z^(j+1)  = sum_v max(0, p^(j) - q)         the normaliser that makes p^(j+1) (appendix, recursive TV lemma)
      theta    = beta^(1) + sum_{i>=2} beta^(i) prod_{j<i} (1 - beta^(j))     total acceptance (Section 4.3)
  beta = beta^(1) = sum min(q, p) = 1 - TV(q, p)   (the acceptance-rate lemma of Section 3.2)

No blocking, no sparse tricks: every quantity is a V-wide numpy expression a reader can hold against
the paper.  Pins: tests/test_diagnostics_oracle.py.
"""
from __future__ import annotations

import numpy as np


def softmax64(z, T):
    x = np.asarray(z, np.float64) / float(T)
    fin = np.isfinite(x)
    m = x[fin].max()
    e = np.where(fin, np.exp(np.where(fin, x, m) - m), 0.0)
    return e / e.sum()


def order_desc(z):
    """Finite entries in the order (logit descending, index ascending)."""
    z = np.asarray(z, np.float64)
    fin = np.nonzero(np.isfinite(z))[0]
    return fin[np.lexsort((fin, -z[fin]))]


def candidate_chain(q, p, c):
    """beta^(1..c), Z^(2..c+1) and theta for draft distribution q (dense) against target p."""
    betas, zs = [], []
    r = p.copy()
    for _ in range(c):
        betas.append(float(np.minimum(q, r).sum()))
        d = np.maximum(0.0, r - q)
        Z = float(d.sum())
        zs.append(Z)
        r = d / Z if Z > 0.0 else r
    theta, stay = 0.0, 1.0
    for b in betas:
        theta += stay * b
        stay *= 1.0 - b
    return np.array(betas), np.array(zs), theta


def row(zq, zp, k_list, num_candidates, Tq=1.0, Tp=1.0):
    q, p = softmax64(zq, Tq), softmax64(zp, Tp)
    order = order_desc(zq)
    beta_j, z_j, theta = candidate_chain(q, p, num_candidates)
    out = dict(beta=beta_j[0], beta_j=beta_j, z_j=z_j, theta=theta, rho=[], beta_hat_j=[], theta_hat=[])
    for K in k_list:
        S = order[:min(int(K), len(order))]
        rho = float(q[S].sum())
        qh = np.zeros_like(q)
        qh[S] = q[S] / rho
        bh, _, th = candidate_chain(qh, p, num_candidates)
        out["rho"].append(rho)
        out["beta_hat_j"].append(bh)
        out["theta_hat"].append(th)
    out["rho"] = np.array(out["rho"])
    out["beta_hat_j"] = np.array(out["beta_hat_j"])
    out["theta_hat"] = np.array(out["theta_hat"])
    return out


def diagnostics(zq_rows, zp_rows, k_list, num_candidates, Tq=1.0, Tp=1.0):
    """zq_rows, zp_rows [rows, V] (float arrays; bf16 inputs are upcast by the caller).  Returns dict of
    arrays: beta [rows], beta_j, z_j [rows, c], theta [rows], rho, theta_hat [rows, nK],
    beta_hat_j [rows, nK, c]."""
    rows = [row(a, b, k_list, num_candidates, Tq, Tp) for a, b in zip(np.asarray(zq_rows, np.float64), np.asarray(zp_rows, np.float64))]
    return {key: np.array([r[key] for r in rows]) for key in rows[0]}


def theorem2_bound(z_j, sigma, j):
    """Right-hand side of Theorem 2 for the j-th candidate (1-based): [sum_{k=1}^{j-1} prod_{s=k+1}^{j}
    2 / Z^(s) + 1] sigma, with Z^(s) = z_j[s - 2] (z_j[0] is Z^(2))."""
    total = 1.0
    for k in range(1, j):
        prod = 1.0
        for s in range(k + 1, j + 1):
            prod *= 2.0 / z_j[s - 2]
        total += prod
    return total * sigma
