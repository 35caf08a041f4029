"""CPU evaluation tool (test infrastructure, fp64): acceptance rates of RRS, RRSw, OTM, OTMw and
SpecHub on small random distributions, after the toy comparison of the paper's appendix
"Comparing SpecHub to OTM in Toy Settings" (Table "Acceptance Rates for Toy Experiments").

Recipe as stated there: |V| = 50, u_p, u_q ~ Unif(0,1)^V, p = softmax(u_p / T),
q = softmax((lambda u_p + (1 - lambda) u_q) / T), averaged over 100 pairs.

Every column is computed exactly here (the paper samples RRSw by Monte Carlo):
  RRS, RRSw  1 - P(both drafts rejected) from Algorithm 1's residual masses;
  SpecHub    1 - R, R the mass of SpecHub's final residual (Section 4);
  OTM, OTMw  the optimum of the simplified LP of Section 3 with Q = q x q, or Q = q(x1) q(x2) /
             (1 - q(x1)) off the diagonal (drafts without replacement).

The printed table is parity unpinned: with the stated recipe the RRS / RRSw / SpecHub columns do
not reproduce the paper's digits (nor with normal logits), so the table is a tool for that
question, not a test fixture.  What the functions compute is pinned in tests/test_toy_table.py.

    python -m oracle.toy_table [--pairs 100] [--vocab 50] [--seed 0]
"""
from __future__ import annotations

import argparse

import numpy as np

from . import oracle as orc

PAPER_GRID = [(0.1, 0.7), (0.1, 0.5), (0.25, 0.7), (0.25, 0.5), (0.5, 0.7), (0.5, 0.5)]


def toy_pair(rng, V, T, lam):
    """One (p, q) of the toy recipe, as fp64 probability vectors."""
    up, uq = rng.random(V), rng.random(V)
    zp = up / T
    zq = (lam * up + (1.0 - lam) * uq) / T
    p = np.exp(zp - zp.max()); p /= p.sum()
    q = np.exp(zq - zq.max()); q /= q.sum()
    return p, q


def acceptance_spechub(p, q):
    """1 - R for SpecHub's coupling (any valid pair gives the row's rates)."""
    a = int(np.argmax(q))
    x = 0 if a != 0 else 1
    node = orc.spechub_verify(p, q, a, x, a, 0.5, 0.5, 0.5)
    return 1.0 - float(node["rate"][2])


def acceptance_rrs(p, q, without_replacement):
    """P(one of the two drafts is accepted) under Algorithm 1, exactly.

    The first draft x1 ~ q is rejected with mass max(q(x1) - p(x1), 0); after that the second
    stage rejects with probability W2(x1) / A1, A1 = sum max(p - q, 0) and W2(x1) the mass of the
    residual after two rejections (for RRS it does not depend on x1)."""
    A1 = float(np.maximum(p - q, 0.0).sum())
    if A1 <= 0.0:
        return 1.0
    if not without_replacement:
        W2 = float(orc.rrs_residual(p, q, 0, False).sum())
        return 1.0 - W2
    rej = 0.0
    for x1 in range(len(p)):
        m = max(q[x1] - p[x1], 0.0)
        if m > 0.0:
            rej += m * float(orc.rrs_residual(p, q, x1, True).sum()) / A1
    return 1.0 - rej


def pair_law(q, without_replacement):
    """Q(x1, x2) of two drafts from q, independent or without replacement."""
    if not without_replacement:
        return np.outer(q, q)
    Q = np.outer(q, q)
    np.fill_diagonal(Q, 0.0)
    rest = 1.0 - q
    with np.errstate(divide="ignore", invalid="ignore"):
        Q = np.where(rest[:, None] > 0.0, Q / rest[:, None], 0.0)
    return Q


def acceptance_lp(p, Q):
    """Optimum of the simplified LP (k = 2): maximise the mass sent to a drafted token,
    sum_i pi(x1, x2 -> x_i) <= Q(x1, x2) for every pair and what reaches y <= p(y)."""
    from scipy.optimize import linprog
    from scipy.sparse import coo_matrix

    V = len(p)
    pairs = [(i, j) for i in range(V) for j in range(V) if Q[i, j] > 0.0]
    rows, cols, cap = [], [], []
    nvar = 0
    for r, (i, j) in enumerate(pairs):
        targets = (i,) if i == j else (i, j)   # a doubled draft has one token to accept
        for y in targets:
            rows += [r, len(pairs) + y]
            cols += [nvar, nvar]
            nvar += 1
        cap.append(Q[i, j])
    A = coo_matrix((np.ones(len(rows)), (rows, cols)), shape=(len(pairs) + V, nvar)).tocsr()
    b = np.concatenate([np.asarray(cap), np.asarray(p, np.float64)])
    res = linprog(-np.ones(nvar), A_ub=A, b_ub=b, bounds=(0, None), method="highs")
    if res.status != 0:
        raise RuntimeError("LP did not solve: %s" % res.message)
    return float(-res.fun)


def acceptance_otm(p, q, without_replacement):
    return acceptance_lp(p, pair_law(q, without_replacement))


COLUMNS = ("RRS", "RRSw", "OTM", "OTMw", "SpecHub")


def row(p, q):
    return (acceptance_rrs(p, q, False), acceptance_rrs(p, q, True), acceptance_otm(p, q, False),
            acceptance_otm(p, q, True), acceptance_spechub(p, q))


def table(pairs=100, V=50, seed=0, grid=PAPER_GRID):
    """Mean acceptance per (T, lambda) over `pairs` toy pairs.  Returns {(T, lambda): 5 floats}."""
    out = {}
    for gi, (T, lam) in enumerate(grid):
        rng = np.random.Generator(np.random.PCG64(seed + 7919 * gi))
        acc = np.zeros(len(COLUMNS))
        for _ in range(pairs):
            acc += np.asarray(row(*toy_pair(rng, V, T, lam)))
        out[(T, lam)] = tuple(acc / pairs)
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--pairs", type=int, default=100)
    ap.add_argument("--vocab", type=int, default=50)
    ap.add_argument("--seed", type=int, default=0)
    a = ap.parse_args()
    t = table(a.pairs, a.vocab, a.seed)
    print("%-6s %-6s " % ("T", "lambda") + " ".join("%-8s" % c for c in COLUMNS))
    for (T, lam), vals in t.items():
        print("%-6g %-6g " % (T, lam) + " ".join("%-8.4f" % v for v in vals))


if __name__ == "__main__":
    main()
