"""Pins of the CPU evaluation tool oracle/toy_table.py (acceptance rates of RRS, RRSw, OTM, OTMw
and SpecHub on small distributions; the paper's appendix "Comparing SpecHub to OTM in Toy
Settings").  The table's digits themselves are parity unpinned; what is pinned here is what each
column computes."""
import numpy as np
import pytest

import oracle
from oracle import toy_table as tt


def rand_pair(rng, V, conc=1.0):
    return rng.dirichlet(np.full(V, conc)), rng.dirichlet(np.full(V, conc))


@pytest.mark.parametrize("without", [False, True])
def test_rrs_acceptance_matches_simulation_of_algorithm_1(without):
    """Exact P(accept) against Algorithm 1 run on random uniforms (draft + verification)."""
    rng = np.random.default_rng(5 + without)
    p, q = rand_pair(rng, 6)
    n, acc = 40000, 0
    u = rng.random((n, 5))
    for i in range(n):
        tk, _, _ = oracle.rrs_draft(q, without, u[i, 0], u[i, 1])
        node = oracle.rrs_verify(p, q, tk[0], tk[1], u[i, 2], u[i, 3], u[i, 4], without)
        acc += node["accept_idx"] >= 0
    exact = tt.acceptance_rrs(p, q, without)
    sd = np.sqrt(exact * (1 - exact) / n)
    assert abs(acc / n - exact) < 4 * sd


def test_spechub_acceptance_matches_simulation_of_algorithm_3():
    rng = np.random.default_rng(8)
    p, q = rand_pair(rng, 6)
    a = int(np.argmax(q))
    n, acc = 40000, 0
    u = rng.random((n, 5))
    for i in range(n):
        tk, _, _, _ = oracle.spechub_draft(q, a, u[i, 0], u[i, 1])
        acc += oracle.spechub_verify(p, q, a, tk[0], tk[1], u[i, 2], u[i, 3], u[i, 4])["accept_idx"] >= 0
    exact = tt.acceptance_spechub(p, q)
    assert abs(acc / n - exact) < 4 * np.sqrt(exact * (1 - exact) / n)


def test_pair_laws_are_distributions_with_the_right_marginals():
    rng = np.random.default_rng(1)
    _, q = rand_pair(rng, 9)
    for without in (False, True):
        Q = tt.pair_law(q, without)
        assert abs(Q.sum() - 1) < 1e-12 and (Q >= 0).all()
        np.testing.assert_allclose(Q.sum(1), q, atol=1e-12)      # x1 ~ q in both schemes
    assert np.all(np.diag(tt.pair_law(q, True)) == 0)


def test_lp_special_cases():
    rng = np.random.default_rng(2)
    p, q = rand_pair(rng, 7)
    # p = q: everything is accepted
    assert abs(tt.acceptance_otm(q, q, False) - 1) < 1e-9
    # a pair law that always drafts (0, 1): exactly min(p0 + p1, 1) can be kept
    Q = np.zeros((7, 7)); Q[0, 1] = 1.0
    assert abs(tt.acceptance_lp(p, Q) - (p[0] + p[1])) < 1e-9
    # both drafts equal (one effective draft): single-draft optimum sum min(p, q)
    assert abs(tt.acceptance_lp(p, np.diag(q)) - np.minimum(p, q).sum()) < 1e-9
    # V = 2 without replacement: the pair is always {0, 1}, so any p can be served
    p2, q2 = rand_pair(rng, 2)
    assert abs(tt.acceptance_otm(p2, q2, True) - 1) < 1e-9
    # V = 2 independent drafts: y is coverable unless both drafts are the other token
    want = min(p2[0], 1 - q2[1] ** 2) + min(p2[1], 1 - q2[0] ** 2)
    assert abs(tt.acceptance_otm(p2, q2, False) - min(want, 1.0)) < 1e-9


def test_lp_dominates_every_coupling_on_the_same_pair_law():
    """The LP optimum bounds any verification rule on its pair law (Section 3): OTM >= RRS,
    OTMw >= RRSw, and with SpecHub's own Q the optimum is SpecHub's 1 - R."""
    rng = np.random.default_rng(3)
    for _ in range(12):
        p, q = rand_pair(rng, 8, conc=0.6)
        assert tt.acceptance_otm(p, q, False) >= tt.acceptance_rrs(p, q, False) - 1e-9
        assert tt.acceptance_otm(p, q, True) >= tt.acceptance_rrs(p, q, True) - 1e-9
        a = int(np.argmax(q))
        Q = np.zeros((8, 8))
        for x in range(8):
            if x != a:
                Q[x, a] = q[x]
                Q[a, x] = q[a] * q[x] / (1 - q[a])
        assert abs(tt.acceptance_lp(p, Q) - tt.acceptance_spechub(p, q)) < 1e-9


def test_lp_equals_the_maximum_flow_of_the_appendix():
    """Appendix "Maximum Flow Problem Formulation": s -> v with capacity sum_x2 Q(v, x2),
    v -> t with p(v), u -> v with Q(u, v).  Capacities scaled to integers for scipy's solver."""
    from scipy.sparse import csr_matrix
    from scipy.sparse.csgraph import maximum_flow

    rng = np.random.default_rng(4)
    scale = 10 ** 9
    for without in (False, True):
        for _ in range(4):
            p, q = rand_pair(rng, 7, conc=0.7)
            Q = tt.pair_law(q, without)
            V = len(p)
            cap = np.zeros((V + 2, V + 2), np.int64)
            s, t = V, V + 1
            for v in range(V):
                cap[s, v] = int(round(Q[v].sum() * scale))
                cap[v, t] = int(round(p[v] * scale))
                for w in range(V):
                    if w != v:
                        cap[v, w] = int(round(Q[v, w] * scale))
            flow = maximum_flow(csr_matrix(cap), s, t).flow_value / scale
            assert abs(flow - tt.acceptance_lp(p, Q)) < 1e-6


def test_table_rows_are_ordered_as_theory_says():
    t = tt.table(pairs=4, V=12, seed=1, grid=[(0.25, 0.7)])
    rrs, rrsw, otm, otmw, hub = t[(0.25, 0.7)]
    assert otm >= rrs - 1e-9 and otmw >= rrsw - 1e-9
    assert all(0.0 < v <= 1.0 for v in (rrs, rrsw, otm, otmw, hub))
