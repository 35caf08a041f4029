"""Pins of the oracle's Algorithm 1 for k > 2 drafts (the paper's ternary trees and its
acceptance-decay experiment use them): the k = 2 case must coincide with the two-draft functions
pinned in test_oracle_pins.py; the emitted token's law must be exactly p, by enumeration of every
draft tuple and outcome; the stage rates of RRS must add up to 1; a Monte-Carlo run end to end."""
import itertools

import numpy as np
import pytest

import oracle


def random_simplex(rng, V, sparsity=0.0):
    x = rng.gamma(0.7, size=V)
    if sparsity > 0:
        x[rng.random(V) < sparsity] = 0.0
        if x.sum() == 0:
            x[rng.integers(V)] = 1.0
    return x / x.sum()


@pytest.mark.parametrize("wo", [False, True])
def test_k2_coincides_with_the_two_draft_oracle(wo):
    rng = np.random.default_rng(31)
    for _ in range(300):
        V = int(rng.integers(2, 9))
        p, q = random_simplex(rng, V, 0.2), random_simplex(rng, V)
        x1, x2 = int(rng.integers(V)), int(rng.integers(V))
        r1, r2, ur = rng.random(3)
        a = oracle.rrs_verify(p, q, x1, x2, r1, r2, ur, wo)
        b = oracle.rrs_k_verify(p, q, [x1, x2], [r1, r2], ur, wo)
        assert (a["accept_idx"], a["token"]) == (b["accept_idx"], b["token"])
        np.testing.assert_allclose(b["beta"], a["beta"], atol=1e-14)
        np.testing.assert_allclose(b["rate"], a["rate"], atol=1e-14)
        u = rng.random(2)
        ta, _, _ = oracle.rrs_draft(q, wo, u[0], u[1])
        tb, _, _ = oracle.rrs_k_draft(q, 2, wo, u)
        np.testing.assert_array_equal(ta, tb)


def law_by_enumeration(p, q, k, wo):
    V = len(p)
    law = np.zeros(V)
    total_q = 0.0
    for xs in itertools.product(range(V), repeat=k):
        if wo and len(set(xs)) < k:
            continue
        Q, rem = 1.0, 1.0
        for x in xs:
            Q *= q[x] / rem if wo else q[x]     # Section 3.3: product of renormalised draws
            if wo:
                rem -= q[x]
        if Q <= 0 or not np.isfinite(Q):
            continue
        total_q += Q
        o = oracle.rrs_k_verify(p, q, xs, [0.5] * k, 0.5, wo)
        reach = Q
        for i, x in enumerate(xs):
            law[x] += reach * o["beta"][i]
            reach *= 1 - o["beta"][i]
        if reach > 1e-15:
            w = oracle.rrs_k_residual(p, q, xs, wo)
            assert w.sum() > 0
            law += reach * w / w.sum()
    return law, total_q


@pytest.mark.parametrize("wo", [False, True])
@pytest.mark.parametrize("k,V", [(3, 3), (3, 4), (4, 4), (3, 5)])
def test_law_is_exactly_p(k, V, wo):
    rng = np.random.default_rng(100 * k + V)
    for it in range(8):
        p = random_simplex(rng, V, 0.3 if it % 3 == 0 else 0.0)
        q = random_simplex(rng, V)
        if wo and np.count_nonzero(q) < k:
            continue
        law, tq = law_by_enumeration(p, q, k, wo)
        assert tq == pytest.approx(1.0, abs=1e-12)
        np.testing.assert_allclose(law, p, atol=1e-12)


def test_rrs_stage_rates_add_up_and_decay():
    rng = np.random.default_rng(7)
    for _ in range(50):
        V, k = 8, 5
        p, q = random_simplex(rng, V), random_simplex(rng, V)
        o = oracle.rrs_k_verify(p, q, [0] * k, [0.5] * k, 0.5, False)
        assert o["rate"].sum() == pytest.approx(1.0, abs=1e-12)
        # a rejected stage removes min(p, q): what is left to accept can only shrink
        assert np.all(np.diff(o["rate"][:k]) <= 1e-12)


@pytest.mark.parametrize("wo", [False, True])
def test_decisions_follow_betas(wo):
    rng = np.random.default_rng(9)
    for _ in range(200):
        V, k = int(rng.integers(3, 8)), 3
        p, q = random_simplex(rng, V, 0.2), random_simplex(rng, V)
        xs = [int(v) for v in (rng.permutation(V)[:k] if wo else rng.integers(0, V, k))]
        if any(q[x] == 0 for x in xs):
            continue
        r, ur = rng.random(k), rng.random()
        o = oracle.rrs_k_verify(p, q, xs, r, ur, wo)
        expect = -1
        for i in range(k):
            if r[i] < o["beta"][i]:
                expect = i
                break
        assert o["accept_idx"] == expect
        if expect >= 0:
            assert o["token"] == xs[expect]
        else:
            w = oracle.rrs_k_residual(p, q, xs, wo)
            assert o["token"] == oracle.inv_cdf(w if w.sum() > 0 else p, ur)[0]


@pytest.mark.parametrize("wo", [False, True])
def test_monte_carlo_k3(wo):
    rng = np.random.default_rng(1234)
    V, n, k = 10, 200000, 3
    lp = rng.normal(0, 1.5, V).astype(np.float32)
    lq = (lp + rng.normal(0, 1.0, V)).astype(np.float32)
    LP = np.broadcast_to(lp, (1, n, V)).copy()
    LQ = np.broadcast_to(lq, (1, n, V)).copy()
    un = rng.random((1, n, 2 * k + 1)).astype(np.float32)
    d = oracle.rrs_k_draft_batch(k, wo, LQ, 0.9, un)
    out = oracle.rrs_k_verify_batch(k, wo, LP, LQ, 0.9, d["tokens"], un)
    p, _ = oracle.softmax(lp, 0.9)
    counts = np.bincount(out["token"][0], minlength=V)
    chi2 = ((counts - n * p) ** 2 / (n * p)).sum()
    assert chi2 < 42.0  # 9 dof
    if wo:
        assert all(len(set(t)) == k for t in d["tokens"][0][:2000])


def test_ternary_walk():
    # complete ternary tree with 13 nodes (levels 1 + 3 + 9), leaves = last level
    kind = np.array([0] * 4 + [1] * 9, np.uint8)
    acc = np.full((2, 13), -1, np.int32)
    tok = np.arange(26, dtype=np.int32).reshape(2, 13) + 100
    acc[0, 0] = 2; acc[0, 3] = 1       # 0 -> child 2 (node 3) -> child 1 (node 11, leaf)
    acc[1, 0] = 0                      # 0 -> node 1, rejected there
    w = oracle.walk_k(3, acc, tok, 3, node_kind=kind)
    np.testing.assert_array_equal(w["path_nodes"], [[0, 3, 11], [0, 1, -1]])
    np.testing.assert_array_equal(w["n_accepted"], [2, 1])
    np.testing.assert_array_equal(w["n_emitted"], [3, 2])
