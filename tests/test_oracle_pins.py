"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these tests touches the CUDA library.  Each one is chosen so that a
plausible mistake in the oracle (a dropped term, a wrong sign or index, a
swapped operand, a wrong child index) makes it fail:

  * the worked example of the captions of Figures 4 and 5 (printed values);
  * Theorem 2 / the known exactness of RRS and RRSw: enumerating every draft
    pair and every outcome, the emitted token is distributed exactly as p;
  * Section 3.2: SpecHub's closed-form acceptance equals the optimum of the
    compact LP restricted to SpecHub's support (brute force with an LP solver);
  * Corollary 1: the hub is emitted with probability exactly p(a);
  * Theorem 3: SpecHub accepts at least as much as RRS when q(a)/(1-q(a)) > 1-alpha;
  * Section 5.2: at T -> 0 SpecHub and RRSw both draft the top-2 tokens;
  * degenerate rows: p = q, one-hot q, disjoint supports;
  * decisions agree with the reported acceptance probabilities; the inverse
    CDF walks ids in ascending order with the stated edge convention;
  * an end-to-end Monte-Carlo run of draft + verify over random uniforms;
  * the reported margins: a uniform moved by less than its margin keeps the outcome, by more changes it.
"""
import os

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "worked_example.txt")


def read_golden():
    vals = {}
    with open(GOLDEN) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            k, v = line.split("=")
            nums = [float(t) for t in v.split()]
            vals[k.strip()] = nums if len(nums) > 1 else nums[0]
    return vals


def random_simplex(rng, V, sparsity=0.0):
    x = rng.gamma(0.7, size=V)
    if sparsity > 0:
        x[rng.random(V) < sparsity] = 0.0
        if x.sum() == 0:
            x[rng.integers(V)] = 1.0
    return x / x.sum()


def token_selecting_u(w, tok):
    lo, hi = oracle.cdf_interval(w, tok)
    return 0.5 * (lo + hi)


def spechub_pairs(q, a):
    """Every draft pair SpecHub can emit with its probability, read off the oracle's sampler."""
    V = len(q)
    pairs = {}
    for x in range(V):
        if q[x] == 0:
            continue
        u1 = token_selecting_u(q, x)
        if x != a:
            tk, pr, _, st = oracle.spechub_draft(q, a, u1, 0.0)
            assert tuple(tk) == (x, a)
            pairs[(x, a)] = pr[1]
        else:
            w = q.copy()
            w[a] = 0.0
            for x2 in range(V):
                if w[x2] == 0:
                    continue
                tk, pr, _, st = oracle.spechub_draft(q, a, u1, token_selecting_u(w, x2))
                assert tuple(tk) == (a, x2)
                pairs[(a, x2)] = pr[1]
    return pairs


def spechub_law(p, q):
    """Law of the emitted token, by enumeration over pairs and outcomes of Algorithm 3."""
    V = len(p)
    a = int(np.argmax(q))
    law = np.zeros(V)
    acc = np.zeros(2)
    hub_mass = 0.0
    for (x1, x2), Q in spechub_pairs(q, a).items():
        o = oracle.spechub_verify(p, q, a, x1, x2, 0.5, 0.5, 0.5)
        b1, b2 = o["beta"]
        x = x1 if x2 == a else x2
        law[x] += Q * b1
        law[a] += Q * (1 - b1) * b2
        hub_mass += Q * (1 - b1) * b2
        i_x = 0 if x2 == a else 1
        acc[i_x] += Q * b1
        acc[1 - i_x] += Q * (1 - b1) * b2
        rej = Q * (1 - b1) * (1 - b2)
        if rej > 0:
            w = oracle.spechub_residual(p, q, a)
            assert w[a] == 0.0
            if w.sum() > 0:
                law += rej * w / w.sum()
            else:
                assert rej < 1e-13  # rounding dust only: no residual mass means no rejection
    return law, acc, hub_mass


def rrs_law(p, q, wo):
    V = len(p)
    law = np.zeros(V)
    cost = 0.0
    for x1 in range(V):
        if q[x1] == 0:
            continue
        for x2 in range(V):
            if wo:
                if x2 == x1 or q[x2] == 0:
                    continue
                Q = q[x1] * q[x2] / (1 - q[x1])  # Section 3.3, sampling without replacement
            else:
                Q = q[x1] * q[x2]
            if Q == 0:
                continue
            o = oracle.rrs_verify(p, q, x1, x2, 0.5, 0.5, 0.5, wo)
            b1, b2 = o["beta"]
            law[x1] += Q * b1
            law[x2] += Q * (1 - b1) * b2
            rej = Q * (1 - b1) * (1 - b2)
            cost += rej
            if rej > 0:
                w = oracle.rrs_residual(p, q, x1, wo)
                if w.sum() > 0:
                    law += rej * w / w.sum()
                else:
                    assert rej < 1e-13
    return law, cost


# ------------------------------------------------------------------------------------------------
# P1: the worked example (captions of Figures 4 and 5)
# ------------------------------------------------------------------------------------------------

def test_worked_example_spechub_pair_probabilities():
    g = read_golden()
    q = np.array(g["q"])
    pairs = spechub_pairs(q, 0)
    assert pairs[(1, 0)] == pytest.approx(g["Q_b_a"], abs=1e-15)
    assert pairs[(2, 0)] == pytest.approx(g["Q_c_a"], abs=1e-15)
    assert pairs[(0, 1)] == pytest.approx(g["Q_a_b"], abs=1e-15)
    assert pairs[(0, 2)] == pytest.approx(g["Q_a_c"], abs=1e-15)
    assert sum(pairs.values()) == pytest.approx(1.0, abs=1e-15)


def test_worked_example_rrsw_transport_cost():
    g = read_golden()
    q, p = np.array(g["q"]), np.array(g["p"])
    law, cost = rrs_law(p, q, wo=True)
    assert cost == pytest.approx(g["rrsw_transport_cost"], abs=1e-12)
    np.testing.assert_allclose(law, p, atol=1e-12)
    # with replacement the same example rejects 0.5 * 0.8 * 0.5 = 0.2 (only (a, a) can fail twice)
    law, cost = rrs_law(p, q, wo=False)
    assert cost == pytest.approx(0.2, abs=1e-12)
    np.testing.assert_allclose(law, p, atol=1e-12)


def test_worked_example_spechub_never_rejects():
    g = read_golden()
    q, p = np.array(g["q"]), np.array(g["p"])
    law, acc, hub_mass = spechub_law(p, q)
    np.testing.assert_allclose(law, p, atol=1e-12)
    # every bit of q's excess on 'a' is routed through the hub: nothing is rejected
    assert acc.sum() == pytest.approx(1.0, abs=1e-12)
    o = oracle.spechub_verify(p, q, 0, 1, 0, 0.5, 0.5, 0.5)
    np.testing.assert_allclose(o["rate"], [0.6, 0.4, 0.0], atol=1e-12)


# ------------------------------------------------------------------------------------------------
# P2 / P5: exact law, rate bookkeeping and hub mass, V <= 8
# ------------------------------------------------------------------------------------------------

@pytest.mark.parametrize("V", [2, 3, 4, 5, 8])
def test_spechub_law_is_exactly_p(V):
    rng = np.random.default_rng(100 + V)
    for it in range(60):
        sp = 0.0 if it % 3 else 0.4
        p = random_simplex(rng, V, sp)
        q = random_simplex(rng, V, sp if it % 2 else 0.0)
        if np.count_nonzero(q) < 2:
            continue
        law, acc, hub_mass = spechub_law(p, q)
        a = int(np.argmax(q))
        np.testing.assert_allclose(law, p, atol=1e-12)
        assert hub_mass == pytest.approx(p[a], abs=1e-12)  # Corollary 1
        # row-level rates reported by the oracle are the enumerated ones
        o = oracle.spechub_verify(p, q, a, a, (a + 1) % V, 0.5, 0.5, 0.5)
        np.testing.assert_allclose(o["rate"][:2], acc, atol=1e-12)
        assert o["rate"].sum() == pytest.approx(1.0, abs=1e-12)


@pytest.mark.parametrize("wo", [False, True])
@pytest.mark.parametrize("V", [2, 3, 5, 7])
def test_rrs_law_is_exactly_p(V, wo):
    rng = np.random.default_rng(200 + V)
    for it in range(40):
        p = random_simplex(rng, V, 0.3 if it % 3 == 0 else 0.0)
        q = random_simplex(rng, V)
        law, cost = rrs_law(p, q, wo)
        np.testing.assert_allclose(law, p, atol=1e-12)
        # rates: for RRS (with replacement) they are unconditional and must add up to 1
        if not wo:
            o = oracle.rrs_verify(p, q, 0, 0, 0.5, 0.5, 0.5, False)
            assert o["rate"].sum() == pytest.approx(1.0, abs=1e-12)
            assert o["rate"][2] == pytest.approx(cost, abs=1e-12)


# ------------------------------------------------------------------------------------------------
# P3: closed form = optimum of the compact LP on SpecHub's support (Section 3.2)
# ------------------------------------------------------------------------------------------------

def lp_optimum_on_hub_support(p, q, a):
    from scipy.optimize import linprog

    V = len(p)
    others = [x for x in range(V) if x != a]
    n = len(others)
    rest = sum(q[x] for x in others)
    # variables: [pi(x,a,x)], [pi(x,a,a)], [pi(a,x,x)], [pi(a,x,a)], each of length n
    A, b = [], []
    for i, x in enumerate(others):
        row = np.zeros(4 * n); row[i] = 1; row[n + i] = 1
        A.append(row); b.append(q[x])                      # <= Q(x,a)
        row = np.zeros(4 * n); row[2 * n + i] = 1; row[3 * n + i] = 1
        A.append(row); b.append(q[a] * q[x] / rest)        # <= Q(a,x)
        row = np.zeros(4 * n); row[i] = 1; row[2 * n + i] = 1
        A.append(row); b.append(p[x])                      # <= p(x)
    row = np.zeros(4 * n); row[n:2 * n] = 1; row[3 * n:] = 1
    A.append(row); b.append(p[a])                          # <= p(a)
    res = linprog(-np.ones(4 * n), A_ub=np.array(A), b_ub=np.array(b), bounds=(0, None),
                  method="highs")
    assert res.status == 0
    return -res.fun


@pytest.mark.parametrize("V", [3, 4, 6, 8])
def test_closed_form_matches_lp(V):
    rng = np.random.default_rng(300 + V)
    for it in range(40):
        p = random_simplex(rng, V, 0.3 if it % 4 == 0 else 0.0)
        q = random_simplex(rng, V)
        a = int(np.argmax(q))
        o = oracle.spechub_verify(p, q, a, a, (a + 1) % V, 0.5, 0.5, 0.5)
        accept = o["rate"][0] + o["rate"][1]
        assert accept == pytest.approx(lp_optimum_on_hub_support(p, q, a), abs=1e-9)
        assert o["rate"][2] == pytest.approx(1.0 - accept, abs=1e-12)


# ------------------------------------------------------------------------------------------------
# P4: Theorem 3
# ------------------------------------------------------------------------------------------------

def test_spechub_beats_rrs_under_theorem3_condition():
    rng = np.random.default_rng(400)
    checked = 0
    for it in range(400):
        V = int(rng.integers(3, 9))
        p = random_simplex(rng, V)
        q = random_simplex(rng, V)
        a = int(np.argmax(q))
        alpha = np.minimum(p, q).sum()
        if not q[a] / (1 - q[a]) > 1 - alpha:
            continue
        checked += 1
        s = oracle.spechub_verify(p, q, a, a, (a + 1) % V, 0.5, 0.5, 0.5)["rate"]
        r = oracle.rrs_verify(p, q, 0, 0, 0.5, 0.5, 0.5, False)["rate"]
        assert s[0] + s[1] >= r[0] + r[1] - 1e-12
    assert checked > 100


# ------------------------------------------------------------------------------------------------
# P6: degenerate rows
# ------------------------------------------------------------------------------------------------

def test_p_equals_q_never_rejects():
    rng = np.random.default_rng(500)
    for V in (2, 5, 8):
        q = random_simplex(rng, V)
        a = int(np.argmax(q))
        for (x1, x2) in spechub_pairs(q, a):
            for r1 in (0.0, 0.3, 0.999999):
                for r2 in (0.0, 0.999999):
                    o = oracle.spechub_verify(q, q, a, x1, x2, r1, r2, 0.5)
                    assert o["accept_idx"] in (0, 1)
                    assert o["rate"][2] == 0.0
        for wo in (False, True):
            o = oracle.rrs_verify(q, q, 1, 0, 0.999999, 0.5, 0.5, wo)
            assert o["accept_idx"] == 0 and o["token"] == 1


def test_one_hot_draft():
    V = 5
    q = np.zeros(V); q[2] = 1.0
    p = np.array([0.1, 0.2, 0.3, 0.15, 0.25])
    tk, pr, _, st = oracle.spechub_draft(q, 2, 0.7, 0.3)
    assert tuple(tk) == (2, 0) and st & oracle.STATUS_BITS["DEGENERATE_Q"]
    # hub accepted with probability p(a), otherwise residual proportional to p off the hub
    o = oracle.spechub_verify(p, q, 2, 2, 0, 0.5, 0.29, 0.5)
    assert o["accept_idx"] == 0 and o["token"] == 2 and o["beta"][1] == pytest.approx(0.3)
    o = oracle.spechub_verify(p, q, 2, 2, 0, 0.5, 0.31, 0.0)
    assert o["accept_idx"] == -1 and o["token"] == 0
    w = oracle.spechub_residual(p, q, 2)
    np.testing.assert_allclose(w, [0.1, 0.2, 0.0, 0.15, 0.25])
    np.testing.assert_allclose(o["rate"], [0.3, 0.0, 0.7], atol=1e-15)
    # RRSw with a one-hot q: nothing left to draw the second draft from
    tk, _, st = oracle.rrs_draft(q, True, 0.5, 0.5)
    assert tk[0] == 2 and st & oracle.STATUS_BITS["DEGENERATE_Q"]
    o = oracle.rrs_verify(p, q, 2, 0, 0.31, 0.0, 0.0, True)
    assert o["accept_idx"] == -1 and o["token"] == 0
    np.testing.assert_allclose(oracle.rrs_residual(p, q, 2, True), [0.1, 0.2, 0.0, 0.15, 0.25])


def test_disjoint_supports_reject_everything():
    p = np.array([0.0, 0.0, 0.5, 0.5, 0.0, 0.0])
    q = np.array([0.6, 0.3, 0.0, 0.0, 0.1, 0.0])
    a = 0
    for (x1, x2) in spechub_pairs(q, a):
        o = oracle.spechub_verify(p, q, a, x1, x2, 0.0, 0.0, 0.6)
        assert o["accept_idx"] == -1 and o["token"] == 3
        np.testing.assert_allclose(o["rate"], [0, 0, 1], atol=1e-15)
    np.testing.assert_allclose(oracle.spechub_residual(p, q, a), p)
    for wo in (False, True):
        o = oracle.rrs_verify(p, q, 0, 1, 0.0, 0.0, 0.4, wo)
        assert o["accept_idx"] == -1 and o["token"] == 2
        w = oracle.rrs_residual(p, q, 0, wo)
        np.testing.assert_allclose(w / w.sum(), p)


# ------------------------------------------------------------------------------------------------
# P7: T -> 0 is top-2 greedy for SpecHub and RRSw (Section 5.2)
# ------------------------------------------------------------------------------------------------

def test_low_temperature_is_top2():
    rng = np.random.default_rng(700)
    V, T = 50, 0.004
    logits = rng.normal(size=(1, 256, V)).astype(np.float32)
    srt = -np.sort(-logits[0], axis=1)
    keep = (srt[:, 0] - srt[:, 1] > 0.05) & (srt[:, 1] - srt[:, 2] > 0.05) & (srt[:, 0] - srt[:, 1] < 2.0)
    logits = np.ascontiguousarray(logits[:, keep])
    n = logits.shape[1]
    assert n > 100
    un = rng.random((1, n, 5)).astype(np.float32)
    top2 = np.argsort(-logits[0], axis=1, kind="stable")[:, :2]
    for method in ("spechub", "rrsw"):
        d = oracle.draft_batch(method, logits, T, un)
        np.testing.assert_array_equal(d["tokens"][0], top2)
    d = oracle.draft_batch("rrs", logits, T, un)  # with replacement: the top token twice
    np.testing.assert_array_equal(d["tokens"][0], np.stack([top2[:, 0]] * 2, 1))


# ------------------------------------------------------------------------------------------------
# P8 + decision/probability consistency
# ------------------------------------------------------------------------------------------------

def test_first_test_is_textbook_speculative_sampling():
    rng = np.random.default_rng(800)
    for _ in range(50):
        V = 6
        p, q = random_simplex(rng, V), random_simplex(rng, V)
        a = int(np.argmax(q))
        x = (a + 1 + int(rng.integers(V - 1))) % V
        ratio = min(1.0, p[x] / q[x])
        assert oracle.spechub_verify(p, q, a, x, a, 0.5, 0.5, 0.5)["beta"][0] == pytest.approx(ratio, rel=1e-14)
        assert oracle.rrs_verify(p, q, x, a, 0.5, 0.5, 0.5, False)["beta"][0] == pytest.approx(ratio, rel=1e-14)
        # a single rejected draft leaves norm(max(p-q,0)): RRS stage-2 target
        o = oracle.rrs_verify(p, q, x, x, 0.5, 0.5, 0.5, False)
        assert o["rate"][0] == pytest.approx(np.minimum(p, q).sum(), rel=1e-13)


def test_decisions_follow_reported_probabilities():
    rng = np.random.default_rng(810)
    for _ in range(200):
        V = int(rng.integers(2, 8))
        p, q = random_simplex(rng, V, 0.2), random_simplex(rng, V)
        a = int(np.argmax(q))
        r1, r2, ur = rng.random(3)
        for (x1, x2) in spechub_pairs(q, a):
            o = oracle.spechub_verify(p, q, a, x1, x2, r1, r2, ur)
            b1, b2 = o["beta"]
            x, ix = (x1, 0) if x2 == a else (x2, 1)
            if r1 < b1:
                assert (o["accept_idx"], o["token"]) == (ix, x)
            elif r2 < b2:
                assert (o["accept_idx"], o["token"]) == (1 - ix, a)
            else:
                w = oracle.spechub_residual(p, q, a)
                assert o["accept_idx"] == -1 and o["token"] == oracle.inv_cdf(w, ur)[0]
        for wo in (False, True):
            x1, x2 = int(rng.integers(V)), int(rng.integers(V))
            if q[x1] == 0 or q[x2] == 0 or (wo and x1 == x2):
                continue
            o = oracle.rrs_verify(p, q, x1, x2, r1, r2, ur, wo)
            b1, b2 = o["beta"]
            if r1 < b1:
                assert (o["accept_idx"], o["token"]) == (0, x1)
            elif r2 < b2:
                assert (o["accept_idx"], o["token"]) == (1, x2)
            else:
                assert o["accept_idx"] == -1


def test_inverse_cdf_convention():
    w = np.array([0.0, 0.2, 0.0, 0.5, 0.3, 0.0])
    assert oracle.inv_cdf(w, 0.0)[0] == 1            # u = 0 gives the first token with mass
    assert oracle.inv_cdf(w, 0.19999)[0] == 1
    assert oracle.inv_cdf(w, 0.2)[0] == 3            # prefix must strictly exceed u*W
    assert oracle.inv_cdf(w, 0.69999)[0] == 3
    assert oracle.inv_cdf(w, 0.7)[0] == 4
    assert oracle.inv_cdf(w, 0.9999999)[0] == 4      # never a zero-mass trailing token
    assert oracle.inv_cdf(np.zeros(4), 0.3)[0] == -1
    tok, W, m = oracle.inv_cdf(3.0 * w, 0.45)        # unnormalised weights, margin in units of W
    assert tok == 3 and W == pytest.approx(3.0) and m == pytest.approx(0.25)
    grid = (np.arange(20000) + 0.5) / 20000
    counts = np.bincount([oracle.inv_cdf(w, u)[0] for u in grid], minlength=6) / 20000
    np.testing.assert_allclose(counts, w, atol=1e-4)
    assert oracle.cdf_interval(w, 3) == pytest.approx((0.2, 0.7))


def test_hub_tie_break_and_softmax():
    l = np.array([1.0, 3.0, 3.0, -np.inf, 2.0], np.float32)
    assert oracle.hub(l) == 1
    pr, st = oracle.softmax(l, 0.5)
    assert st == 0 and pr[3] == 0.0
    e = np.exp(np.array([2.0, 6.0, 6.0, -np.inf, 4.0]) - 6.0)
    np.testing.assert_allclose(pr, e / e.sum(), rtol=1e-15)
    assert oracle.softmax(np.array([0.0, np.nan], np.float32))[1] & 1
    assert oracle.softmax(np.array([-np.inf, -np.inf], np.float32))[1] & 1


def test_malformed_pairs_are_flagged():
    p = np.array([0.2, 0.3, 0.5]); q = np.array([0.5, 0.25, 0.25])
    for pair in [(1, 2), (0, 0), (0, 3), (-1, 0)]:
        o = oracle.spechub_verify(p, q, 0, pair[0], pair[1], 0.1, 0.1, 0.1)
        assert o["status"] & oracle.STATUS_BITS["TOKEN_RANGE"] and o["token"] == -1
    o = oracle.rrs_verify(p, q, 0, 5, 0.1, 0.1, 0.1, False)
    assert o["status"] & oracle.STATUS_BITS["TOKEN_RANGE"] and o["token"] == -1


# ------------------------------------------------------------------------------------------------
# P11: end-to-end Monte-Carlo (draft + verify through the batch entry points)
# ------------------------------------------------------------------------------------------------

@pytest.mark.parametrize("method", ["spechub", "rrs", "rrsw"])
def test_monte_carlo_law(method):
    rng = np.random.default_rng(1100)
    V, n = 12, 300000
    lp = rng.normal(0, 1.5, V).astype(np.float32)
    lq = (lp + rng.normal(0, 1.0, V)).astype(np.float32)
    T = 0.8
    LP = np.broadcast_to(lp, (1, n, V)).copy()
    LQ = np.broadcast_to(lq, (1, n, V)).copy()
    un = rng.random((1, n, 5)).astype(np.float32)
    d = oracle.draft_batch(method, LQ, T, un)
    out = oracle.verify_batch(method, LP, LQ, T, d["tokens"], un)
    assert (out["status"] == 0).all()
    p, _ = oracle.softmax(lp, T)
    counts = np.bincount(out["token"][0], minlength=V)
    chi2 = ((counts - n * p) ** 2 / (n * p)).sum()
    assert chi2 < 45.0  # 11 dof: P(chi2 > 45) ~ 5e-6
    # empirical acceptance by child position against the reported rates (SpecHub, RRS)
    if method != "rrsw":
        rate = out["rate"][0, 0]
        emp = np.array([(out["accept_idx"][0] == i).mean() for i in (0, 1, -1)])
        np.testing.assert_allclose(emp, rate, atol=5e-3)


def test_tree_walk():
    # 7-node heap tree, 2 sequences; leaves are nodes 3..6
    kind = np.array([0, 0, 0, 1, 1, 1, 1], np.uint8)
    acc = np.array([[1, -1, 0, -1, -1, -1, -1], [-1, 0, 0, -1, -1, -1, -1]], np.int32)
    tok = np.array([[10, 11, 12, 13, 14, 15, 16], [20, 21, 22, 23, 24, 25, 26]], np.int32)
    w = oracle.walk(acc, tok, 3, node_kind=kind)
    np.testing.assert_array_equal(w["path_nodes"], [[0, 2, 5], [0, -1, -1]])
    np.testing.assert_array_equal(w["path_tokens"], [[10, 12, 15], [20, -1, -1]])
    np.testing.assert_array_equal(w["n_accepted"], [2, 0])
    np.testing.assert_array_equal(w["n_emitted"], [3, 1])
    # custom child table: an unbalanced chain 0 -> 1 -> 2, second children missing
    child = np.array([[1, -1], [2, -1], [-1, -1]], np.int32)
    acc = np.array([[0, 0, 0]], np.int32)
    w = oracle.walk(acc, np.array([[5, 6, 7]], np.int32), 4, child=child)
    np.testing.assert_array_equal(w["path_nodes"], [[0, 1, 2, -1]])
    np.testing.assert_array_equal(w["n_accepted"], [3])


@pytest.mark.parametrize("method", ["spechub", "rrs", "rrsw"])
def test_margins_are_the_distance_to_the_point_where_the_outcome_changes(method):
    """margin[] is what the parity checker's near-threshold rule rests on.  Pinned by behaviour: moving
    a uniform by a little less than its margin never changes the outcome of that test or draw, moving
    it by a little more (towards the threshold) does."""
    rng = np.random.default_rng(77)
    flips = holds = 0
    for _ in range(200):
        V = int(rng.integers(3, 9))
        p, q = random_simplex(rng, V), random_simplex(rng, V)
        a = int(np.argmax(q))
        if method == "spechub":
            x = int(rng.choice([y for y in range(V) if y != a]))
            x1, x2 = (x, a) if rng.random() < 0.5 else (a, x)
            run = lambda r1, r2, u: oracle.spechub_verify(p, q, a, x1, x2, r1, r2, u)
        else:
            x1, x2 = int(rng.integers(V)), int(rng.integers(V))
            if method == "rrsw" and x2 == x1:
                x2 = (x1 + 1) % V
            run = lambda r1, r2, u: oracle.rrs_verify(p, q, x1, x2, r1, r2, u, method == "rrsw")
        r = [float(rng.random()), float(rng.random()), float(rng.random())]
        o = run(*r)
        # uniform i decides test 1, test 2 (if performed), the residual draw (if both rejected)
        for i in range(3):
            m = float(o["margin"][i])
            if not np.isfinite(m) or m <= 1e-9 or m >= 0.5:
                continue
            for sign in (+1, -1):
                for scale, must_hold in ((1 - 1e-6, True), (1 + 1e-6, False)):
                    rr = list(r)
                    rr[i] = r[i] + sign * m * scale
                    if not 0.0 <= rr[i] < 1.0:
                        continue
                    o2 = run(*rr)
                    same = (o2["accept_idx"] == o["accept_idx"] and o2["token"] == o["token"])
                    if must_hold:
                        assert same, (method, i, sign, r, m)
                        holds += 1
                    elif not same:
                        flips += 1
            # beyond the margin, on one of the two sides, the outcome does change
            changed = False
            for sign in (+1, -1):
                v = r[i] + sign * m * (1 + 1e-6)
                if 0.0 <= v < 1.0:
                    rr = list(r); rr[i] = v
                    o2 = run(*rr)
                    changed |= not (o2["accept_idx"] == o["accept_idx"] and o2["token"] == o["token"])
                else:
                    changed = True   # the threshold lies outside [0, 1) on that side: nothing to cross
            assert changed, (method, i, r, m, dict(acc=int(o["accept_idx"]), tok=int(o["token"])))
    assert holds > 120 and flips > 60
