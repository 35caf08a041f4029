"""GPU-vs-oracle comparison rules shared by the parity tests, the smoke check and nothing else.

The rule: decisions (accept / reject), hub and token ids must be identical,
except where a uniform lies within NEAR = 1e-6 of the threshold it is compared
with -- then the GPU may sit on the other side of that one threshold, and what
follows is checked against the oracle re-run on that side.  For a sampled token
"threshold" means an edge of the token's interval in the oracle's fp64 CDF.

Probabilities: |gpu - oracle| <= RTOL * |oracle| + floor, RTOL = 1e-5, with a
floor of 1e-12 for values below 1e-7.  Two kinds of output are not plain sums
of positive terms and carry a further, derived, term:

  * the rates are built from differences of probabilities: rate[0] and rate[1]
    are differences of O(1) sums (e.g. the mass accepted at child 0 is
    (1 - q(a)) - S1 + min(p(a), S2)), and every term of rate[2] is a clipped
    difference max(p - q - c q, 0) whose operands (p, q, c q: each family sums
    to at most 1) carry the fp32 error of a single probability.  So a rate has
    an absolute error of a few 1e-7 whatever its size, and a small rate cannot
    meet a relative bar (a rejection mass of 2e-4 on a two-token vocabulary was
    off by 1e-8: 5e-5 relative).  They get the per-row bound EPS(row) below (at
    least ATOL_DIFF = 1e-6); the measurement records how little of it is used.
  * an acceptance probability N/D whose numerator is a difference (p(x) - q(x),
    p(a) - S2) is ill-conditioned when the operands nearly cancel: a relative
    error EPS in every fp32 p(y), q(y) moves N/D by EPS * cond, where cond is
    reported by the oracle (pinned in tests/test_oracle_cond.py: it bounds the
    summed magnitudes of the derivatives of N/D, within a small factor).
    EPS is the fp32 path's bound on a single probability: 2 ulp from
    ex2.approx (2.4e-7), and the exponent (l - l_ref) log2(e) / T itself: the
    FMA that forms it rounds to half an ulp of a number as large as the row's
    spread E = (max l - min l) log2(e) / T, and log2(e) / T is an fp32 number
    too, so 2 * E * 2^-24 absolute in the exponent, times ln 2 in the
    exponential: EPS(row) = 2.5e-7 + 8.5e-8 * E, at least 1e-6 (E = 26 on the
    128K-vocabulary configuration, 43 on the 32K one at T = 0.6).  The rates'
    absolute term is EPS(row) as well.  beta_i gets EPS * cond_i, and
    the band around the threshold inside which the GPU may decide the other
    way is max(NEAR, EPS * cond_i): 1e-6 for a well-conditioned test, wider
    only where fp32 cannot resolve the threshold itself.  Rows that use the
    wider band are counted (wide_band).

Every comparison is also measured: per field, the largest |gpu - oracle| /
|oracle| and how many values meet the plain 1e-5 bar without the derived term.
"""
from __future__ import annotations

import numpy as np

import oracle

NEAR = 1e-6
RTOL = 1e-5
FLOOR = 1e-12       # absolute floor, for values below 1e-7
ATOL_DIFF = 1e-6    # the rates: sums of (clipped) differences of probabilities
ATOL = ATOL_DIFF    # (the k-draft rates m_j - m_{j+1} are differences too)
EPS = 1e-6          # smallest per-probability error bound; see row_eps


def row_eps(lp_row, lq_row, T):
    """fp32 bound on the relative error of one probability of this row pair (module docstring)."""
    spread = 0.0
    for row in (lp_row, lq_row):
        f = row[np.isfinite(row)]
        if f.size:
            spread = max(spread, float(f.max() - f.min()))
    E = min(spread * 1.4426950408889634 / float(T), 126.0)
    return max(EPS, 2.5e-7 + 8.5e-8 * E)

FATAL = oracle.STATUS_BITS["NONFINITE"] | oracle.STATUS_BITS["TOKEN_RANGE"]


class Field:
    """Measurement of one output field over everything compared so far."""

    def __init__(self):
        self.n = 0            # values compared
        self.strict = 0       # of them, within RTOL * |oracle| + FLOOR (no derived term needed)
        self.max_rel = 0.0    # largest |gpu - oracle| / |oracle| among values >= 1e-7
        self.max_abs = 0.0    # largest |gpu - oracle|

    def add(self, other):
        self.n += other.n; self.strict += other.strict
        self.max_rel = max(self.max_rel, other.max_rel); self.max_abs = max(self.max_abs, other.max_abs)

    def __repr__(self):
        return "n=%d strict=%.4f max_rel=%.1e max_abs=%.1e" % (
            self.n, self.strict / max(self.n, 1), self.max_rel, self.max_abs)


class Stats:
    def __init__(self):
        self.rows = 0
        self.exact = 0
        self.exempt_test = 0
        self.exempt_token = 0
        self.wide_band = 0
        self.max_rel = 0.0
        self.fields = {}

    def add(self, other):
        """Fold another Stats in (totals over methods, layouts, variants)."""
        self.rows += other.rows; self.exact += other.exact
        self.exempt_test += other.exempt_test; self.exempt_token += other.exempt_token
        self.wide_band += other.wide_band
        self.max_rel = max(self.max_rel, other.max_rel)
        for k, f in other.fields.items():
            self.fields.setdefault(k, Field()).add(f)
        return self

    def exempt_fraction(self):
        return (self.exempt_test + self.exempt_token) / max(self.rows, 1)

    def __repr__(self):
        head = "rows=%d exact=%d exempt_test=%d exempt_token=%d (%.2f%% exempt) wide_band=%d max_prob_err=%.2e" % (
            self.rows, self.exact, self.exempt_test, self.exempt_token, 100 * self.exempt_fraction(),
            self.wide_band, self.max_rel)
        return head + "".join("\n    %-10s %r" % (k, f) for k, f in sorted(self.fields.items()))


def _close(g, o, what, ctx, stats, extra=0.0):
    """|g - o| <= RTOL |o| + FLOOR + extra (extra: the field's derived term, scalar or per value)."""
    g = np.atleast_1d(np.asarray(g, np.float64))
    o = np.atleast_1d(np.asarray(o, np.float64))
    err = np.abs(g - o)
    strict_tol = RTOL * np.abs(o) + FLOOR
    tol = strict_tol + extra
    if not np.all(err <= tol):
        raise AssertionError("%s mismatch %s: gpu=%s oracle=%s tol=%s" % (what, ctx, g, o, tol))
    f = stats.fields.setdefault(what, Field())
    f.n += err.size
    f.strict += int(np.sum(err <= strict_tol))
    big = np.abs(o) >= 1e-7
    if np.any(big):
        f.max_rel = max(f.max_rel, float(np.max(err[big] / np.abs(o[big]))))
    f.max_abs = max(f.max_abs, float(np.max(err)))
    stats.max_rel = max(stats.max_rel, float(np.max(err / (np.abs(o) + extra + FLOOR))))


def _token_consistent(w, tok, u):
    """Is `tok` an admissible inverse-CDF draw of weights w with uniform u, within NEAR?"""
    if tok < 0 or tok >= len(w):
        return False
    lo, hi = oracle.cdf_interval(w, tok)
    return lo - NEAR <= u <= hi + NEAR


def check_draft_row(method, lq_row, T, u, g_tokens, g_hub, g_prob, g_status, o_tokens, o_hub, o_prob,
                    o_status, ctx, stats):
    """One row of the draft step.  o_* come from oracle.draft_batch on the same inputs."""
    stats.rows += 1
    if o_status & FATAL:
        assert g_status & FATAL and tuple(g_tokens) == (-1, -1), ("draft fatal row", ctx, g_tokens, g_status)
        return
    assert not (g_status & FATAL), ("unexpected fatal status", ctx, g_status)
    if method == "spechub":
        assert g_hub == o_hub, ("hub", ctx, g_hub, o_hub)
    if tuple(g_tokens) == tuple(o_tokens):
        stats.exact += 1
        assert g_status == o_status, ("status", ctx, g_status, o_status)
        if method == "spechub" and g_prob is not None:
            _close(g_prob[0], o_prob[0], "q(a)", ctx, stats)
            _close(g_prob[1], o_prob[1], "Q(pair)", ctx, stats)
        return
    # tokens differ: the GPU's choices must each be admissible given its earlier choices
    q, st = oracle.softmax(lq_row, T)
    stats.exempt_token += 1
    x1, x2 = int(g_tokens[0]), int(g_tokens[1])
    assert _token_consistent(q, x1, u[0]), ("x1 not admissible", ctx, g_tokens, o_tokens)
    if method == "spechub":
        a = o_hub
        if x1 != a:
            assert x2 == a, ("x2 must be the hub", ctx, g_tokens)
        else:
            w = q.copy(); w[a] = 0.0
            assert _token_consistent(w, x2, u[1]), ("x2 not admissible", ctx, g_tokens, o_tokens)
    elif method == "rrs":
        assert _token_consistent(q, x2, u[1]), ("x2 not admissible", ctx, g_tokens, o_tokens)
    else:
        w = q.copy(); w[x1] = 0.0
        assert _token_consistent(w, x2, u[1]), ("x2 not admissible", ctx, g_tokens, o_tokens)


def _oracle_row(method, p, q, a, x1, x2, r1, r2, ur):
    if method == "spechub":
        return oracle.spechub_verify(p, q, a, x1, x2, r1, r2, ur)
    return oracle.rrs_verify(p, q, x1, x2, r1, r2, ur, method == "rrsw")


def check_verify_row(method, lp_row, lq_row, T, tokens, u, leaf, g, o, ctx, stats):
    """One row of verification.  g: dict of python scalars/arrays from the GPU
    (accept_idx, token, hub, beta[2], rate[3], status); o: the oracle's NODE_DTYPE record."""
    stats.rows += 1
    o_st = int(o["status"])
    if o_st & FATAL:
        assert g["status"] & FATAL == o_st & FATAL, ("fatal status", ctx, g["status"], o_st)
        assert g["token"] == -1 and g["accept_idx"] == -1, ("fatal row output", ctx, g)
        return
    assert not (g["status"] & FATAL), ("unexpected fatal status", ctx, g["status"])
    r1, r2, ur = float(u[2]), float(u[3]), float(u[4])
    if leaf:
        assert g["accept_idx"] == -1
        if g["token"] == o["token"]:
            stats.exact += 1
            return
        p, _ = oracle.softmax(lp_row, T)
        assert _token_consistent(p, g["token"], ur), ("leaf token", ctx, g["token"], o["token"])
        stats.exempt_token += 1
        return
    if method == "spechub":
        assert g["hub"] == o["hub"], ("hub", ctx, g["hub"], o["hub"])
    # probabilities first: they do not depend on the uniforms
    eps = row_eps(lp_row, lq_row, T)
    for i in range(2):
        _close(g["beta"][i], o["beta"][i], "beta[%d]" % i, ctx, stats, extra=eps * float(o["cond"][i]))
    for i in range(3):
        _close(g["rate"][i], o["rate"][i], "rate[%d]" % i, ctx, stats, extra=eps)
    if g["accept_idx"] == o["accept_idx"] and g["token"] == o["token"]:
        stats.exact += 1
        soft = oracle.STATUS_BITS["ZERO_RESIDUAL"]
        assert (g["status"] | soft) == (o_st | soft), ("status", ctx, g["status"], o_st)
        return
    # something differs: find the admissible alternative
    p, _ = oracle.softmax(lp_row, T)
    q, _ = oracle.softmax(lq_row, T)
    a = int(o["hub"])
    x1, x2 = int(tokens[0]), int(tokens[1])
    cands = [(r1, r2)]
    m1 = float(o["margin"][0])
    band1 = max(NEAR, eps * float(o["cond"][0]))
    r1s = [r1] + ([min(max(r1 - 2 * m1 - 1e-9, 0.0), 1.0), min(r1 + 2 * m1 + 1e-9, 1.0)] if m1 <= band1 else [])
    wide = False
    for rr1 in r1s:
        o1 = _oracle_row(method, p, q, a, x1, x2, rr1, r2, ur)
        mm2 = float(o1["margin"][1])
        band2 = max(NEAR, eps * float(o1["cond"][1]))
        if (band1 > NEAR and NEAR < m1 <= band1) or (band2 > NEAR and NEAR < mm2 <= band2):
            wide = True   # a threshold this row may cross lies outside the plain 1e-6 band
        r2s = [r2] + ([min(max(r2 - 2 * mm2 - 1e-9, 0.0), 1.0), min(r2 + 2 * mm2 + 1e-9, 1.0)] if mm2 <= band2 else [])
        for rr2 in r2s:
            cands.append((rr1, rr2))
    if wide:
        stats.wide_band += 1
    for (rr1, rr2) in cands:
        alt = _oracle_row(method, p, q, a, x1, x2, rr1, rr2, ur)
        if alt["accept_idx"] != g["accept_idx"]:
            continue
        if g["accept_idx"] >= 0:
            if alt["token"] == g["token"]:
                stats.exempt_test += 1
                return
            continue
        # both rejected: the residual token must be admissible
        if alt["token"] == g["token"]:
            stats.exempt_test += 1
            return
        if alt["status"] & oracle.STATUS_BITS["ZERO_RESIDUAL"]:
            w = p
        elif method == "spechub":
            w = oracle.spechub_residual(p, q, a)
        else:
            w = oracle.rrs_residual(p, q, x1, method == "rrsw")
        if _token_consistent(w, g["token"], ur):
            stats.exempt_token += 1
            return
    raise AssertionError("decision/token mismatch %s: gpu=(%d,%d) oracle=(%d,%d) margins=%s u=%s" % (
        ctx, g["accept_idx"], g["token"], o["accept_idx"], o["token"], o["margin"], (r1, r2, ur)))


def temps_array(T, B):
    t = np.asarray(T, np.float32)
    return np.full(B, float(t), np.float32) if t.ndim == 0 else t


def check_verify(method, lp, lq, T, tokens, uniforms, node_kind, gpu, stats=None, label="", pool=None,
                 oracle_out=None):
    """All rows of a [B][N][V] problem.  gpu: dict of numpy arrays as returned by the binding.
    pool: an oracle.fanout.Pool to run the oracle's batch call on several cores (same results).
    oracle_out: the oracle's records of an earlier check of the same problem (not computed again)."""
    stats = stats or Stats()
    B, N, V = lp.shape
    t = temps_array(T, B)
    o = oracle_out if oracle_out is not None else (pool or oracle).verify_batch(method, lp, lq, t, tokens, uniforms, node_kind)
    for b in range(B):
        for n in range(N):
            g = dict(accept_idx=int(gpu["accept_idx"][b, n]), token=int(gpu["token"][b, n]),
                     hub=int(gpu["hub"][b, n]), beta=gpu["beta"][b, n], rate=gpu["rate"][b, n],
                     status=int(gpu["status"][b, n]))
            leaf = node_kind is not None and node_kind[n] == 1
            check_verify_row(method, lp[b, n], lq[b, n], float(t[b]), tokens[b, n], uniforms[b, n], leaf,
                             g, o[b, n], "%s[%s b=%d n=%d V=%d]" % (label, method, b, n, V), stats)
    return stats, o


def check_draft(method, lq, T, uniforms, gpu, stats=None, label="", pool=None):
    stats = stats or Stats()
    B, N, V = lq.shape
    t = temps_array(T, B)
    o = (pool or oracle).draft_batch(method, lq, t, uniforms)
    for b in range(B):
        for n in range(N):
            gp = gpu["prob"][b, n] if "prob" in gpu and gpu["prob"] is not None else None
            gh = int(gpu["hub"][b, n]) if "hub" in gpu and gpu["hub"] is not None else -1
            check_draft_row(method, lq[b, n], float(t[b]), uniforms[b, n], gpu["tokens"][b, n], gh, gp,
                            int(gpu["status"][b, n]), o["tokens"][b, n], int(o["hub"][b, n]),
                            o["prob"][b, n], int(o["status"][b, n]),
                            "%s[%s b=%d n=%d V=%d]" % (label, method, b, n, V), stats)
    return stats, o


def to_numpy(d):
    return {k: (v.detach().cpu().numpy() if hasattr(v, "detach") else v) for k, v in d.items()}
