/*
 * CPU oracle for the sampling-verification step of multi-draft speculative
 * decoding: SpecHub (k = 2), Recursive Rejection Sampling (RRS) and RRS
 * without replacement (RRSw), arXiv 2411.05289.
 *
 * THIS FILE IS TEST INFRASTRUCTURE.  It is a plain, slow, single-threaded,
 * double-precision restatement of the paper's algorithms, written to be
 * checked against the paper by eye.  It shares no code with the CUDA library
 * and must never be called from the product path; only the tests, the smoke
 * check and the benchmark's CPU-baseline leg use it.
 *
 * Notation is the paper's (Section 2): p = target distribution, q = draft
 * distribution, both over the vocabulary V; a = argmax q = the hub token
 * (Section 4); (x1, x2) = the k = 2 draft tokens of a node; r1, r2 = the
 * uniforms of the first and second acceptance test performed; u_res = the
 * uniform that drives the residual draw.
 *
 * Conventions the paper leaves open (all stated where they are used):
 *   - hub ties: lowest token id among the maxima of the draft logits;
 *   - an acceptance test "accept with probability min(N/D, 1)" is taken as
 *     the strict multiplicative test  r * D < N  with r in [0,1); D = 0
 *     rejects;
 *   - inverse-CDF sampling walks token ids in ascending order and returns the
 *     first id whose inclusive prefix sum exceeds u * W (W = total weight);
 *   - the residual after a SpecHub rejection has no mass on the hub
 *     (Corollary 1 fixes the hub's accepted mass at exactly p(a));
 *   - the hub token is offered first to pairs (a, x) and the remainder to
 *     pairs (x, a), as in the proof of Theorem 2.
 *
 * Every sum is a Neumaier-compensated double sum in ascending token order.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORC_NONFINITE        1u   /* NaN / +inf logit, or a row with no finite logit */
#define ORC_TOKEN_RANGE      2u   /* draft token out of range, or pair malformed       */
#define ORC_DEGENERATE_Q     4u   /* draft mass outside the excluded token is zero     */
#define ORC_ZERO_MASS_DRAFT  8u   /* a performed test had denominator 0                */
#define ORC_ZERO_RESIDUAL    16u  /* residual mass 0 on rejection: drew from p         */

/* ---- compensated summation ------------------------------------------------ */
typedef struct { double s, c; } nsum;
static void ns_init(nsum *k) { k->s = 0.0; k->c = 0.0; }
static void ns_add(nsum *k, double x) {
    double t = k->s + x;
    if (fabs(k->s) >= fabs(x)) k->c += (k->s - t) + x; else k->c += (x - t) + k->s;
    k->s = t;
}
static double ns_val(const nsum *k) { return k->s + k->c; }

static double dmax(double a, double b) { return a > b ? a : b; }
static double dmin(double a, double b) { return a < b ? a : b; }

/* ---- Section 2 / 5.1: distribution of a model at temperature T ------------- */
/* prob(y) = exp(l(y)/T) / sum_y' exp(l(y')/T), evaluated with the usual
 * max-shift.  -inf logits are allowed (probability 0).  Returns status bits. */
unsigned orc_softmax(const float *logits, int V, double T, double *prob) {
    double m = -INFINITY;
    for (int y = 0; y < V; ++y) {
        double l = (double)logits[y];
        if (isnan(l) || l == INFINITY) return ORC_NONFINITE;
        double z = l / T;
        if (z > m) m = z;
    }
    if (m == -INFINITY) return ORC_NONFINITE;
    nsum Z; ns_init(&Z);
    for (int y = 0; y < V; ++y) {
        double e = exp((double)logits[y] / T - m);
        prob[y] = e;
        ns_add(&Z, e);
    }
    double z = ns_val(&Z);
    for (int y = 0; y < V; ++y) prob[y] /= z;
    return 0u;
}

/* ---- Section 4, Algorithm 3 first step: the hub a = argmax_x q(x) ---------- */
/* Decided on the draft logits (softmax is monotone), lowest id on ties. */
int orc_hub(const float *draft_logits, int V) {
    int a = 0;
    for (int y = 1; y < V; ++y) if (draft_logits[y] > draft_logits[a]) a = y;
    return a;
}

/* ---- inverse-CDF draw from unnormalised non-negative weights ---------------- */
/* token = min{ j : sum_{i<=j} w(i) > u*W };  if rounding leaves none, the last
 * j with w(j) > 0.  Returns -1 when W = 0.  *margin (may be NULL) receives the
 * distance from u to the nearest *deciding* edge of the chosen token's CDF
 * interval, in units of W (an edge with no mass beyond it decides nothing and
 * counts as infinitely far).  *W_out (may be NULL) receives W. */
int orc_inv_cdf(const double *w, int V, double u, double *W_out, double *margin) {
    nsum tot; ns_init(&tot);
    int last_pos = -1;
    for (int j = 0; j < V; ++j) if (w[j] > 0.0) { ns_add(&tot, w[j]); last_pos = j; }
    double W = ns_val(&tot);
    if (W_out) *W_out = W;
    if (margin) *margin = INFINITY;
    if (last_pos < 0 || !(W > 0.0)) return -1;
    double t = u * W;
    nsum run; ns_init(&run);
    int tok = -1; double lo = 0.0, hi = 0.0;
    int first_pos = -1;
    for (int j = 0; j < V; ++j) {
        if (!(w[j] > 0.0)) continue;
        if (first_pos < 0) first_pos = j;
        double before = ns_val(&run);
        ns_add(&run, w[j]);
        double after = ns_val(&run);
        if (after > t) { tok = j; lo = before; hi = after; break; }
    }
    if (tok < 0) { tok = last_pos; lo = W; hi = W; if (margin) *margin = 0.0; return tok; }
    if (margin) {
        double dlo = (tok == first_pos) ? INFINITY : (t - lo) / W;
        double dhi = (tok == last_pos) ? INFINITY : (hi - t) / W;
        *margin = dmin(dlo, dhi);
    }
    return tok;
}

/* CDF interval [lo, hi) of `token` under weights w, in units of W.  Used by the
 * parity checker to decide whether another token is within the allowed
 * distance of u.  Returns 0 if w(token) = 0 or W = 0 (lo = hi = prefix). */
int orc_cdf_interval(const double *w, int V, int token, double *lo, double *hi) {
    nsum tot; ns_init(&tot);
    for (int j = 0; j < V; ++j) if (w[j] > 0.0) ns_add(&tot, w[j]);
    double W = ns_val(&tot);
    *lo = *hi = 0.0;
    if (!(W > 0.0) || token < 0 || token >= V) return 0;
    nsum run; ns_init(&run);
    for (int j = 0; j < token; ++j) if (w[j] > 0.0) ns_add(&run, w[j]);
    *lo = ns_val(&run) / W;
    if (w[token] > 0.0) ns_add(&run, w[token]);
    *hi = ns_val(&run) / W;
    return w[token] > 0.0;
}

/* Per-node result.  Doubles first so that the layout has no padding surprises. */
typedef struct {
    double beta[2];    /* acceptance probability min(N/D,1) of test 1 / test 2 for this pair  */
    double rate[3];    /* row-level masses: accept child 0, accept child 1, reject              */
    double margin[3];  /* |r1 - N1/D1|, |r2 - N2/D2| (inf if not performed), residual-draw margin */
    double cond[2];    /* conditioning of N/D for test 1 / test 2: (|N| + beta |D|) / D, where |.|
                          is the sum of the absolute values of the terms the quantity is formed
                          from, each weighted by the number of perturbed factors it has
                          (Q(a,y) = q(a) q(y) / (1 - q(a)) has three, RRSw's q(y) / (1 - q(x1))
                          two); a relative error eps in every p(y), q(y) moves N/D by at most
                          eps * cond to first order.  Used only by the parity checker to size
                          its tolerance. */
    int32_t accept_idx; /* 0 / 1 = accepted child, -1 = rejected (token is the residual draw)  */
    int32_t token;      /* emitted token of this node                                          */
    int32_t hub;        /* a (SpecHub) or -1                                                   */
    uint32_t status;
} orc_node;

static void node_clear(orc_node *o) {
    memset(o, 0, sizeof(*o));
    o->accept_idx = -1; o->token = -1; o->hub = -1;
    o->margin[0] = o->margin[1] = o->margin[2] = INFINITY;
}

/* One strict multiplicative acceptance test: accept iff D > 0 and r*D < N. */
static int accept_test(double r, double N, double D, double normN, double normD, double *beta,
                       double *cond, double *margin, int performed, uint32_t *status) {
    *beta = (D > 0.0) ? dmin(N / D, 1.0) : 0.0;
    *cond = (D > 0.0) ? (normN + *beta * normD) / D : 0.0;
    if (!performed) return 0;
    if (!(D > 0.0)) { *status |= ORC_ZERO_MASS_DRAFT; *margin = INFINITY; return 0; }
    *margin = fabs(r - N / D);
    return r * D < N;
}

/* ---- Section 4: SpecHub's sparse joint draft distribution Q ----------------
 * Q(x, a) = q(x),  Q(a, x) = q(a) q(x) / (1 - q(a))  for x != a, 0 elsewhere.
 * Drawing (x1, x2) ~ Q:  the first coordinate has marginal q (sum over x of
 * Q(a, x) is q(a)), so x1 ~ q with u1; if x1 != a the pair is (x1, a); if
 * x1 = a then x2 ~ q restricted to x != a, with u2.
 * prob[0] = q(a), prob[1] = Q(x1, x2).  margin[i] = margin of draw i (inf if
 * not drawn).  1 - q(a) is summed directly as rest = sum_{x != a} q(x).
 * If rest = 0 (one-hot q) Q(a, .) is 0/0: the filler x2 = lowest id != a is
 * returned with ORC_DEGENERATE_Q; it carries no mass and is always rejected. */
unsigned orc_spechub_draft(const double *q, int V, int a, double u1, double u2,
                           int32_t tokens[2], double prob[2], double margin[2]) {
    unsigned st = 0u;
    margin[0] = margin[1] = INFINITY;
    nsum rs; ns_init(&rs);
    for (int x = 0; x < V; ++x) if (x != a) ns_add(&rs, q[x]);
    double rest = ns_val(&rs);
    int x1 = orc_inv_cdf(q, V, u1, NULL, &margin[0]);
    prob[0] = q[a];
    if (x1 != a) {
        tokens[0] = x1; tokens[1] = a; prob[1] = q[x1];
        return st;
    }
    tokens[0] = a;
    if (!(rest > 0.0)) {
        tokens[1] = (a == 0) ? 1 : 0; prob[1] = 0.0;
        return st | ORC_DEGENERATE_Q;
    }
    double *w = (double *)malloc(sizeof(double) * (size_t)V);
    memcpy(w, q, sizeof(double) * (size_t)V);
    w[a] = 0.0;
    int x2 = orc_inv_cdf(w, V, u2, NULL, &margin[1]);
    free(w);
    tokens[1] = x2; prob[1] = q[a] * q[x2] / rest;
    return st;
}

/* ---- Algorithm 2 (GetResidual) applied to one column/row of Q --------------- */
/* For x != a: p'(x) = max(p(x) - Qcol(x), 0), Q'(x) = max(Qcol(x) - p(x), 0);
 * p'(a) = p(a), Q'(a) = 0. */
static void get_residual(const double *p, const double *Qcol, int V, int a, double *p_out,
                         double *Q_out) {
    for (int x = 0; x < V; ++x) {
        if (x == a) continue;
        p_out[x] = dmax(p[x] - Qcol[x], 0.0);
        Q_out[x] = dmax(Qcol[x] - p[x], 0.0);
    }
    p_out[a] = p[a];
    Q_out[a] = 0.0;
}

/* SpecHub residual weights p''(x) = max(max(p(x)-q(x),0) - Q(a,x), 0), x != a,
 * and 0 on the hub (proof of Theorem 2, Corollary 1).  w has V entries. */
void orc_spechub_residual(const double *p, const double *q, int V, int a, double *w) {
    nsum rs; ns_init(&rs);
    for (int x = 0; x < V; ++x) if (x != a) ns_add(&rs, q[x]);
    double rest = ns_val(&rs);
    double c = rest > 0.0 ? q[a] / rest : 0.0;
    for (int x = 0; x < V; ++x) {
        if (x == a) { w[x] = 0.0; continue; }
        double p1 = dmax(p[x] - q[x], 0.0);
        w[x] = dmax(p1 - c * q[x], 0.0);
    }
}

/* ---- Algorithm 3: verification of one SpecHub draft pair --------------------
 * Steps, in the algorithm's order:
 *   Q(x,a) = q(x), Q(a,x) = q(a) q(x)/(1-q(a)).
 *   [pair (x1, a)]  accept x1 with probability min(p(x1)/Q(x1,a), 1).
 *   p', Q'(*,a) = GetResidual(p, Q(*,a), a).
 *   [pair (a, x2)]  accept x2 with probability min(p'(x2)/Q(a,x2), 1).
 *   p'', Q'(a,*) = GetResidual(p', Q(a,*), a).
 *   S2 = sum_x Q'(a,x), S1 = sum_x Q'(x,a)  (leftover mass of the two pair families).
 *   [pair (a, x2)]  accept a with probability min(p(a)/S2, 1).
 *   p'(a) = max(p(a) - S2, 0)   -- the hub mass that pairs (a, .) could not absorb.
 *   [pair (x1, a)]  accept a with probability min(p'(a)/S1, 1).
 *   otherwise draw from norm(p''), which has no mass on a.
 * Child index: child i is draft token x_i (i = 0 for x1, 1 for x2). */
void orc_spechub_verify(const double *p, const double *q, int V, int a, int x1, int x2, double r1,
                        double r2, double u_res, orc_node *out) {
    node_clear(out);
    out->hub = a;
    int pair_xa = (x2 == a && x1 != a);   /* (x, a): non-hub first  */
    int pair_ax = (x1 == a && x2 != a);   /* (a, x): hub first      */
    int x = pair_xa ? x1 : x2;
    if (!(pair_xa || pair_ax) || x < 0 || x >= V) { out->status |= ORC_TOKEN_RANGE; return; }

    double *Qxa = (double *)malloc(sizeof(double) * (size_t)V * 6);
    double *Qax = Qxa + V, *p1 = Qax + V, *Q1xa = p1 + V, *p2 = Q1xa + V, *Q1ax = p2 + V;

    nsum rs; ns_init(&rs);
    for (int y = 0; y < V; ++y) if (y != a) ns_add(&rs, q[y]);
    double rest = ns_val(&rs);                 /* 1 - q(a), summed directly */
    int degenerate = !(rest > 0.0);
    if (degenerate) out->status |= ORC_DEGENERATE_Q;
    for (int y = 0; y < V; ++y) {
        Qxa[y] = (y == a) ? 0.0 : q[y];
        Qax[y] = (y == a || degenerate) ? 0.0 : q[a] * q[y] / rest;
    }
    get_residual(p, Qxa, V, a, p1, Q1xa);      /* p',  Q'(*,a) */
    get_residual(p1, Qax, V, a, p2, Q1ax);     /* p'', Q'(a,*) */
    p2[a] = 0.0;                               /* residual carries no hub mass */

    nsum s1, s2, m1, m2, rr; ns_init(&s1); ns_init(&s2); ns_init(&m1); ns_init(&m2); ns_init(&rr);
    double nS1 = 0.0, nS2 = 0.0;               /* term magnitudes, for cond[] only */
    for (int y = 0; y < V; ++y) {
        if (y == a) continue;
        if (Q1xa[y] > 0.0) nS1 += Qxa[y] + p[y];
#ifndef ORC_PLANT_COND_NS2   /* (the pins of cond[] build a copy with the term dropped and must then fail) */
        if (Q1ax[y] > 0.0) nS2 += 3.0 * Qax[y] + (p1[y] > 0.0 ? p[y] + Qxa[y] : 0.0);
#else
        if (Q1ax[y] > 0.0) nS2 += 3.0 * Qax[y];
#endif
        ns_add(&s1, Q1xa[y]);
        ns_add(&s2, Q1ax[y]);
        ns_add(&m1, dmin(p[y], Qxa[y]));       /* pi(x,a,x) */
        ns_add(&m2, dmin(p1[y], Qax[y]));      /* pi(a,x,x) */
        ns_add(&rr, p2[y]);
    }
    double S1 = ns_val(&s1), S2 = ns_val(&s2), R = ns_val(&rr);
    if (degenerate) { S2 = q[a]; nS2 = q[a]; } /* all of Q(a, .)'s mass is leftover */
    double hub_after_ax = dmax(p[a] - S2, 0.0);
    out->rate[0] = ns_val(&m1) + dmin(p[a], S2);
    out->rate[1] = ns_val(&m2) + dmin(hub_after_ax, S1);
    out->rate[2] = R;

    int acc = 0;
    if (pair_xa) {
        acc = accept_test(r1, p[x], Qxa[x], p[x], Qxa[x], &out->beta[0], &out->cond[0],
                          &out->margin[0], 1, &out->status);
        if (acc) { out->accept_idx = 0; out->token = x; }
        int acc2 = accept_test(r2, hub_after_ax, S1, p[a] + nS2, nS1, &out->beta[1], &out->cond[1],
                               &out->margin[1], !acc, &out->status);
        if (!acc && acc2) { out->accept_idx = 1; out->token = a; acc = 1; }
    } else {
        acc = accept_test(r1, p1[x], Qax[x], p[x] + Qxa[x], 3.0 * Qax[x], &out->beta[0], &out->cond[0],
                          &out->margin[0], 1, &out->status);
        if (acc) { out->accept_idx = 1; out->token = x; }
        int acc2 = accept_test(r2, p[a], S2, p[a], nS2, &out->beta[1], &out->cond[1],
                               &out->margin[1], !acc, &out->status);
        if (!acc && acc2) { out->accept_idx = 0; out->token = a; acc = 1; }
    }
    if (!acc) {
        int tok = orc_inv_cdf(p2, V, u_res, NULL, &out->margin[2]);
        if (tok < 0) {                          /* no residual mass: draw from p */
            out->status |= ORC_ZERO_RESIDUAL;
            tok = orc_inv_cdf(p, V, u_res, NULL, &out->margin[2]);
        }
        out->accept_idx = -1; out->token = tok;
    }
    free(Qxa);
}

/* ---- Algorithm 1, draft step: k = 2 samples from q ---------------------------
 * independently (RRS), or without replacement (RRSw): the second draw is from
 * q with q(x1) set to 0 and renormalised. */
unsigned orc_rrs_draft(const double *q, int V, int without_replacement, double u1, double u2,
                       int32_t tokens[2], double margin[2]) {
    unsigned st = 0u;
    margin[0] = margin[1] = INFINITY;
    int x1 = orc_inv_cdf(q, V, u1, NULL, &margin[0]);
    tokens[0] = x1;
    if (!without_replacement) {
        tokens[1] = orc_inv_cdf(q, V, u2, NULL, &margin[1]);
        return st;
    }
    double *w = (double *)malloc(sizeof(double) * (size_t)V);
    memcpy(w, q, sizeof(double) * (size_t)V);
    w[x1] = 0.0;
    int x2 = orc_inv_cdf(w, V, u2, NULL, &margin[1]);
    free(w);
    if (x2 < 0) { x2 = (x1 == 0) ? 1 : 0; st |= ORC_DEGENERATE_Q; margin[1] = INFINITY; }
    tokens[1] = x2;
    return st;
}

/* Stage-2 quantities of Algorithm 1 for a rejected first draft x1:
 * p_1 = norm(max(p - q, 0)) with A1 = sum max(p - q, 0);  q_1 = q (RRS) or q
 * with q(x1) zeroed and renormalised (RRSw).  Returns A1; fills p1, q1. */
static double rrs_stage2(const double *p, const double *q, int V, int x1, int without_replacement,
                         double *p1, double *q1, uint32_t *status) {
    nsum a1; ns_init(&a1);
    for (int y = 0; y < V; ++y) { p1[y] = dmax(p[y] - q[y], 0.0); ns_add(&a1, p1[y]); }
    double A1 = ns_val(&a1);
    if (A1 > 0.0) for (int y = 0; y < V; ++y) p1[y] /= A1;
    if (!without_replacement) {
        memcpy(q1, q, sizeof(double) * (size_t)V);
    } else {
        nsum d; ns_init(&d);
        for (int y = 0; y < V; ++y) if (y != x1) ns_add(&d, q[y]);
        double den = ns_val(&d);
        if (!(den > 0.0)) {
            if (status) *status |= ORC_DEGENERATE_Q;
            for (int y = 0; y < V; ++y) q1[y] = 0.0;
        } else {
            for (int y = 0; y < V; ++y) q1[y] = (y == x1) ? 0.0 : q[y] / den;
        }
    }
    return A1;
}

/* RRS / RRSw residual weights after both drafts are rejected, scaled by A1:
 * w(y) = A1 * max(p_1(y) - q_1(y), 0). */
void orc_rrs_residual(const double *p, const double *q, int V, int x1, int without_replacement,
                      double *w) {
    double *p1 = (double *)malloc(sizeof(double) * (size_t)V * 2), *q1 = p1 + V;
    double A1 = rrs_stage2(p, q, V, x1, without_replacement, p1, q1, NULL);
    for (int y = 0; y < V; ++y) w[y] = A1 * dmax(p1[y] - q1[y], 0.0);
    free(p1);
}

/* ---- Algorithm 1: verification of the k = 2 drafts ---------------------------
 *   i = 1: accept x1 iff r1 < p(x1)/q(x1);
 *          else p <- norm(max(p - q, 0)); [RRSw: q(x1) <- 0, q <- norm(q)]
 *   i = 2: accept x2 iff r2 < p(x2)/q(x2) with the updated p, q;
 *          else p <- norm(max(p - q, 0));
 *   return x ~ p.
 * rate[] = (sum min(p,q), A1 * sum min(p_1,q_1), A1 * sum max(p_1-q_1,0)):
 * the masses of accepting the first draft, of accepting the second after the
 * first was rejected, and of rejecting both; for RRSw the last two are for
 * the given first draft x1 (q_1 depends on it). */
void orc_rrs_verify(const double *p, const double *q, int V, int x1, int x2, double r1, double r2,
                    double u_res, int without_replacement, orc_node *out) {
    node_clear(out);
    if (x1 < 0 || x1 >= V || x2 < 0 || x2 >= V) { out->status |= ORC_TOKEN_RANGE; return; }
    double *p1 = (double *)malloc(sizeof(double) * (size_t)V * 3), *q1 = p1 + V, *p2 = q1 + V;
    uint32_t st2 = 0u;
    double A1 = rrs_stage2(p, q, V, x1, without_replacement, p1, q1, &st2);
    nsum m1, m2, w2; ns_init(&m1); ns_init(&m2); ns_init(&w2);
    double nA1 = 0.0;                           /* term magnitudes of A1, for cond[] only */
    for (int y = 0; y < V; ++y) if (p[y] > q[y]) nA1 += p[y] + q[y];
    for (int y = 0; y < V; ++y) {
        ns_add(&m1, dmin(p[y], q[y]));
        ns_add(&m2, dmin(p1[y], q1[y]));
        p2[y] = dmax(p1[y] - q1[y], 0.0);
        ns_add(&w2, p2[y]);
    }
    out->rate[0] = ns_val(&m1);
    out->rate[1] = A1 * ns_val(&m2);
    out->rate[2] = A1 * ns_val(&w2);

    int acc = accept_test(r1, p[x1], q[x1], p[x1], q[x1], &out->beta[0], &out->cond[0],
                          &out->margin[0], 1, &out->status);
    if (acc) { out->accept_idx = 0; out->token = x1; }
    if (!acc) out->status |= st2;
    int acc2 = 0;
    if (A1 > 0.0) {
        /* p_1(x2) = max(p - q, 0)(x2) / A1: both its own subtraction and A1's terms enter */
#ifndef ORC_PLANT_COND_NN    /* (as above: a planted mistake for the pins of cond[]) */
        double nN = (p[x2] + q[x2]) / A1 + p1[x2] * nA1 / A1;
#else
        double nN = (p[x2] + q[x2]) / A1;
#endif
        acc2 = accept_test(r2, p1[x2], q1[x2], nN, (without_replacement ? 2.0 : 1.0) * q1[x2], &out->beta[1],
                           &out->cond[1],
                           &out->margin[1], !acc, &out->status);
    } else {
        out->beta[1] = 0.0;
    }
    if (!acc && acc2) { out->accept_idx = 1; out->token = x2; acc = 1; }
    if (!acc) {
        int tok = (A1 > 0.0) ? orc_inv_cdf(p2, V, u_res, NULL, &out->margin[2]) : -1;
        if (tok < 0) {
            out->status |= ORC_ZERO_RESIDUAL;
            tok = orc_inv_cdf(p, V, u_res, NULL, &out->margin[2]);
        }
        out->accept_idx = -1; out->token = tok;
    }
    free(p1);
}

/* ======================= batch / tree level ================================= */
/* Layout shared by all batch calls: logits [B][N][V] (float, already holding
 * the storage-rounded values), uniforms [B][N][5] = (u_d1, u_d2, r1, r2,
 * u_res), draft tokens [B][N][2], temperature per sequence [B].
 * method: 0 = SpecHub, 1 = RRS, 2 = RRSw. */

void orc_draft_batch(int method, const float *draft_logits, const float *temperature, int B, int N,
                     int V, const float *uniforms, int32_t *tokens, int32_t *hub, double *prob,
                     double *margin, uint32_t *status) {
    double *q = (double *)malloc(sizeof(double) * (size_t)V);
    for (long r = 0; r < (long)B * N; ++r) {
        const float *lq = draft_logits + (size_t)r * V;
        const float *u = uniforms + (size_t)r * 5;
        int32_t *tk = tokens + r * 2;
        tk[0] = tk[1] = -1; hub[r] = -1; prob[2 * r] = prob[2 * r + 1] = 0.0;
        margin[2 * r] = margin[2 * r + 1] = INFINITY;
        unsigned st = orc_softmax(lq, V, (double)temperature[r / N], q);
        if (st) { status[r] = st; continue; }
        if (method == 0) {
            int a = orc_hub(lq, V);
            hub[r] = a;
            st = orc_spechub_draft(q, V, a, u[0], u[1], tk, prob + 2 * r, margin + 2 * r);
        } else {
            st = orc_rrs_draft(q, V, method == 2, u[0], u[1], tk, margin + 2 * r);
        }
        status[r] = st;
    }
    free(q);
}

/* node_kind[n] (may be NULL = all 0): 0 = verify the node's two children,
 * 1 = leaf: draw the bonus token from p with u_res (Figure 2: the token
 * generated after the last accepted draft). */
void orc_verify_batch(int method, const float *target_logits, const float *draft_logits,
                      const float *temperature, int B, int N, int V, const uint8_t *node_kind,
                      const int32_t *draft_tokens, const float *uniforms, orc_node *out) {
    double *p = (double *)malloc(sizeof(double) * (size_t)V * 2), *q = p + V;
    for (long r = 0; r < (long)B * N; ++r) {
        int n = (int)(r % N);
        const float *u = uniforms + (size_t)r * 5;
        orc_node *o = out + r;
        node_clear(o);
        double T = (double)temperature[r / N];
        unsigned st = orc_softmax(target_logits + (size_t)r * V, V, T, p);
        if (st) { o->status = st; continue; }
        if (node_kind && node_kind[n] == 1) {
            o->token = orc_inv_cdf(p, V, u[4], NULL, &o->margin[2]);
            o->rate[2] = 1.0;
            continue;
        }
        st = orc_softmax(draft_logits + (size_t)r * V, V, T, q);
        if (st) { o->status = st; continue; }
        int x1 = draft_tokens[2 * r], x2 = draft_tokens[2 * r + 1];
        if (method == 0) {
            int a = orc_hub(draft_logits + (size_t)r * V, V);
            orc_spechub_verify(p, q, V, a, x1, x2, u[2], u[3], u[4], o);
        } else {
            orc_rrs_verify(p, q, V, x1, x2, u[2], u[3], u[4], method == 2, o);
        }
    }
    free(p);
}

/* ---- Figure 2: walk the token tree ------------------------------------------
 * Start at the root; at a verify node follow the accepted child, or stop with
 * the residual token; at a leaf stop with the bonus token.  child[n][i] is the
 * node reached by accepting draft i of node n (NULL = heap order 2n+1+i); a
 * child < 0 or >= N ends the walk after the accepted token.  At most `levels`
 * nodes are visited.  path_nodes / path_tokens are [B][levels], padded with -1.
 * A node whose token is -1 (flagged row) ends the walk without emitting. */
void orc_walk(const int32_t *accept_idx, const int32_t *token, int B, int N, const int32_t *child,
              const uint8_t *node_kind, int levels, int32_t *n_accepted, int32_t *n_emitted,
              int32_t *path_nodes, int32_t *path_tokens) {
    for (int b = 0; b < B; ++b) {
        int32_t *pn = path_nodes + (size_t)b * levels, *pt = path_tokens + (size_t)b * levels;
        for (int i = 0; i < levels; ++i) { pn[i] = -1; pt[i] = -1; }
        int n = 0, acc = 0, emitted = 0;
        for (int step = 0; step < levels && n >= 0 && n < N; ++step) {
            long r = (long)b * N + n;
            pn[step] = n;
            if (token[r] < 0) break;
            pt[step] = token[r];
            ++emitted;
            if (node_kind && node_kind[n] == 1) break;
            int idx = accept_idx[r];
            if (idx < 0) break;
            ++acc;
            n = child ? child[2 * n + idx] : 2 * n + 1 + idx;
        }
        n_accepted[b] = acc; n_emitted[b] = emitted;
    }
}


/* ======================= Algorithm 1 for general k ============================
 * The paper states Algorithm 1 for k candidates (its ternary trees and the
 * 10-draft acceptance decay of Appendix C use k > 2).  Layout of the uniforms
 * of a node: (u_d1..u_dk, r_1..r_k, u_res), 2k+1 values.
 *
 * Draft step: k samples from q independently (RRS) or without replacement
 * (RRSw: after each draw q(x_i) <- 0 and q is renormalised). */
unsigned orc_rrs_k_draft(const double *q, int V, int k, int without_replacement, const double *u,
                         int32_t *tokens, double *margin) {
    unsigned st = 0u;
    double *w = (double *)malloc(sizeof(double) * (size_t)V);
    memcpy(w, q, sizeof(double) * (size_t)V);
    for (int i = 0; i < k; ++i) {
        margin[i] = INFINITY;
        int x = orc_inv_cdf(w, V, u[i], NULL, &margin[i]);
        if (x < 0) {              /* nothing left to draw from: lowest id not drawn yet */
            st |= ORC_DEGENERATE_Q;
            margin[i] = INFINITY;
            for (x = 0; x < V; ++x) {
                int used = 0;
                for (int j = 0; j < i; ++j) used |= (tokens[j] == x);
                if (!used) break;
            }
            if (x >= V) x = 0;
        }
        tokens[i] = x;
        if (without_replacement) w[x] = 0.0;   /* the draw normalises by the remaining mass */
    }
    free(w);
    return st;
}

/* Verification of k drafts, Algorithm 1 step by step:
 *   for i = 1..k: accept x_i iff r_i < p(x_i)/q(x_i) (strict, multiplicative; q(x_i) = 0 rejects);
 *                 else p <- norm(max(p - q, 0)); [RRSw: q(x_i) <- 0, q <- norm(q)]
 *   return x ~ p.
 * Outputs: accept_idx in {-1, 0..k-1}; token; beta[k] (acceptance probability of test i, given
 * that it is reached); rate[k+1] (mass of accepting at stage i for these drafts -- unconditional
 * for RRS stage 1 only -- and of rejecting all); margin[k+1]; cond[k]; status.
 * If a residual has no mass (p = q so far) the draw falls back to the original p with
 * ORC_ZERO_RESIDUAL, and later tests have beta = 0. */
void orc_rrs_k_verify(const double *p0, const double *q0, int V, int k, const int32_t *x,
                      const double *r, double u_res, int without_replacement, int32_t *accept_idx,
                      int32_t *token, double *beta, double *rate, double *margin, double *cond,
                      uint32_t *status) {
    *accept_idx = -1; *token = -1; *status = 0u;
    for (int i = 0; i < k; ++i) { beta[i] = 0.0; cond[i] = 0.0; margin[i] = INFINITY; rate[i] = 0.0; }
    margin[k] = INFINITY; rate[k] = 0.0;
    for (int i = 0; i < k; ++i)
        if (x[i] < 0 || x[i] >= V) { *status |= ORC_TOKEN_RANGE; return; }
    double *p = (double *)malloc(sizeof(double) * (size_t)V * 3), *q = p + V, *mag = q + V;
    memcpy(p, p0, sizeof(double) * (size_t)V);
    memcpy(q, q0, sizeof(double) * (size_t)V);
    for (int y = 0; y < V; ++y) mag[y] = p0[y];     /* |terms| of p(y), for cond[] only */
    double mass = 1.0;       /* probability of reaching the current stage with these drafts' stages */
    double amp = 1.0;        /* growth of the relative error through the normalisations          */
    int accepted = 0, alive = 1;
    for (int i = 0; i < k; ++i) {
        int performed = alive && !accepted;
        int xi = x[i];
        double N = p[xi], D = q[xi];
        beta[i] = (alive && D > 0.0) ? dmin(N / D, 1.0) : 0.0;
        cond[i] = (alive && D > 0.0) ? (mag[xi] * amp + beta[i] * D) / D : 0.0;
        /* mass accepted at this stage: sum_y min(p, q) of the current pair, times the mass so far */
        nsum acc; ns_init(&acc);
        if (alive) for (int y = 0; y < V; ++y) ns_add(&acc, dmin(p[y], q[y]));
        rate[i] = alive ? mass * ns_val(&acc) : 0.0;
        if (performed) {
            if (!(D > 0.0)) { *status |= ORC_ZERO_MASS_DRAFT; }
            else {
                margin[i] = fabs(r[i] - N / D);
                if (r[i] * D < N) { accepted = 1; *accept_idx = i; *token = xi; }
            }
        }
        if (!alive) continue;
        /* p <- norm(max(p - q, 0)) */
        nsum a; ns_init(&a);
        double nA = 0.0;
        for (int y = 0; y < V; ++y) {
            double d = p[y] - q[y];
            if (d > 0.0) { mag[y] = mag[y] + q[y]; nA += mag[y]; p[y] = d; } else { p[y] = 0.0; mag[y] = 0.0; }
            ns_add(&a, p[y]);
        }
        double A = ns_val(&a);
        mass *= A;
        if (A > 0.0) {
            for (int y = 0; y < V; ++y) { p[y] /= A; mag[y] /= A; }
            amp += nA / A;
        } else {
            alive = 0;
        }
        if (without_replacement && alive) {
            q[xi] = 0.0;
            nsum d; ns_init(&d);
            for (int y = 0; y < V; ++y) ns_add(&d, q[y]);
            double den = ns_val(&d);
            if (den > 0.0) { for (int y = 0; y < V; ++y) q[y] /= den; }
            else { if (!accepted) *status |= ORC_DEGENERATE_Q; }
        }
    }
    rate[k] = mass;
    if (!accepted) {
        int tok = alive ? orc_inv_cdf(p, V, u_res, NULL, &margin[k]) : -1;
        if (tok < 0) {
            *status |= ORC_ZERO_RESIDUAL;
            tok = orc_inv_cdf(p0, V, u_res, NULL, &margin[k]);
        }
        *token = tok;
    }
    free(p);
}

/* Residual weights after all k drafts were rejected (unnormalised); 0 mass if none. */
void orc_rrs_k_residual(const double *p0, const double *q0, int V, int k, const int32_t *x,
                        int without_replacement, double *w) {
    double *q = (double *)malloc(sizeof(double) * (size_t)V);
    memcpy(w, p0, sizeof(double) * (size_t)V);
    memcpy(q, q0, sizeof(double) * (size_t)V);
    for (int i = 0; i < k; ++i) {
        nsum a; ns_init(&a);
        for (int y = 0; y < V; ++y) { w[y] = dmax(w[y] - q[y], 0.0); ns_add(&a, w[y]); }
        double A = ns_val(&a);
        if (!(A > 0.0)) break;
        for (int y = 0; y < V; ++y) w[y] /= A;
        if (without_replacement) {
            q[x[i]] = 0.0;
            nsum d; ns_init(&d);
            for (int y = 0; y < V; ++y) ns_add(&d, q[y]);
            double den = ns_val(&d);
            if (den > 0.0) for (int y = 0; y < V; ++y) q[y] /= den;
        }
    }
    free(q);
}

void orc_rrs_k_draft_batch(int k, int without_replacement, const float *draft_logits,
                           const float *temperature, int B, int N, int V, const float *uniforms,
                           int32_t *tokens, double *margin, uint32_t *status) {
    double *q = (double *)malloc(sizeof(double) * (size_t)V);
    double u[64];
    const int nu = 2 * k + 1;
    for (long r = 0; r < (long)B * N; ++r) {
        for (int i = 0; i < k; ++i) { tokens[r * k + i] = -1; margin[r * k + i] = INFINITY; }
        unsigned st = orc_softmax(draft_logits + (size_t)r * V, V, (double)temperature[r / N], q);
        if (st) { status[r] = st; continue; }
        for (int i = 0; i < k; ++i) u[i] = (double)uniforms[(size_t)r * nu + i];
        status[r] = orc_rrs_k_draft(q, V, k, without_replacement, u, tokens + r * k, margin + r * k);
    }
    free(q);
}

void orc_rrs_k_verify_batch(int k, int without_replacement, const float *target_logits,
                            const float *draft_logits, const float *temperature, int B, int N, int V,
                            const uint8_t *node_kind, const int32_t *draft_tokens,
                            const float *uniforms, int32_t *accept_idx, int32_t *token, double *beta,
                            double *rate, double *margin, double *cond, uint32_t *status) {
    double *p = (double *)malloc(sizeof(double) * (size_t)V * 2), *q = p + V;
    double rr[64];
    const int nu = 2 * k + 1;
    for (long r = 0; r < (long)B * N; ++r) {
        int n = (int)(r % N);
        const float *u = uniforms + (size_t)r * nu;
        accept_idx[r] = -1; token[r] = -1; status[r] = 0u;
        for (int i = 0; i < k; ++i) { beta[r * k + i] = 0.0; cond[r * k + i] = 0.0; }
        for (int i = 0; i <= k; ++i) { rate[r * (k + 1) + i] = 0.0; margin[r * (k + 1) + i] = INFINITY; }
        double T = (double)temperature[r / N];
        unsigned st = orc_softmax(target_logits + (size_t)r * V, V, T, p);
        if (st) { status[r] = st; continue; }
        if (node_kind && node_kind[n] == 1) {
            token[r] = orc_inv_cdf(p, V, u[2 * k], NULL, &margin[r * (k + 1) + k]);
            rate[r * (k + 1) + k] = 1.0;
            continue;
        }
        st = orc_softmax(draft_logits + (size_t)r * V, V, T, q);
        if (st) { status[r] = st; continue; }
        for (int i = 0; i < k; ++i) rr[i] = (double)u[k + i];
        orc_rrs_k_verify(p, q, V, k, draft_tokens + r * k, rr, (double)u[2 * k], without_replacement,
                         accept_idx + r, token + r, beta + r * k, rate + r * (k + 1),
                         margin + r * (k + 1), cond + r * k, status + r);
    }
    free(p);
}

/* Tree walk with k children per node: child[n][i] (NULL = complete k-ary tree in level order,
 * child i of n is k*n + 1 + i). */
void orc_walk_k(int k, const int32_t *accept_idx, const int32_t *token, int B, int N,
                const int32_t *child, const uint8_t *node_kind, int levels, int32_t *n_accepted,
                int32_t *n_emitted, int32_t *path_nodes, int32_t *path_tokens) {
    for (int b = 0; b < B; ++b) {
        int32_t *pn = path_nodes + (size_t)b * levels, *pt = path_tokens + (size_t)b * levels;
        for (int i = 0; i < levels; ++i) { pn[i] = -1; pt[i] = -1; }
        int n = 0, acc = 0, emitted = 0;
        for (int step = 0; step < levels && n >= 0 && n < N; ++step) {
            long r = (long)b * N + n;
            pn[step] = n;
            if (token[r] < 0) break;
            pt[step] = token[r];
            ++emitted;
            if (node_kind && node_kind[n] == 1) break;
            int idx = accept_idx[r];
            if (idx < 0) break;
            ++acc;
            n = child ? child[k * n + idx] : k * n + 1 + idx;
        }
        n_accepted[b] = acc; n_emitted[b] = emitted;
    }
}

size_t orc_node_size(void) { return sizeof(orc_node); }
