// General streaming kernels: one CTA per (sequence, node) row, any vocabulary
// size, fp32 or bf16 logits, aligned or not.  Pass A reads the row(s) from HBM;
// the later passes re-read them, which hit L2 while the row pair is still
// there.  Large bf16 vocabularies with aligned rows take the kernels of
// spechub_lean.cuh instead; these remain the path for every other shape.
#pragma once

#include "spechub.h"
#include "spechub_common.cuh"

namespace spechub {

struct RowArgs {
    const void *target;   // [B][N][V] (verify only)
    const void *draft;    // [B][N][V]
    const float *uniforms;  // [B][N][5]
    const int32_t *draft_tokens_in;  // verify: [B][N][2]
    int32_t *draft_tokens_out;       // draft: [B][N][2]
    int32_t *hub;
    float *draft_prob;
    int32_t *accept_idx;
    int32_t *token;
    float *beta;
    float *rate;
    uint32_t *status;
    const float *temperature_per_seq;
    const uint8_t *node_kind;
    float temperature;
    int nodes, vocab;
    long long stride_seq, stride_node;
    // per-row statistics of the draft logits, handed from the draft step to verification: [B][N] DraftStat
    void *draft_stats_out;       // draft step, may be NULL
    const void *draft_stats_in;  // verification through a *_stats entry point
};

// What the draft step knows about a row of draft logits once it has read it, and what verification would
// otherwise have to read the row for a second time to find out (Section 4: a = argmax q; q(a); 1 - q(a)).
struct DraftStat {
    float ml;       // the row's maximum logit
    float sx;       // sum over ids != argmax of 2^(k l - k ml), k = log2(e) / T
    int idx;        // argmax, lowest id on ties
    unsigned tag;   // kDraftStatTag ^ bits of k: a record of another library version or temperature is refused
};
constexpr unsigned kDraftStatTag = 0x51a75u << 12;
// a draft kernel that keeps no statistics leaves a record that no verification accepts
__device__ __forceinline__ void void_draft_stat(const RowArgs &a, long long r) {
    if (a.draft_stats_out) static_cast<uint4 *>(a.draft_stats_out)[r] = make_uint4(0u, 0u, 0u, 0u);
}

enum Method { kSpecHub = 0, kRRS = 1, kRRSw = 2 };

struct WarpPart {  // per-warp (max, argmax, sum without the argmax) of one row
    float ml[kMaxWarps], sx[kMaxWarps];
    int idx[kMaxWarps];
};
struct Partials {  // per-warp partials kept for the samplers, in shared memory
    WarpPart p, q;
    float acc[4][kMaxWarps];
    float mass[kMaxWarps];
    float bc[16];
    int bi[8];
    int tok;
};

__device__ __forceinline__ float temperature_of(const RowArgs &a, int b) {
    return a.temperature_per_seq ? a.temperature_per_seq[b] : a.temperature;
}

// Pass A over one row: per-warp (max, argmax, sum without the argmax) to shared memory; the
// block-wide result is returned to every thread.  Target and draft rows go through the same
// arithmetic, so identical rows give bit-identical probabilities (p = q then cancels exactly).
template <typename LT, bool AL>
__device__ ArgMaxSum pass_a(const Geo &g, const LT *row, float k, WarpPart &wp) {
    constexpr int VW = VecOf<LT>::W;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    ArgMaxSum st;
    st.init();
    for (int vi = g.seg_lo(warp) + lane; vi < g.seg_hi(warp); vi += 32) {
        float v[VW];
        load_vec<LT, AL>(row, vi, g.V, v);
        argmaxsum_push<VW>(st, v, vi * VW, k);
    }
    st = argmaxsum_warp(st, k);
    if (lane == 0) { wp.ml[warp] = st.ml; wp.sx[warp] = st.sx; wp.idx[warp] = st.idx; }
    __syncthreads();
    ArgMaxSum tot;
    tot.init();
    for (int w = 0; w < g.nwarps; ++w) {
        ArgMaxSum o;
        o.ml = wp.ml[w]; o.c = shift_of(o.ml, k); o.sx = wp.sx[w]; o.idx = wp.idx[w];
        tot = argmaxsum_merge(tot, o, k);
    }
    return tot;
}

// Probability of one logit.  The product is rounded on its own (no contraction into a later
// subtraction), so that identical target and draft rows give p(y) - q(y) = 0 exactly.
__device__ __forceinline__ float prob_of(float logit, float k, float c, float invZ) {
    return __fmul_rn(ex2(__fmaf_rn(logit, k, -c)), invZ);
}
// d = p - q and t = max(p - q, 0) - s*q, with pinned rounding so that the sums of pass B and
// the weights the sampler recomputes are the same numbers.
__device__ __forceinline__ void transport_terms(float pp, float qq, float s, float &d, float &t) {
    d = __fsub_rn(pp, qq);
    t = __fmaf_rn(-s, qq, fmaxf(d, 0.f));
}

__device__ __forceinline__ bool finite_pos(float x) { return x > 0.f && x < __int_as_float(0x7f800000); }

// Draw from softmax(row) with token `excl` removed (excl < 0: nothing removed).
// Uses the per-warp partials of pass_a; `hubtok` is the row's argmax, cQ its shift.
template <typename LT, bool AL>
__device__ int sample_row(const Geo &g, const LT *row, float k, float cQ, int hubtok, int excl,
                          float u, const WarpPart &wp, Partials &sh) {
    constexpr int VW = VecOf<LT>::W;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x < g.nwarps) {
        const int w = threadIdx.x;
        const float ml = wp.ml[w];
        const bool holds_hub = (wp.idx[w] == hubtok);
        // the warp's partial leaves out its own argmax: add it back unless it is the excluded hub
        const float own = (holds_hub && excl == hubtok) ? 0.f : own_term(ml, k);
        sh.mass[w] = (wp.sx[w] + own) * rescale(ml, shift_of(ml, k), cQ);
    }
    __syncthreads();
    if (excl >= 0 && excl != hubtok) {
        // an arbitrary token is removed (RRS without replacement): its warp re-sums its range
        const int wex = (excl / VW) / g.seg;
        if (warp == wex) {
            float s = 0.f;
            for (int vi = g.seg_lo(warp) + lane; vi < g.seg_hi(warp); vi += 32) {
                float v[VW];
                load_vec<LT, AL>(row, vi, g.V, v);
#pragma unroll
                for (int i = 0; i < VW; ++i) s += (vi * VW + i == excl) ? 0.f : ex2(fmaf(v[i], k, -cQ));
            }
            s = warp_sum(s);
            if (lane == 0) sh.mass[warp] = s;
        }
        __syncthreads();
    }
    auto wf = [&](int vi, float(&w)[VW]) {
        float v[VW];
        load_vec<LT, AL>(row, vi, g.V, v);
#pragma unroll
        for (int i = 0; i < VW; ++i) w[i] = (vi * VW + i == excl) ? 0.f : ex2(fmaf(v[i], k, -cQ));
    };
    return block_sample<VW>(g, wf, sh.mass, u, &sh.tok);
}

// ------------------------------------------------------------------------------------------------
// Draft step (Section 4 / Algorithm 3 for SpecHub; Algorithm 1 for RRS, RRSw).
// ------------------------------------------------------------------------------------------------
template <typename LT, bool AL>
__global__ void __launch_bounds__(512) draft_rows_kernel(RowArgs a, int method) {
    constexpr int VW = VecOf<LT>::W;
    __shared__ Partials sh;
    const long long r = blockIdx.x;
    const int b = static_cast<int>(r / a.nodes), n = static_cast<int>(r % a.nodes);
    const LT *rowq = static_cast<const LT *>(a.draft) + b * a.stride_seq + n * a.stride_node;
    const Geo g = make_geo(a.vocab, VW);
    const float k = kLog2e / temperature_of(a, b);
    const float u1 = a.uniforms[r * 5 + 0], u2 = a.uniforms[r * 5 + 1];

    const ArgMaxSum q = pass_a<LT, AL>(g, rowq, k, sh.q);
    const float eq_a = q.own(k);   // the hub's own term, 2^(k l(a) - c)
    const float Zq = q.sx + eq_a;
    uint32_t st = 0;
    int x1 = -1, x2 = -1, hubtok = -1;
    float prob0 = 0.f, prob1 = 0.f;
    if (!(q.ml > neg_inf()) || !finite_pos(Zq) || !(q.ml < -neg_inf())) {
        st = SPECHUB_ST_NONFINITE;
    } else {
        hubtok = q.idx;
        x1 = sample_row<LT, AL>(g, rowq, k, q.c, hubtok, -1, u1, sh.q, sh);
        if (method == kSpecHub) {
            prob0 = eq_a / Zq;
            if (x1 != hubtok) {
                x2 = hubtok;
                prob1 = ex2(fmaf(load_one<LT>(rowq, x1), k, -q.c)) / Zq;
            } else if (!(q.sx > 0.f)) {
                x2 = (hubtok == 0) ? 1 : 0;
                st |= SPECHUB_ST_DEGENERATE_Q;
            } else {
                x2 = sample_row<LT, AL>(g, rowq, k, q.c, hubtok, hubtok, u2, sh.q, sh);
                prob1 = prob0 * ex2(fmaf(load_one<LT>(rowq, x2), k, -q.c)) / q.sx;
            }
        } else if (method == kRRS) {
            x2 = sample_row<LT, AL>(g, rowq, k, q.c, hubtok, -1, u2, sh.q, sh);
        } else {
            x2 = sample_row<LT, AL>(g, rowq, k, q.c, hubtok, x1, u2, sh.q, sh);
            if (x2 < 0) {
                x2 = (x1 == 0) ? 1 : 0;
                st |= SPECHUB_ST_DEGENERATE_Q;
            }
        }
    }
    if (threadIdx.x == 0) {
        void_draft_stat(a, r);
        a.draft_tokens_out[2 * r] = x1;
        a.draft_tokens_out[2 * r + 1] = x2;
        if (a.hub) a.hub[r] = (method == kSpecHub) ? hubtok : -1;
        if (a.draft_prob) { a.draft_prob[2 * r] = prob0; a.draft_prob[2 * r + 1] = prob1; }
        if (a.status) a.status[r] = st;
    }
}

// ------------------------------------------------------------------------------------------------
// Verification of one row.
// ------------------------------------------------------------------------------------------------
struct NodeResult {
    int accept_idx, token, hub;
    float beta[2], rate[3];
    uint32_t status;
};

__device__ __forceinline__ void write_node(const RowArgs &a, long long r, const NodeResult &o) {
    a.accept_idx[r] = o.accept_idx;
    a.token[r] = o.token;
    if (a.hub) a.hub[r] = o.hub;
    if (a.beta) { a.beta[2 * r] = o.beta[0]; a.beta[2 * r + 1] = o.beta[1]; }
    if (a.rate) { a.rate[3 * r] = o.rate[0]; a.rate[3 * r + 1] = o.rate[1]; a.rate[3 * r + 2] = o.rate[2]; }
    if (a.status) a.status[r] = o.status;
}

// strict multiplicative acceptance test; fills beta = min(N/D, 1)
__device__ __forceinline__ bool accept_test(float r, float N, float D, float &beta, bool performed,
                                            uint32_t &status) {
    beta = (D > 0.f) ? fminf(N / D, 1.f) : 0.f;
    if (!performed) return false;
    if (!(D > 0.f)) { status |= SPECHUB_ST_ZERO_MASS_DRAFT; return false; }
    return r * D < N;
}

// Block-wide sum of up to 4 per-thread accumulators; per-warp values stay in sh.acc[i][w].
template <int NACC>
__device__ __forceinline__ void block_sums(const Geo &g, float (&x)[NACC], Partials &sh) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
#pragma unroll
    for (int i = 0; i < NACC; ++i) {
        const float s = warp_sum(x[i]);
        if (lane == 0) sh.acc[i][warp] = s;
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < NACC; ++i) {
        float t = 0.f;
        for (int w = 0; w < g.nwarps; ++w) t += sh.acc[i][w];
        x[i] = t;
    }
}
// sh.acc may be rewritten only after every thread has read it
__device__ __forceinline__ void release_sums() { __syncthreads(); }

template <typename LT, bool AL, int METHOD>
__global__ void __launch_bounds__(512) verify_rows_kernel(RowArgs a) {
    constexpr int VW = VecOf<LT>::W;
    __shared__ Partials sh;
    const long long r = blockIdx.x;
    const int b = static_cast<int>(r / a.nodes), n = static_cast<int>(r % a.nodes);
    const LT *rowp = static_cast<const LT *>(a.target) + b * a.stride_seq + n * a.stride_node;
    const LT *rowq = static_cast<const LT *>(a.draft) + b * a.stride_seq + n * a.stride_node;
    const Geo g = make_geo(a.vocab, VW);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const float k = kLog2e / temperature_of(a, b);
    const float r1 = a.uniforms[r * 5 + 2], r2 = a.uniforms[r * 5 + 3], ures = a.uniforms[r * 5 + 4];
    const float pinf = -neg_inf();

    NodeResult o;
    o.accept_idx = -1; o.token = -1; o.hub = -1; o.status = 0;
    o.beta[0] = o.beta[1] = 0.f; o.rate[0] = o.rate[1] = o.rate[2] = 0.f;

    const ArgMaxSum P = pass_a<LT, AL>(g, rowp, k, sh.p);
    const float Zp = P.sx + P.own(k);
    if (!(P.ml > neg_inf()) || !(P.ml < pinf) || !finite_pos(Zp)) {
        o.status = SPECHUB_ST_NONFINITE;
        if (threadIdx.x == 0) write_node(a, r, o);
        return;
    }
    const float cP = P.c, invZp = 1.f / Zp;

    if (a.node_kind && a.node_kind[n] == SPECHUB_NODE_LEAF) {
        // bonus token after the last accepted draft (Figure 2): a draw from p
        o.token = sample_row<LT, AL>(g, rowp, k, cP, P.idx, -1, ures, sh.p, sh);
        o.rate[2] = 1.f;
        if (threadIdx.x == 0) write_node(a, r, o);
        return;
    }

    const ArgMaxSum Q = pass_a<LT, AL>(g, rowq, k, sh.q);
    const float eq_a = Q.own(k);   // the hub's own term, 2^(k l(a) - c)
    const float Zq = Q.sx + eq_a;
    if (!(Q.ml > neg_inf()) || !(Q.ml < pinf) || !finite_pos(Zq)) {
        o.status = SPECHUB_ST_NONFINITE;
        if (threadIdx.x == 0) write_node(a, r, o);
        return;
    }
    const float cQ = Q.c, invZq = 1.f / Zq;
    const int x1 = a.draft_tokens_in[2 * r], x2 = a.draft_tokens_in[2 * r + 1];
    auto prob_p = [&](int y) { return prob_of(load_one<LT>(rowp, y), k, cP, invZp); };
    auto prob_q = [&](int y) { return prob_of(load_one<LT>(rowq, y), k, cQ, invZq); };

    if (METHOD == kSpecHub) {
        const int hubtok = Q.idx;
        o.hub = hubtok;
        const bool pair_xa = (x2 == hubtok && x1 != hubtok), pair_ax = (x1 == hubtok && x2 != hubtok);
        const int x = pair_xa ? x1 : x2;
        if (!(pair_xa || pair_ax) || x < 0 || x >= a.vocab) {
            o.status = SPECHUB_ST_TOKEN_RANGE;
            if (threadIdx.x == 0) write_node(a, r, o);
            return;
        }
        const bool degenerate = !(Q.sx > 0.f);           // 1 - q(a) = 0
        const float c = degenerate ? 0.f : eq_a / Q.sx;    // q(a) / (1 - q(a))
        const float qa = eq_a * invZq, rest = Q.sx * invZq;
        if (!a.beta && !a.rate) {
            // No probability is asked for: the first test needs scalars only, and if it accepts the
            // transport sums decide nothing.
            const float px0 = prob_p(x), qx0 = prob_q(x);
            const bool acc0 = pair_xa ? accept_test(r1, px0, qx0, o.beta[0], true, o.status)
                                      : accept_test(r1, fmaxf(__fsub_rn(px0, qx0), 0.f), c * qx0, o.beta[0], true, o.status);
            if (acc0) {
                o.accept_idx = pair_xa ? 0 : 1;
                o.token = x;
                if (degenerate) o.status |= SPECHUB_ST_DEGENERATE_Q;
                if (threadIdx.x == 0) write_node(a, r, o);
                return;
            }
            o.status = 0;
        }
        // pass B: transport sums over ids != a (Section 4, Appendix B.1)
        float acc[3] = {0.f, 0.f, 0.f};  // S1, S2, R
        const int hubvec = hubtok / VW, hublane = hubtok % VW;
        for (int vi = g.seg_lo(warp) + lane; vi < g.seg_hi(warp); vi += 32) {
            float vp[VW], vq[VW];
            load_vec<LT, AL>(rowp, vi, g.V, vp);
            load_vec<LT, AL>(rowq, vi, g.V, vq);
            if (vi == hubvec) {
#pragma unroll
                for (int i = 0; i < VW; ++i)
                    if (i == hublane) { vp[i] = neg_inf(); vq[i] = neg_inf(); }
            }
#pragma unroll
            for (int i = 0; i < VW; ++i) {
                const float pp = prob_of(vp[i], k, cP, invZp);
                const float qq = prob_of(vq[i], k, cQ, invZq);
                float d, t;                              // d = p - q, t = p'(y) - Q(a, y)
                transport_terms(pp, qq, c, d, t);
                acc[0] += fmaxf(-d, 0.f);                // Q'(y, a)
                acc[1] += fmaxf(-t, 0.f);                // Q'(a, y)
                acc[2] += fmaxf(t, 0.f);                 // p''(y)
            }
        }
        block_sums<3>(g, acc, sh);
        const float S1 = acc[0], S2 = degenerate ? qa : acc[1], R = acc[2];
        const float pa = prob_p(hubtok);
        const float hub_left = fmaxf(pa - S2, 0.f);
        o.rate[0] = fmaxf(rest - S1, 0.f) + fminf(pa, S2);
        o.rate[1] = (degenerate ? 0.f : fmaxf(qa - S2, 0.f)) + fminf(hub_left, S1);
        o.rate[2] = R;
        if (degenerate) o.status |= SPECHUB_ST_DEGENERATE_Q;
        const float px = prob_p(x), qx = prob_q(x);
        bool acc1, acc2;
        if (pair_xa) {
            acc1 = accept_test(r1, px, qx, o.beta[0], true, o.status);
            if (acc1) { o.accept_idx = 0; o.token = x; }
            acc2 = accept_test(r2, hub_left, S1, o.beta[1], !acc1, o.status);
            if (!acc1 && acc2) { o.accept_idx = 1; o.token = hubtok; }
        } else {
            acc1 = accept_test(r1, fmaxf(__fsub_rn(px, qx), 0.f), c * qx, o.beta[0], true, o.status);
            if (acc1) { o.accept_idx = 1; o.token = x; }
            acc2 = accept_test(r2, pa, S2, o.beta[1], !acc1, o.status);
            if (!acc1 && acc2) { o.accept_idx = 0; o.token = hubtok; }
        }
        if (!(acc1 || acc2)) {
            if (threadIdx.x < g.nwarps) sh.mass[threadIdx.x] = sh.acc[2][threadIdx.x];
            __syncthreads();
            auto wf = [&](int vi, float(&w)[VW]) {
                float vp[VW], vq[VW];
                load_vec<LT, AL>(rowp, vi, g.V, vp);
                load_vec<LT, AL>(rowq, vi, g.V, vq);
#pragma unroll
                for (int i = 0; i < VW; ++i) {
                    const float pp = prob_of(vp[i], k, cP, invZp);
                    const float qq = prob_of(vq[i], k, cQ, invZq);
                    float d, t;
                    transport_terms(pp, qq, c, d, t);
                    w[i] = (vi * VW + i == hubtok) ? 0.f : fmaxf(t, 0.f);
                }
            };
            int tok = block_sample<VW>(g, wf, sh.mass, ures, &sh.tok);
            if (tok < 0) {
                o.status |= SPECHUB_ST_ZERO_RESIDUAL;
                tok = sample_row<LT, AL>(g, rowp, k, cP, P.idx, -1, ures, sh.p, sh);
            }
            o.accept_idx = -1;
            o.token = tok;
        }
    } else {
        // Algorithm 1 with k = 2
        if (x1 < 0 || x1 >= a.vocab || x2 < 0 || x2 >= a.vocab) {
            o.status = SPECHUB_ST_TOKEN_RANGE;
            if (threadIdx.x == 0) write_node(a, r, o);
            return;
        }
        if (!a.beta && !a.rate) {
            // no probability asked for: an accepted first draft needs no sum at all
            if (accept_test(r1, prob_p(x1), prob_q(x1), o.beta[0], true, o.status)) {
                o.accept_idx = 0;
                o.token = x1;
                if (threadIdx.x == 0) write_node(a, r, o);
                return;
            }
            o.status = 0;
        }
        // pass B: A1 = sum max(p - q, 0); RRSw also sums q outside x1 directly
        float acc[2] = {0.f, 0.f};
        for (int vi = g.seg_lo(warp) + lane; vi < g.seg_hi(warp); vi += 32) {
            float vp[VW], vq[VW];
            load_vec<LT, AL>(rowp, vi, g.V, vp);
            load_vec<LT, AL>(rowq, vi, g.V, vq);
#pragma unroll
            for (int i = 0; i < VW; ++i) {
                const float pp = prob_of(vp[i], k, cP, invZp);
                const float qq = prob_of(vq[i], k, cQ, invZq);
                acc[0] += fmaxf(__fsub_rn(pp, qq), 0.f);
                if (METHOD == kRRSw) acc[1] += (vi * VW + i == x1) ? 0.f : qq;
            }
        }
        block_sums<2>(g, acc, sh);
        release_sums();
        const float A1 = acc[0];
        const float den = acc[1];                       // 1 - q(x1), RRSw
        const bool q1_zero = (METHOD == kRRSw) && !(den > 0.f);
        const float gq = (METHOD == kRRSw) ? (q1_zero ? 0.f : 1.f / den) : 1.f;  // q1 = gq * q off x1
        const float A1g = A1 * gq;
        // pass C: mass of the residual after two rejections
        float w2[1] = {0.f};
        for (int vi = g.seg_lo(warp) + lane; vi < g.seg_hi(warp); vi += 32) {
            float vp[VW], vq[VW];
            load_vec<LT, AL>(rowp, vi, g.V, vp);
            load_vec<LT, AL>(rowq, vi, g.V, vq);
#pragma unroll
            for (int i = 0; i < VW; ++i) {
                const float pp = prob_of(vp[i], k, cP, invZp);
                const float qq = prob_of(vq[i], k, cQ, invZq);
                float d, t;                              // t = max(p - q, 0) - A1 q1(y)
                transport_terms(pp, qq, (METHOD == kRRSw && vi * VW + i == x1) ? 0.f : A1g, d, t);
                w2[0] += fmaxf(t, 0.f);
            }
        }
        block_sums<1>(g, w2, sh);
        const float W2 = w2[0];
        o.rate[0] = fmaxf(1.f - A1, 0.f);
        o.rate[1] = fmaxf(A1 - W2, 0.f);
        o.rate[2] = W2;
        const float px1 = prob_p(x1), qx1 = prob_q(x1), px2 = prob_p(x2), qx2 = prob_q(x2);
        const bool acc1 = accept_test(r1, px1, qx1, o.beta[0], true, o.status);
        if (acc1) { o.accept_idx = 0; o.token = x1; }
        if (!acc1 && q1_zero) o.status |= SPECHUB_ST_DEGENERATE_Q;
        bool acc2 = false;
        if (A1 > 0.f) {
            const float q1x2 = (METHOD == kRRSw && x2 == x1) ? 0.f : A1g * qx2;
            acc2 = accept_test(r2, fmaxf(__fsub_rn(px2, qx2), 0.f), q1x2, o.beta[1], !acc1, o.status);
        }
        if (!acc1 && acc2) { o.accept_idx = 1; o.token = x2; }
        if (!(acc1 || acc2)) {
            int tok = -1;
            if (A1 > 0.f) {
                if (threadIdx.x < g.nwarps) sh.mass[threadIdx.x] = sh.acc[0][threadIdx.x];
                __syncthreads();
                auto wf = [&](int vi, float(&w)[VW]) {
                    float vp[VW], vq[VW];
                    load_vec<LT, AL>(rowp, vi, g.V, vp);
                    load_vec<LT, AL>(rowq, vi, g.V, vq);
#pragma unroll
                    for (int i = 0; i < VW; ++i) {
                        const float pp = prob_of(vp[i], k, cP, invZp);
                        const float qq = prob_of(vq[i], k, cQ, invZq);
                        float d, t;
                        transport_terms(pp, qq, (METHOD == kRRSw && vi * VW + i == x1) ? 0.f : A1g, d, t);
                        w[i] = fmaxf(t, 0.f);
                    }
                };
                tok = block_sample<VW>(g, wf, sh.mass, ures, &sh.tok);
            }
            if (tok < 0) {
                o.status |= SPECHUB_ST_ZERO_RESIDUAL;
                tok = sample_row<LT, AL>(g, rowp, k, cP, P.idx, -1, ures, sh.p, sh);
            }
            o.accept_idx = -1;
            o.token = tok;
        }
    }
    if (threadIdx.x == 0) write_node(a, r, o);
}

// ------------------------------------------------------------------------------------------------
// Tree walk (Figure 2): one thread per sequence.
// ------------------------------------------------------------------------------------------------
struct WalkArgs {
    const int32_t *accept_idx, *token, *child;
    const uint8_t *node_kind;
    int32_t *n_accepted, *n_emitted, *path_nodes, *path_tokens;
    int batch, nodes, levels;
};

__global__ void walk_kernel(WalkArgs a) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= a.batch) return;
    int n = 0, acc = 0, emitted = 0, step = 0;
    for (; step < a.levels && n >= 0 && n < a.nodes; ++step) {
        const long long r = static_cast<long long>(b) * a.nodes + n;
        const int tok = a.token[r];
        if (a.path_nodes) a.path_nodes[static_cast<long long>(b) * a.levels + step] = n;
        if (a.path_tokens) a.path_tokens[static_cast<long long>(b) * a.levels + step] = tok;
        if (tok < 0) { ++step; break; }
        ++emitted;
        if (a.node_kind && a.node_kind[n] == SPECHUB_NODE_LEAF) { ++step; break; }
        const int idx = a.accept_idx[r];
        if (idx < 0 || idx > 1) { ++step; break; }   // (a caller-supplied index outside {0, 1} ends the walk)
        ++acc;
        n = a.child ? a.child[2 * n + idx] : 2 * n + 1 + idx;
    }
    for (; step < a.levels; ++step) {
        if (a.path_nodes) a.path_nodes[static_cast<long long>(b) * a.levels + step] = -1;
        if (a.path_tokens) a.path_tokens[static_cast<long long>(b) * a.levels + step] = -1;
    }
    if (a.n_accepted) a.n_accepted[b] = acc;
    if (a.n_emitted) a.n_emitted[b] = emitted;
}

}  // namespace spechub
