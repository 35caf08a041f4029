// Recursive Rejection Sampling with k > 2 drafts per node (Algorithm 1 of arXiv 2411.05289 is
// stated for k candidates; the paper's ternary trees and its acceptance-decay experiment use
// them).  One CTA per (sequence, node) row, any vocabulary size, fp32 or bf16 logits, built
// from the same pieces as the general two-draft kernels.
//
// Unnormalised form of Algorithm 1.  With P_0 = p, m_0 = 1 and, for stage j = 1..k,
//   q_j = q                                   (RRS)
//   q_j = q with q(x_1..x_{j-1}) zeroed / den_j, den_j = sum of q outside x_1..x_{j-1}   (RRSw)
//   test j:  accept x_j  iff  r_j * m_{j-1} q_j(x_j) < P_{j-1}(x_j)
//   P_j = max(P_{j-1} - m_{j-1} q_j, 0),   m_j = sum_y P_j(y)
// the token after k rejections is drawn from P_k.  m_j needs m_{j-1}, so stage j is one more
// pass over the row (which hits L2): 1 + k passes in all.
#pragma once

#include "spechub.h"
#include "spechub_common.cuh"
#include "spechub_stream.cuh"

namespace spechub {

constexpr int kMaxK = SPECHUB_MAX_K;

struct KaryArgs {
    RowArgs r;
    int k;
    int without_replacement;
};

// Is token y one of x[0..n)?
__device__ __forceinline__ bool in_set(const int *x, int n, int y) {
    bool f = false;
    for (int i = 0; i < n; ++i) f |= (x[i] == y);
    return f;
}

// P_j(y) from p(y), q(y): j subtractions with the stage coefficients; for RRSw a token already
// drawn before stage l carries no draft mass there.
__device__ __forceinline__ float stage_value(float pp, float qq, int y, int j, const float *coef, const int *x,
                                             bool wo, bool check_set) {
    float v = pp;
    for (int l = 0; l < j; ++l) {
        const float ql = (wo && check_set && in_set(x, l, y)) ? 0.f : qq;
        v = fmaxf(__fmaf_rn(-coef[l], ql, v), 0.f);
    }
    return v;
}

// Draw from softmax(row) without the tokens excl[0..nex).  Per-warp partials of pass_a in wp.
template <typename LT, bool AL>
__device__ int sample_row_multi(const Geo &g, const LT *row, float k, float cQ, int hubtok, const int *excl,
                                int nex, float u, const WarpPart &wp, Partials &sh) {
    constexpr int VW = VecOf<LT>::W;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const bool hub_out = in_set(excl, nex, hubtok);
    if (threadIdx.x < g.nwarps) {
        const int w = threadIdx.x;
        const float ml = wp.ml[w];
        const bool holds_hub = (wp.idx[w] == hubtok);
        const float own = (holds_hub && hub_out) ? 0.f : own_term(ml, k);
        sh.mass[w] = (wp.sx[w] + own) * rescale(ml, shift_of(ml, k), cQ);
    }
    __syncthreads();
    // a warp whose range holds a removed token (other than the row argmax) re-sums its range
    bool mine = false;
    for (int i = 0; i < nex; ++i)
        if (excl[i] != hubtok && excl[i] >= 0 && excl[i] < g.V) mine |= (g.warp_of_vec(excl[i] / VW) == warp);
    if (mine) {
        float s = 0.f;
        for (int vi = g.seg_lo(warp) + lane; vi < g.seg_hi(warp); vi += 32) {
            float v[VW];
            load_vec<LT, AL>(row, vi, g.V, v);
#pragma unroll
            for (int i = 0; i < VW; ++i) s += in_set(excl, nex, vi * VW + i) ? 0.f : ex2(fmaf(v[i], k, -cQ));
        }
        s = warp_sum(s);
        if (lane == 0) sh.mass[warp] = s;
    }
    __syncthreads();
    auto wf = [&](int vi, float(&w)[VW]) {
        float v[VW];
        load_vec<LT, AL>(row, vi, g.V, v);
#pragma unroll
        for (int i = 0; i < VW; ++i) w[i] = in_set(excl, nex, vi * VW + i) ? 0.f : ex2(fmaf(v[i], k, -cQ));
    };
    return block_sample<VW>(g, wf, sh.mass, u, &sh.tok);
}

// ---- draft step -----------------------------------------------------------------------------------
template <typename LT, bool AL>
__global__ void __launch_bounds__(512) kary_draft_kernel(KaryArgs A) {
    constexpr int VW = VecOf<LT>::W;
    __shared__ Partials sh;
    const RowArgs &a = A.r;
    const int K = A.k;
    const long long r = blockIdx.x;
    const int b = static_cast<int>(r / a.nodes), n = static_cast<int>(r % a.nodes);
    const LT *rowq = static_cast<const LT *>(a.draft) + b * a.stride_seq + n * a.stride_node;
    const Geo g = make_geo(a.vocab, VW);
    const float k = kLog2e / temperature_of(a, b);
    const float *un = a.uniforms + r * (2 * K + 1);

    const ArgMaxSum q = pass_a<LT, AL>(g, rowq, k, sh.q);
    const float Zq = q.sx + q.own(k);
    uint32_t st = 0;
    int x[kMaxK];
    for (int i = 0; i < K; ++i) x[i] = -1;
    if (!(q.ml > neg_inf()) || !finite_pos(Zq) || !(q.ml < -neg_inf())) {
        st = SPECHUB_ST_NONFINITE;
    } else {
        for (int i = 0; i < K; ++i) {
            const int nex = A.without_replacement ? i : 0;
            int t = sample_row_multi<LT, AL>(g, rowq, k, q.c, q.idx, x, nex, un[i], sh.q, sh);
            if (t < 0) {  // nothing left to draw from: lowest id not drawn yet
                st |= SPECHUB_ST_DEGENERATE_Q;
                for (t = 0; t < a.vocab && in_set(x, i, t); ++t) {}
                if (t >= a.vocab) t = 0;
            }
            x[i] = t;
        }
    }
    if (threadIdx.x == 0) {
        void_draft_stat(a, r);
        for (int i = 0; i < K; ++i) a.draft_tokens_out[K * r + i] = x[i];
        if (a.status) a.status[r] = st;
    }
}

// ---- verification ---------------------------------------------------------------------------------
template <typename LT, bool AL>
__global__ void __launch_bounds__(512) kary_verify_kernel(KaryArgs A) {
    constexpr int VW = VecOf<LT>::W;
    __shared__ Partials sh;
    const RowArgs &a = A.r;
    const int K = A.k;
    const bool wo = A.without_replacement != 0;
    const long long r = blockIdx.x;
    const int b = static_cast<int>(r / a.nodes), n = static_cast<int>(r % a.nodes);
    const LT *rowp = static_cast<const LT *>(a.target) + b * a.stride_seq + n * a.stride_node;
    const LT *rowq = static_cast<const LT *>(a.draft) + b * a.stride_seq + n * a.stride_node;
    const Geo g = make_geo(a.vocab, VW);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const float k = kLog2e / temperature_of(a, b);
    const float *un = a.uniforms + r * (2 * K + 1);
    const float ures = un[2 * K];
    const float pinf = -neg_inf();

    int accept_idx = -1, token = -1;
    uint32_t status = 0;
    float beta[kMaxK], rate[kMaxK + 1];
    for (int i = 0; i < K; ++i) beta[i] = 0.f;
    for (int i = 0; i <= K; ++i) rate[i] = 0.f;
    auto write_out = [&]() {
        if (threadIdx.x != 0) return;
        a.accept_idx[r] = accept_idx;
        a.token[r] = token;
        if (a.hub) a.hub[r] = -1;
        if (a.beta) for (int i = 0; i < K; ++i) a.beta[K * r + i] = beta[i];
        if (a.rate) for (int i = 0; i <= K; ++i) a.rate[(K + 1) * r + i] = rate[i];
        if (a.status) a.status[r] = status;
    };

    const ArgMaxSum P = pass_a<LT, AL>(g, rowp, k, sh.p);
    const float Zp = P.sx + P.own(k);
    if (!(P.ml > neg_inf()) || !(P.ml < pinf) || !finite_pos(Zp)) { status = SPECHUB_ST_NONFINITE; write_out(); return; }
    const float cP = P.c, invZp = 1.f / Zp;
    if (a.node_kind && a.node_kind[n] == SPECHUB_NODE_LEAF) {
        token = sample_row<LT, AL>(g, rowp, k, cP, P.idx, -1, ures, sh.p, sh);
        rate[K] = 1.f;
        write_out();
        return;
    }
    const ArgMaxSum Q = pass_a<LT, AL>(g, rowq, k, sh.q);
    const float Zq = Q.sx + Q.own(k);
    if (!(Q.ml > neg_inf()) || !(Q.ml < pinf) || !finite_pos(Zq)) { status = SPECHUB_ST_NONFINITE; write_out(); return; }
    const float cQ = Q.c, invZq = 1.f / Zq;
    int x[kMaxK];
    bool bad = false;
    for (int i = 0; i < K; ++i) { x[i] = a.draft_tokens_in[K * r + i]; bad |= (x[i] < 0 || x[i] >= a.vocab); }
    if (bad) { status = SPECHUB_ST_TOKEN_RANGE; write_out(); return; }
    float px[kMaxK], qx[kMaxK];
    for (int i = 0; i < K; ++i) {
        px[i] = prob_of(load_one<LT>(rowp, x[i]), k, cP, invZp);
        qx[i] = prob_of(load_one<LT>(rowq, x[i]), k, cQ, invZq);
    }

    // vectors that hold a draft token take the slow path with the membership test (RRSw)
    auto vec_has_token = [&](int vi) {
        bool f = false;
        for (int i = 0; i < K; ++i) f |= (x[i] / VW == vi);
        return f;
    };

    float coef[kMaxK];   // coef[l] = m_l * g_{l+1}: what stage l+1 subtracts per unit of q
    float m[kMaxK + 1];  // m[j] = mass of P_j
    float den[kMaxK];    // den[l] = sum of q outside x[0..l)   (RRSw; 1 for RRS)
    m[0] = 1.f;
    for (int l = 0; l < K; ++l) den[l] = 1.f;
    for (int j = 1; j <= K; ++j) {
        // stage coefficient from what is known so far
        const float gj = wo ? (den[j - 1] > 0.f ? 1.f / den[j - 1] : 0.f) : 1.f;
        coef[j - 1] = m[j - 1] * gj;
        // pass j: m_j = sum_y P_j(y); the first pass of RRSw also sums q outside all drafts but the last
        float acc[2] = {0.f, 0.f};
        for (int vi = g.seg_lo(warp) + lane; vi < g.seg_hi(warp); vi += 32) {
            float vp[VW], vq[VW];
            load_vec<LT, AL>(rowp, vi, g.V, vp);
            load_vec<LT, AL>(rowq, vi, g.V, vq);
            const bool slow = wo && vec_has_token(vi);
#pragma unroll
            for (int i = 0; i < VW; ++i) {
                const float pp = prob_of(vp[i], k, cP, invZp), qq = prob_of(vq[i], k, cQ, invZq);
                acc[0] += stage_value(pp, qq, vi * VW + i, j, coef, x, wo, slow);
                if (wo && j == 1) acc[1] += (slow && in_set(x, K - 1, vi * VW + i)) ? 0.f : qq;
            }
        }
        block_sums<2>(g, acc, sh);
        release_sums();
        m[j] = acc[0];
        if (wo && j == 1) {
            // den[l] = (q outside x[0..K-1)) + q of the distinct tokens among x[l..K-1) not in x[0..l)
            for (int l = 1; l < K; ++l) {  // den[0] = 1: nothing removed yet
                float d = acc[1];
                for (int t = l; t < K - 1; ++t)
                    if (!in_set(x, l, x[t]) && !in_set(x + l, t - l, x[t])) d += qx[t];
                den[l] = d;
            }
        }
    }
    // per-warp masses of P_K for the residual draw are in sh.acc[0] (last pass) -- copy before reuse
    if (threadIdx.x < g.nwarps) sh.mass[threadIdx.x] = sh.acc[0][threadIdx.x];
    __syncthreads();

    // decisions
    bool accepted = false;
    for (int i = 0; i < K; ++i) {
        const bool alive = m[i] > 0.f;
        rate[i] = alive ? fmaxf(m[i] - m[i + 1], 0.f) : 0.f;
        const float gi = wo ? (den[i] > 0.f ? 1.f / den[i] : 0.f) : 1.f;
        const bool gone = wo && in_set(x, i, x[i]);
        const float D = gone ? 0.f : m[i] * gi * qx[i];
        const float N = stage_value(px[i], qx[i], x[i], i, coef, x, wo, true);
        beta[i] = (alive && D > 0.f) ? fminf(N / D, 1.f) : 0.f;
        if (alive && !accepted) {
            if (wo && i > 0 && !(den[i] > 0.f)) status |= SPECHUB_ST_DEGENERATE_Q;
            if (!(D > 0.f)) status |= SPECHUB_ST_ZERO_MASS_DRAFT;
            else if (un[K + i] * D < N) { accepted = true; accept_idx = i; token = x[i]; }
        }
    }
    rate[K] = m[K];
    if (!accepted) {
        int tok = -1;
        if (m[K] > 0.f) {
            auto wf = [&](int vi, float(&w)[VW]) {
                float vp[VW], vq[VW];
                load_vec<LT, AL>(rowp, vi, g.V, vp);
                load_vec<LT, AL>(rowq, vi, g.V, vq);
                const bool slow = wo && vec_has_token(vi);
#pragma unroll
                for (int i = 0; i < VW; ++i)
                    w[i] = stage_value(prob_of(vp[i], k, cP, invZp), prob_of(vq[i], k, cQ, invZq), vi * VW + i, K,
                                       coef, x, wo, slow);
            };
            tok = block_sample<VW>(g, wf, sh.mass, ures, &sh.tok);
        }
        if (tok < 0) {
            status |= SPECHUB_ST_ZERO_RESIDUAL;
            tok = sample_row<LT, AL>(g, rowp, k, cP, P.idx, -1, ures, sh.p, sh);
        }
        token = tok;
    }
    write_out();
}

// ---- tree walk with k children per node -------------------------------------------------------------
struct WalkKArgs {
    WalkArgs w;
    int k;
};
__global__ void walk_k_kernel(WalkKArgs A) {
    const WalkArgs &a = A.w;
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
        if (idx < 0 || idx >= A.k) { ++step; break; }
        ++acc;
        n = a.child ? a.child[A.k * n + idx] : A.k * n + 1 + idx;
    }
    for (; step < a.levels; ++step) {
        if (a.path_nodes) a.path_nodes[static_cast<long long>(b) * a.levels + step] = -1;
        if (a.path_tokens) a.path_tokens[static_cast<long long>(b) * a.levels + step] = -1;
    }
    if (a.n_accepted) a.n_accepted[b] = acc;
    if (a.n_emitted) a.n_emitted[b] = emitted;
}

}  // namespace spechub
