// RRS / RRSw (Algorithm 1, k = 2) with the vocabulary axis sharded over ranks: the phases of
// spechub_shard.cuh for the comparison methods.  Verification needs one exchange more than
// SpecHub's, because the second-stage residual mass W2 depends on the row-wide A1; the draft step
// without replacement needs a second round, because q without x1 is known only once x1 is.
//
//   sums (1st call) A1 = sum max(p - q, 0) over the slice; RRSw: sum of q outside x1; p, q at x1, x2
//   sums (2nd call) W2 = sum max(max(p - q, 0) - A1 q1, 0) over the slice
//   decide          Algorithm 1's two tests; residual token by the rank that holds the target
//   draft           x1 ~ q; x2 ~ q (RRS, same round) or ~ q without x1 (RRSw, second round)
#pragma once

#include "spechub_shard.cuh"

namespace spechub {

struct RrsRow {
    ShardStat P, Q;
    float invZp, invZq;
    int x1, x2;
    bool ok;
};
__device__ __forceinline__ RrsRow rrs_row(const ShardArgs &a, const ShardRow &w) {
    RrsRow s;
    s.P = shard_merge(a, w.r, 0, w.k);
    s.Q = shard_merge(a, w.r, 1, w.k);
    s.invZp = 1.f / (s.P.sx + s.P.own);
    s.invZq = 1.f / (s.Q.sx + s.Q.own);
    s.x1 = a.r.draft_tokens_in[2 * w.r];
    s.x2 = a.r.draft_tokens_in[2 * w.r + 1];
    s.ok = s.x1 >= 0 && s.x1 < a.vocab_total && s.x2 >= 0 && s.x2 < a.vocab_total;
    return s;
}
// A1, the renormaliser of q1 and A1 q1's coefficient from the gathered first-round sums
struct RrsStage {
    float A1, A1g;
    bool q1_zero;
};
__device__ __forceinline__ RrsStage rrs_stage(const ShardArgs &a, long long row) {
    float A1 = 0.f, den = 0.f;
    for (int c = 0; c < a.nranks; ++c) {
        const float *gs = a.gsums + ((long long)c * a.rows + row) * kShardRecord;
        A1 += gs[0];
        den += gs[1];
    }
    RrsStage st;
    st.A1 = A1;
    st.q1_zero = a.without_replacement && !(den > 0.f);
    const float gq = a.without_replacement ? (st.q1_zero ? 0.f : 1.f / den) : 1.f;
    st.A1g = A1 * gq;
    return st;
}

template <typename LT, bool AL>
__global__ void __launch_bounds__(512) rrs_shard_sums_kernel(ShardArgs a) {
    constexpr int VW = VecOf<LT>::W;
    __shared__ Partials sh;
    const ShardRow w = shard_row(a);
    const Geo g = make_geo(a.r.vocab, VW);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    float rec[kShardRecord] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    const bool leaf = a.r.node_kind && a.r.node_kind[w.n] == SPECHUB_NODE_LEAF;
    const RrsRow s = rrs_row(a, w);
    if (!leaf && !shard_bad(s.P) && !shard_bad(s.Q) && s.ok) {
        const LT *rowp = static_cast<const LT *>(a.r.target) + w.b * a.r.stride_seq + w.n * a.r.stride_node;
        const LT *rowq = static_cast<const LT *>(a.r.draft) + w.b * a.r.stride_seq + w.n * a.r.stride_node;
        const int x1loc = s.x1 - a.id_offset, x2loc = s.x2 - a.id_offset;
        if (!a.gsums) {
            float acc[2] = {0.f, 0.f};
            for (int vi = g.seg_lo(warp) + lane; vi < g.seg_hi(warp); vi += 32) {
                float vp[VW], vq[VW];
                load_vec<LT, AL>(rowp, vi, g.V, vp);
                load_vec<LT, AL>(rowq, vi, g.V, vq);
#pragma unroll
                for (int i = 0; i < VW; ++i) {
                    const float pp = prob_of(vp[i], w.k, s.P.C, s.invZp);
                    const float qq = prob_of(vq[i], w.k, s.Q.C, s.invZq);
                    acc[0] += fmaxf(__fsub_rn(pp, qq), 0.f);
                    if (a.without_replacement) acc[1] += (vi * VW + i == x1loc) ? 0.f : qq;
                }
            }
            block_sums<2>(g, acc, sh);
            rec[0] = acc[0]; rec[1] = acc[1];
            if (x1loc >= 0 && x1loc < a.r.vocab) {
                rec[3] = prob_of(load_one<LT>(rowp, x1loc), w.k, s.P.C, s.invZp);
                rec[4] = prob_of(load_one<LT>(rowq, x1loc), w.k, s.Q.C, s.invZq);
            }
            if (x2loc >= 0 && x2loc < a.r.vocab) {
                rec[5] = prob_of(load_one<LT>(rowp, x2loc), w.k, s.P.C, s.invZp);
                rec[6] = prob_of(load_one<LT>(rowq, x2loc), w.k, s.Q.C, s.invZq);
            }
        } else {
            const RrsStage st = rrs_stage(a, w.r);
            float w2[1] = {0.f};
            for (int vi = g.seg_lo(warp) + lane; vi < g.seg_hi(warp); vi += 32) {
                float vp[VW], vq[VW];
                load_vec<LT, AL>(rowp, vi, g.V, vp);
                load_vec<LT, AL>(rowq, vi, g.V, vq);
#pragma unroll
                for (int i = 0; i < VW; ++i) {
                    const float pp = prob_of(vp[i], w.k, s.P.C, s.invZp);
                    const float qq = prob_of(vq[i], w.k, s.Q.C, s.invZq);
                    float d, t;
                    transport_terms(pp, qq, (a.without_replacement && vi * VW + i == x1loc) ? 0.f : st.A1g, d, t);
                    w2[0] += fmaxf(t, 0.f);
                }
            }
            block_sums<1>(g, w2, sh);
            rec[0] = w2[0];
        }
    }
    if (threadIdx.x < kShardRecord) a.out[w.r * kShardRecord + threadIdx.x] = rec[threadIdx.x];
}

template <typename LT, bool AL>
__global__ void __launch_bounds__(512) rrs_shard_decide_kernel(ShardArgs a) {
    constexpr int VW = VecOf<LT>::W;
    __shared__ Partials sh;
    const ShardRow w = shard_row(a);
    const Geo g = make_geo(a.r.vocab, VW);
    const float r1 = a.r.uniforms[w.r * 5 + 2], r2 = a.r.uniforms[w.r * 5 + 3], ures = a.r.uniforms[w.r * 5 + 4];
    const bool leaf = a.r.node_kind && a.r.node_kind[w.n] == SPECHUB_NODE_LEAF;
    const LT *rowp = static_cast<const LT *>(a.r.target) + w.b * a.r.stride_seq + w.n * a.r.stride_node;
    const LT *rowq = static_cast<const LT *>(a.r.draft) + w.b * a.r.stride_seq + w.n * a.r.stride_node;

    NodeResult o;
    o.accept_idx = -1; o.token = -1; o.hub = -1; o.status = 0;
    o.beta[0] = o.beta[1] = 0.f; o.rate[0] = o.rate[1] = o.rate[2] = 0.f;

    const ShardStat P = shard_merge(a, w.r, 0, w.k);
    auto draw_from_p = [&]() {
        auto part = [&](int c) { return shard_mass(a, c, w.r, 0, w.k, P, -1); };
        auto wf = [&](int vi, float(&wt)[VW]) {
            float v[VW];
            load_vec<LT, AL>(rowp, vi, g.V, v);
#pragma unroll
            for (int i = 0; i < VW; ++i) wt[i] = ex2(fmaf(v[i], w.k, -P.C));
        };
        return shard_draw<VW>(a, g, part, wf, ures, sh);
    };
    do {
        if (shard_bad(P)) { o.status = SPECHUB_ST_NONFINITE; break; }
        if (leaf) {
            o.token = draw_from_p();
            o.rate[2] = 1.f;
            break;
        }
        const RrsRow s = rrs_row(a, w);
        if (shard_bad(s.Q)) { o.status = SPECHUB_ST_NONFINITE; break; }
        if (!s.ok) { o.status = SPECHUB_ST_TOKEN_RANGE; break; }
        const RrsStage st = rrs_stage(a, w.r);
        float sc[4] = {0.f, 0.f, 0.f, 0.f}, W2 = 0.f;   // p(x1), q(x1), p(x2), q(x2) from their owners
        for (int c = 0; c < a.nranks; ++c) {
            const float *gs = a.gsums + ((long long)c * a.rows + w.r) * kShardRecord;
#pragma unroll
            for (int i = 0; i < 4; ++i) sc[i] += gs[3 + i];
            W2 += a.gw2[((long long)c * a.rows + w.r) * kShardRecord];
        }
        const float A1 = st.A1;
        o.rate[0] = fmaxf(1.f - A1, 0.f);
        o.rate[1] = fmaxf(A1 - W2, 0.f);
        o.rate[2] = W2;
        const bool acc1 = accept_test(r1, sc[0], sc[1], o.beta[0], true, o.status);
        if (acc1) { o.accept_idx = 0; o.token = s.x1; }
        if (!acc1 && st.q1_zero) o.status |= SPECHUB_ST_DEGENERATE_Q;
        bool acc2 = false;
        if (A1 > 0.f) {
            const float q1x2 = (a.without_replacement && s.x2 == s.x1) ? 0.f : st.A1g * sc[3];
            acc2 = accept_test(r2, fmaxf(__fsub_rn(sc[2], sc[3]), 0.f), q1x2, o.beta[1], !acc1, o.status);
        }
        if (!acc1 && acc2) { o.accept_idx = 1; o.token = s.x2; }
        if (acc1 || acc2) break;
        o.accept_idx = -1;
        int tok = -1;
        if (A1 > 0.f) {
            const int x1loc = s.x1 - a.id_offset;
            auto part = [&](int c) { return a.gw2[((long long)c * a.rows + w.r) * kShardRecord]; };
            auto wf = [&](int vi, float(&wt)[VW]) {
                float vp[VW], vq[VW];
                load_vec<LT, AL>(rowp, vi, g.V, vp);
                load_vec<LT, AL>(rowq, vi, g.V, vq);
#pragma unroll
                for (int i = 0; i < VW; ++i) {
                    const float pp = prob_of(vp[i], w.k, s.P.C, s.invZp);
                    const float qq = prob_of(vq[i], w.k, s.Q.C, s.invZq);
                    float d, t;
                    transport_terms(pp, qq, (a.without_replacement && vi * VW + i == x1loc) ? 0.f : st.A1g, d, t);
                    wt[i] = fmaxf(t, 0.f);
                }
            };
            tok = shard_draw<VW>(a, g, part, wf, ures, sh);
        }
        if (tok == -1) {
            o.status |= SPECHUB_ST_ZERO_RESIDUAL;
            tok = draw_from_p();
        }
        o.token = tok;
    } while (false);
    if (threadIdx.x == 0) write_node(a.r, w.r, o);
}

// Draft calls.  First call (x1_known == NULL): x1 ~ q, RRS also x2 ~ q; x1's owner publishes the
// exponential of its logit.  Second call (RRSw): x2 ~ q with q(x1) set to 0.
template <typename LT, bool AL>
__global__ void __launch_bounds__(512) rrs_shard_draft_kernel(ShardArgs a) {
    constexpr int VW = VecOf<LT>::W;
    __shared__ Partials sh;
    const ShardRow w = shard_row(a);
    const Geo g = make_geo(a.r.vocab, VW);
    const float u1 = a.r.uniforms[w.r * 5 + 0], u2 = a.r.uniforms[w.r * 5 + 1];
    const LT *rowq = static_cast<const LT *>(a.r.draft) + w.b * a.r.stride_seq + w.n * a.r.stride_node;
    const ShardStat Q = shard_merge(a, w.r, 1, w.k);
    int c0 = -1, c1 = -1;
    float e1 = -1.f;
    if (!shard_bad(Q)) {
        auto wf_all = [&](int vi, float(&wt)[VW]) {
            float v[VW];
            load_vec<LT, AL>(rowq, vi, g.V, v);
#pragma unroll
            for (int i = 0; i < VW; ++i) wt[i] = ex2(fmaf(v[i], w.k, -Q.C));
        };
        auto mass_all = [&](int c) { return shard_mass(a, c, w.r, 1, w.k, Q, -1); };
        if (!a.x1_known) {
            c0 = shard_draw<VW>(a, g, mass_all, wf_all, u1, sh);
            if (c0 >= 0) e1 = ex2(fmaf(load_one<LT>(rowq, c0 - a.id_offset), w.k, -Q.C));
            if (!a.without_replacement) c1 = shard_draw<VW>(a, g, mass_all, wf_all, u2, sh);
        } else {
            const int x1 = a.x1_known[2 * w.r];
            const float ex1 = a.ex1_known[w.r];
            const int x1loc = x1 - a.id_offset;
            auto mass_wo = [&](int c) {   // slice c without x1: its published sum minus x1's term, unless x1 is its argmax
                float m = shard_mass(a, c, w.r, 1, w.k, Q, x1);
                const float *sr = a.gstats + ((long long)c * a.rows + w.r) * kShardRecord;
                const int off = __float_as_int(sr[3]), wid = __float_as_int(sr[7]);
                if (x1 >= off && x1 < off + wid && __float_as_int(sr[6]) != x1) m = fmaxf(m - ex1, 0.f);
                return m;
            };
            auto wf_wo = [&](int vi, float(&wt)[VW]) {
                float v[VW];
                load_vec<LT, AL>(rowq, vi, g.V, v);
#pragma unroll
                for (int i = 0; i < VW; ++i) wt[i] = (vi * VW + i == x1loc) ? 0.f : ex2(fmaf(v[i], w.k, -Q.C));
            };
            c1 = shard_draw<VW>(a, g, mass_wo, wf_wo, u2, sh);
        }
    }
    if (threadIdx.x == 0) {
        if (!a.x1_known) {
            a.cand_out[2 * w.r] = c0;
            a.cand_out[2 * w.r + 1] = c1;
            if (a.ex1_out) a.ex1_out[w.r] = e1;
        } else {
            a.cand_out[2 * w.r] = a.x1_known[2 * w.r];
            a.cand_out[2 * w.r + 1] = c1;
        }
    }
}

// One thread per row: (x1, x2) from the exchanged candidates.
__global__ void rrs_shard_draft_finish_kernel(ShardArgs a) {
    const long long r = blockIdx.x * (long long)blockDim.x + threadIdx.x;
    if (r >= a.rows) return;
    const int b = static_cast<int>(r / a.r.nodes);
    const float k = kLog2e / temperature_of(a.r, b);
    const ShardStat Q = shard_merge(a, r, 1, k);
    int x1 = -1, x2 = -1;
    uint32_t st = 0;
    if (shard_bad(Q)) {
        st = SPECHUB_ST_NONFINITE;
    } else {
        x1 = a.cand[2 * r];
        x2 = a.cand[2 * r + 1];
        if (a.without_replacement && x2 < 0) {   // nothing left to draw from: lowest id not drawn yet
            x2 = (x1 == 0) ? 1 : 0;
            st |= SPECHUB_ST_DEGENERATE_Q;
        }
    }
    a.r.draft_tokens_out[2 * r] = x1;
    a.r.draft_tokens_out[2 * r + 1] = x2;
    if (a.r.hub) a.r.hub[r] = -1;
    if (a.r.status) a.r.status[r] = st;
}

}  // namespace spechub
