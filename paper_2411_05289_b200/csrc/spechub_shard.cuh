// SpecHub with the vocabulary axis sharded over ranks (a tensor-parallel LM head): every rank
// holds the logits of a contiguous range of token ids, [id_offset, id_offset + local vocab), of
// every row.  The work is cut into phases at the points where a row-wide quantity is needed;
// between phases the caller exchanges a few floats per row (an all-gather of the phase output in
// rank order, or an element-wise maximum of candidate tokens).  Every rank then merges the
// gathered partials in rank order, so all ranks hold bit-identical row statistics and take
// identical decisions; only the rank whose slice holds an inverse-CDF target draws the token.
//
//   stats   per rank: (max, argmax, sum of exponentials without the argmax) of its slice of p, q
//   sums    S1, S2, R over its slice (Section 4, Appendix B.1) and p(x), q(x), p(a) if it owns them
//   decide  Algorithm 3's tests from the merged sums; residual / bonus token by the owning rank
//   draft   x1 ~ q and the candidate x2 ~ q without the hub, each by the owning rank
#pragma once

#include "spechub.h"
#include "spechub_common.cuh"
#include "spechub_stream.cuh"

namespace spechub {

constexpr int kShardRecord = 8;  // floats per row in a phase output

struct ShardArgs {
    RowArgs r;             // r.target / r.draft: this rank's slices; r.vocab: their width
    int rank, nranks, id_offset, vocab_total;
    long long rows;
    const float *gstats;   // [nranks][rows][8]: (ml, sx, idx) of p then of q, per rank
    const float *gsums;    // [nranks][rows][8]
    const float *gw2;      // [nranks][rows][8] (RRS / RRSw: second-stage residual masses)
    int without_replacement;
    const int32_t *x1_known;  // RRSw draft, second round: [rows][2] candidates after the maximum
    const float *ex1_known;   // ... and the exponential of x1's logit, [rows]
    float *ex1_out;           // first round: that exponential from x1's owner, -1 elsewhere
    const int32_t *cand;   // [rows][2] after the element-wise maximum over ranks
    float *out;            // [rows][8] phase output
    int32_t *cand_out;     // [rows][2]
};

struct ShardStat {
    float ml, C, sx;
    float own;   // the row argmax's own term 2^(k ml - C)
    int idx;
};

__device__ __forceinline__ ArgMaxSum shard_partial(const ShardArgs &a, int c, long long row, int which, float k) {
    const float *s = a.gstats + ((long long)c * a.rows + row) * kShardRecord + 4 * which;
    ArgMaxSum o;
    o.ml = s[0]; o.c = shift_of(o.ml, k); o.sx = s[1]; o.idx = __float_as_int(s[2]);
    return o;
}
// Row statistics from the ranks' partials, merged in rank order (a = argmax q, lowest id on ties).
__device__ __forceinline__ ShardStat shard_merge(const ShardArgs &a, long long row, int which, float k) {
    ArgMaxSum tot;
    tot.init();
    for (int c = 0; c < a.nranks; ++c) tot = argmaxsum_merge(tot, shard_partial(a, c, row, which, k), k);
    ShardStat st;
    st.ml = tot.ml; st.C = tot.c; st.sx = tot.sx; st.idx = tot.idx; st.own = tot.own(k);
    return st;
}
// Mass of rank c's slice in a draw from softmax(row) without token excl, on the row's scale.
__device__ __forceinline__ float shard_mass(const ShardArgs &a, int c, long long row, int which, float k,
                                            const ShardStat &st, int excl) {
    const ArgMaxSum o = shard_partial(a, c, row, which, k);
    const float own = (o.idx != excl) ? o.own(k) : 0.f;
    return (o.sx + own) * rescale(o.ml, o.c, st.C);
}

// Per-warp sums of weights(vi, w[]) over this CTA's warp ranges, to mass[] (shared memory).
template <int VW, class WF>
__device__ __forceinline__ void warp_masses(const Geo &g, WF weights, float *mass) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    float s = 0.f;
    for (int vi = g.seg_lo(warp) + lane; vi < g.seg_hi(warp); vi += 32) {
        float w[VW];
        weights(vi, w);
#pragma unroll
        for (int i = 0; i < VW; ++i) s += w[i];
    }
    s = warp_sum(s);
    if (lane == 0) mass[warp] = s;
    __syncthreads();
}

// Inverse-CDF draw over all ranks' slices: part(c) is rank c's mass.  Returns the global id when
// this rank's slice holds the target, -2 when another rank's does, -1 when there is no mass.
template <int VW, class PF, class WF>
__device__ int shard_draw(const ShardArgs &a, const Geo &g, PF part, WF weights, float u, Partials &sh) {
    float total = 0.f;
    for (int c = 0; c < a.nranks; ++c) total += part(c);
    if (!(total > 0.f)) return -1;
    const float t = u * total;
    int sel = -1, last = -1;
    float base = 0.f, lastbase = 0.f, run = 0.f;
    for (int c = 0; c < a.nranks; ++c) {
        const float m = part(c);
        if (m > 0.f) {
            last = c;
            lastbase = run;
            if (sel < 0 && run + m > t) { sel = c; base = run; }
        }
        run += m;
    }
    if (sel < 0) { sel = last; base = lastbase; }
    if (sel != a.rank) return -2;
    warp_masses<VW>(g, weights, sh.mass);
    const int tok = block_sample_at<VW>(g, weights, sh.mass, t - base, &sh.tok);
    return tok < 0 ? -2 : tok + a.id_offset;
}

struct ShardRow {
    long long r;
    int b, n;
    float k;
};
__device__ __forceinline__ ShardRow shard_row(const ShardArgs &a) {
    ShardRow w;
    w.r = blockIdx.x;
    w.b = static_cast<int>(w.r / a.r.nodes);
    w.n = static_cast<int>(w.r % a.r.nodes);
    w.k = kLog2e / temperature_of(a.r, w.b);
    return w;
}
__device__ __forceinline__ bool shard_bad(const ShardStat &s) {
    return !(s.ml > neg_inf()) || !(s.ml < -neg_inf()) || !finite_pos(s.sx + s.own);
}

// ---- phase "stats" ------------------------------------------------------------------------------
template <typename LT, bool AL>
__global__ void __launch_bounds__(512) shard_stats_kernel(ShardArgs a) {
    constexpr int VW = VecOf<LT>::W;
    __shared__ Partials sh;
    const ShardRow w = shard_row(a);
    const Geo g = make_geo(a.r.vocab, VW);
    float rec[kShardRecord] = {neg_inf(), 0.f, __int_as_float(0x7fffffff), 0.f, neg_inf(), 0.f, __int_as_float(0x7fffffff), 0.f};
    if (a.r.target) {
        const LT *rowp = static_cast<const LT *>(a.r.target) + w.b * a.r.stride_seq + w.n * a.r.stride_node;
        const ArgMaxSum P = pass_a<LT, AL>(g, rowp, w.k, sh.p);
        rec[0] = P.ml; rec[1] = P.sx;
        rec[2] = __int_as_float(P.ml > neg_inf() ? P.idx + a.id_offset : 0x7fffffff);
    }
    // verification reads no q on a leaf row; the draft step (no target given) drafts on every row
    const bool leaf = a.r.target && a.r.node_kind && a.r.node_kind[w.n] == SPECHUB_NODE_LEAF;
    if (a.r.draft && !leaf) {
        const LT *rowq = static_cast<const LT *>(a.r.draft) + w.b * a.r.stride_seq + w.n * a.r.stride_node;
        const ArgMaxSum Q = pass_a<LT, AL>(g, rowq, w.k, sh.q);
        rec[4] = Q.ml; rec[5] = Q.sx;
        rec[6] = __int_as_float(Q.ml > neg_inf() ? Q.idx + a.id_offset : 0x7fffffff);
    }
    // spare lanes: this slice's id range, so that every rank can tell which slice holds a given token
    rec[3] = __int_as_float(a.id_offset);
    rec[7] = __int_as_float(a.r.vocab);
    if (threadIdx.x < kShardRecord) a.out[w.r * kShardRecord + threadIdx.x] = rec[threadIdx.x];
}

// What the sums and decide phases share about one verified row.
struct ShardPair {
    ShardStat P, Q;
    float invZp, invZq, c;
    int hub, x;          // global ids; x = the pair's non-hub token
    bool pair_xa, ok, degenerate;
};
__device__ __forceinline__ ShardPair shard_pair(const ShardArgs &a, const ShardRow &w) {
    ShardPair s;
    s.P = shard_merge(a, w.r, 0, w.k);
    s.Q = shard_merge(a, w.r, 1, w.k);
    s.invZp = 1.f / (s.P.sx + s.P.own);
    s.invZq = 1.f / (s.Q.sx + s.Q.own);
    s.hub = s.Q.idx;
    s.degenerate = !(s.Q.sx > 0.f);
    s.c = s.degenerate ? 0.f : s.Q.own / s.Q.sx;
    const int x1 = a.r.draft_tokens_in[2 * w.r], x2 = a.r.draft_tokens_in[2 * w.r + 1];
    s.pair_xa = (x2 == s.hub && x1 != s.hub);
    const bool pair_ax = (x1 == s.hub && x2 != s.hub);
    s.x = s.pair_xa ? x1 : x2;
    s.ok = (s.pair_xa || pair_ax) && s.x >= 0 && s.x < a.vocab_total;
    return s;
}

// ---- phase "sums" -------------------------------------------------------------------------------
template <typename LT, bool AL>
__global__ void __launch_bounds__(512) shard_sums_kernel(ShardArgs a) {
    constexpr int VW = VecOf<LT>::W;
    __shared__ Partials sh;
    const ShardRow w = shard_row(a);
    const Geo g = make_geo(a.r.vocab, VW);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    float rec[kShardRecord] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    const bool leaf = a.r.node_kind && a.r.node_kind[w.n] == SPECHUB_NODE_LEAF;
    const ShardPair s = shard_pair(a, w);
    if (!leaf && !shard_bad(s.P) && !shard_bad(s.Q) && s.ok) {
        const LT *rowp = static_cast<const LT *>(a.r.target) + w.b * a.r.stride_seq + w.n * a.r.stride_node;
        const LT *rowq = static_cast<const LT *>(a.r.draft) + w.b * a.r.stride_seq + w.n * a.r.stride_node;
        const int hubloc = s.hub - a.id_offset;  // outside [0, vocab) when another rank owns the hub
        float acc[3] = {0.f, 0.f, 0.f};
        for (int vi = g.seg_lo(warp) + lane; vi < g.seg_hi(warp); vi += 32) {
            float vp[VW], vq[VW];
            load_vec<LT, AL>(rowp, vi, g.V, vp);
            load_vec<LT, AL>(rowq, vi, g.V, vq);
#pragma unroll
            for (int i = 0; i < VW; ++i) {
                const bool is_hub = (vi * VW + i == hubloc);
                const float pp = is_hub ? 0.f : prob_of(vp[i], w.k, s.P.C, s.invZp);
                const float qq = is_hub ? 0.f : prob_of(vq[i], w.k, s.Q.C, s.invZq);
                float d, t;
                transport_terms(pp, qq, s.c, d, t);
                acc[0] += fmaxf(-d, 0.f);
                acc[1] += fmaxf(-t, 0.f);
                acc[2] += fmaxf(t, 0.f);
            }
        }
        block_sums<3>(g, acc, sh);
        rec[0] = acc[0]; rec[1] = acc[1]; rec[2] = acc[2];
        const int xloc = s.x - a.id_offset;
        if (xloc >= 0 && xloc < a.r.vocab) {
            rec[3] = prob_of(load_one<LT>(rowp, xloc), w.k, s.P.C, s.invZp);
            rec[4] = prob_of(load_one<LT>(rowq, xloc), w.k, s.Q.C, s.invZq);
        }
        if (hubloc >= 0 && hubloc < a.r.vocab) rec[5] = prob_of(load_one<LT>(rowp, hubloc), w.k, s.P.C, s.invZp);
    }
    if (threadIdx.x < kShardRecord) a.out[w.r * kShardRecord + threadIdx.x] = rec[threadIdx.x];
}

// ---- phase "decide" -----------------------------------------------------------------------------
template <typename LT, bool AL>
__global__ void __launch_bounds__(512) shard_decide_kernel(ShardArgs a) {
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
    // bonus token or fallback: a draw from p over all ranks
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
        const ShardPair s = shard_pair(a, w);
        if (shard_bad(s.Q)) { o.status = SPECHUB_ST_NONFINITE; break; }
        o.hub = s.hub;
        if (!s.ok) { o.status = SPECHUB_ST_TOKEN_RANGE; break; }
        float tot[6] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        for (int c = 0; c < a.nranks; ++c) {
            const float *gs = a.gsums + ((long long)c * a.rows + w.r) * kShardRecord;
#pragma unroll
            for (int i = 0; i < 6; ++i) tot[i] += gs[i];
        }
        const float qa = s.Q.own * s.invZq, rest = s.Q.sx * s.invZq;
        const float S1 = tot[0], S2 = s.degenerate ? qa : tot[1], R = tot[2];
        const float px = tot[3], qx = tot[4], pa = tot[5];
        const float hub_left = fmaxf(pa - S2, 0.f);
        o.rate[0] = fmaxf(rest - S1, 0.f) + fminf(pa, S2);
        o.rate[1] = (s.degenerate ? 0.f : fmaxf(qa - S2, 0.f)) + fminf(hub_left, S1);
        o.rate[2] = R;
        if (s.degenerate) o.status |= SPECHUB_ST_DEGENERATE_Q;
        bool acc1, acc2;
        if (s.pair_xa) {
            acc1 = accept_test(r1, px, qx, o.beta[0], true, o.status);
            if (acc1) { o.accept_idx = 0; o.token = s.x; }
            acc2 = accept_test(r2, hub_left, S1, o.beta[1], !acc1, o.status);
            if (!acc1 && acc2) { o.accept_idx = 1; o.token = s.hub; }
        } else {
            acc1 = accept_test(r1, fmaxf(__fsub_rn(px, qx), 0.f), s.c * qx, o.beta[0], true, o.status);
            if (acc1) { o.accept_idx = 1; o.token = s.x; }
            acc2 = accept_test(r2, pa, S2, o.beta[1], !acc1, o.status);
            if (!acc1 && acc2) { o.accept_idx = 0; o.token = s.hub; }
        }
        if (acc1 || acc2) break;
        o.accept_idx = -1;
        const int hubloc = s.hub - a.id_offset;
        auto part = [&](int c) { return a.gsums[((long long)c * a.rows + w.r) * kShardRecord + 2]; };
        auto wf = [&](int vi, float(&wt)[VW]) {   // the residual of Section 4, zero on the hub
            float vp[VW], vq[VW];
            load_vec<LT, AL>(rowp, vi, g.V, vp);
            load_vec<LT, AL>(rowq, vi, g.V, vq);
#pragma unroll
            for (int i = 0; i < VW; ++i) {
                const bool is_hub = (vi * VW + i == hubloc);
                const float pp = is_hub ? 0.f : prob_of(vp[i], w.k, s.P.C, s.invZp);
                const float qq = is_hub ? 0.f : prob_of(vq[i], w.k, s.Q.C, s.invZq);
                float d, t;
                transport_terms(pp, qq, s.c, d, t);
                wt[i] = fmaxf(t, 0.f);
            }
        };
        int tok = shard_draw<VW>(a, g, part, wf, ures, sh);
        if (tok == -1) {
            o.status |= SPECHUB_ST_ZERO_RESIDUAL;
            tok = draw_from_p();
        }
        o.token = tok;
    } while (false);
    if (threadIdx.x == 0) write_node(a.r, w.r, o);
}

// ---- phase "draft" ------------------------------------------------------------------------------
template <typename LT, bool AL>
__global__ void __launch_bounds__(512) shard_draft_kernel(ShardArgs a) {
    constexpr int VW = VecOf<LT>::W;
    __shared__ Partials sh;
    const ShardRow w = shard_row(a);
    const Geo g = make_geo(a.r.vocab, VW);
    const float u1 = a.r.uniforms[w.r * 5 + 0], u2 = a.r.uniforms[w.r * 5 + 1];
    const LT *rowq = static_cast<const LT *>(a.r.draft) + w.b * a.r.stride_seq + w.n * a.r.stride_node;
    const ShardStat Q = shard_merge(a, w.r, 1, w.k);
    int c0 = -1, c1 = -1;
    if (!shard_bad(Q)) {
        const int hub = Q.idx, hubloc = Q.idx - a.id_offset;
        auto wf_all = [&](int vi, float(&wt)[VW]) {
            float v[VW];
            load_vec<LT, AL>(rowq, vi, g.V, v);
#pragma unroll
            for (int i = 0; i < VW; ++i) wt[i] = ex2(fmaf(v[i], w.k, -Q.C));
        };
        auto wf_nohub = [&](int vi, float(&wt)[VW]) {
            float v[VW];
            load_vec<LT, AL>(rowq, vi, g.V, v);
#pragma unroll
            for (int i = 0; i < VW; ++i) wt[i] = (vi * VW + i == hubloc) ? 0.f : ex2(fmaf(v[i], w.k, -Q.C));
        };
        // x1 ~ q; the second draw of the pair (a, x), x ~ q without the hub, is made in any case:
        // whether it is used depends on x1, which only its owner knows before the exchange
        c0 = shard_draw<VW>(a, g, [&](int c) { return shard_mass(a, c, w.r, 1, w.k, Q, -1); }, wf_all, u1, sh);
        if (Q.sx > 0.f)
            c1 = shard_draw<VW>(a, g, [&](int c) { return shard_mass(a, c, w.r, 1, w.k, Q, hub); }, wf_nohub, u2, sh);
    }
    if (threadIdx.x == 0) { a.cand_out[2 * w.r] = c0; a.cand_out[2 * w.r + 1] = c1; }
}

// One thread per row: the pair from the exchanged candidates (Section 4: (x, a) if x1 != a, else
// (a, x) with x ~ q without a).
__global__ void shard_draft_finish_kernel(ShardArgs a) {
    const long long r = blockIdx.x * (long long)blockDim.x + threadIdx.x;
    if (r >= a.rows) return;
    const int b = static_cast<int>(r / a.r.nodes);
    const float k = kLog2e / temperature_of(a.r, b);
    const ShardStat Q = shard_merge(a, r, 1, k);
    int x1 = -1, x2 = -1, hub = -1;
    uint32_t st = 0;
    if (shard_bad(Q)) {
        st = SPECHUB_ST_NONFINITE;
    } else {
        hub = Q.idx;
        x1 = a.cand[2 * r];
        if (x1 != hub) {
            x2 = hub;
        } else if (!(Q.sx > 0.f)) {
            x2 = (hub == 0) ? 1 : 0;
            st |= SPECHUB_ST_DEGENERATE_Q;
        } else {
            x2 = a.cand[2 * r + 1];
        }
    }
    a.r.draft_tokens_out[2 * r] = x1;
    a.r.draft_tokens_out[2 * r + 1] = x2;
    if (a.r.hub) a.r.hub[r] = hub;
    if (a.r.status) a.r.status[r] = st;
}

}  // namespace spechub
