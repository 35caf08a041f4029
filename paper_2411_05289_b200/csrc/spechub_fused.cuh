// SpecHub, RRS and RRSw on the same rows in one kernel (large-vocabulary bf16 shapes).
//
// The three methods read the same p and q.  Pass A (max, sum of exponentials, hub) is common to
// them; one pass B forms p(y), q(y) once and feeds SpecHub's transport sums, RRS's A1 and RRSw's
// renormaliser; one pass C gives the two second-stage residual masses.  Three passes over a row
// pair instead of 2 + 3 + 3, 6 ex2 per vocabulary pair instead of 16.  Every sum is accumulated
// exactly as in lean_verify_kernel / lean_draft_kernel, so the results are bit-identical to the
// separate calls.
#pragma once

#include "spechub.h"
#include "spechub_common.cuh"
#include "spechub_stream.cuh"
#include "spechub_lean.cuh"

namespace spechub {

struct FusedArgs {
    RowArgs r;                 // target, draft, uniforms, temperature, node_kind, shape
    const int32_t *tok[3];     // draft tokens of SpecHub, RRS, RRSw (verify)
    int32_t *tok_out[3];       // (draft)
    NodeOutPtrs out[3];
    uint32_t *dstatus[3];      // draft status
};

__device__ __forceinline__ void write_node3(const NodeOutPtrs &p, long long r, const NodeResult &o, bool tok_elsewhere) {
    p.accept_idx[r] = o.accept_idx;
    if (!tok_elsewhere) p.token[r] = o.token;
    if (p.hub) p.hub[r] = o.hub;
    if (p.beta) { p.beta[2 * r] = o.beta[0]; p.beta[2 * r + 1] = o.beta[1]; }
    if (p.rate) { p.rate[3 * r] = o.rate[0]; p.rate[3 * r + 1] = o.rate[1]; p.rate[3 * r + 2] = o.rate[2]; }
    if (p.status) p.status[r] = o.status;
}

// STATS: as in lean_verify_kernel -- the draft row's maximum, argmax and sum come from the record the draft
// step left, pass A reads the target row only, and a row pair that turns out to be one row twice is redone
// with p's normaliser set to q's.
template <int THREADS, bool STATS = false>
__global__ void __launch_bounds__(THREADS, 1024 / THREADS) fused_verify_kernel(FusedArgs A) {
    __shared__ LeanShared sh;
    const RowArgs &a = A.r;
    const long long r = blockIdx.x;
    const int b = static_cast<int>(r / a.nodes), n = static_cast<int>(r % a.nodes);
    const __nv_bfloat16 *rowp = static_cast<const __nv_bfloat16 *>(a.target) + b * a.stride_seq + n * a.stride_node;
    const __nv_bfloat16 *rowq = static_cast<const __nv_bfloat16 *>(a.draft) + b * a.stride_seq + n * a.stride_node;
    const uint4 *vp = reinterpret_cast<const uint4 *>(rowp), *vq = reinterpret_cast<const uint4 *>(rowq);
    const Geo g = make_geo(a.vocab, 8);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int lo = g.seg_lo(warp), hi = g.seg_hi(warp);
    const int last_vi = (lo + lane < hi) ? lo + lane + ((hi - 1 - lo - lane) / 32) * 32 : lo - 1;
    const float k = kLog2e / temperature_of(a, b);
    const float r1 = a.uniforms[r * 5 + 2], r2 = a.uniforms[r * 5 + 3], ures = a.uniforms[r * 5 + 4];
    const float pinf = -neg_inf();
    const bool leaf = a.node_kind && a.node_kind[n] == SPECHUB_NODE_LEAF;
    const bool t0 = threadIdx.x == 0;

    NodeResult o[3];
    bool elsewhere[3] = {false, false, false};
#pragma unroll
    for (int m = 0; m < 3; ++m) {
        o[m].accept_idx = -1; o[m].token = -1; o[m].hub = -1; o[m].status = 0;
        o[m].beta[0] = o[m].beta[1] = 0.f; o[m].rate[0] = o[m].rate[1] = o[m].rate[2] = 0.f;
    }
    auto finish = [&]() {
        if (!t0) return;
#pragma unroll
        for (int m = 0; m < 3; ++m) write_node3(A.out[m], r, o[m], elsewhere[m]);
    };

    if (leaf) return;   // leaf rows belong to lean_leaf_kernel
    LeanAcc tp, tq;
    if (STATS) lean_pass_a_deep(vp, lo, hi, lane, k, tp);
    else lean_pass_a<true>(vp, vq, lo, hi, lane, k, tp, tq);
    {
        ArgMaxSum Ps, Qs;
        if (STATS) lean_reduce2<false>(tp, tq, vp, vq, lo, hi, k, sh, Ps, Qs);
        else lean_reduce2<true>(tp, tq, vp, vq, lo, hi, k, sh, Ps, Qs);
        if (t0) {
            sh.x_ml[0] = Ps.ml; sh.x_sx[0] = Ps.sx; sh.x_idx[0] = Ps.idx;
            if (STATS) {
                const DraftStat ds = static_cast<const DraftStat *>(a.draft_stats_in)[r];
                bool ok = ds.tag == (kDraftStatTag ^ __float_as_uint(k));
                if (ok && ds.ml > neg_inf() && ds.ml < pinf && finite_pos(ds.sx + 1.f))
                    ok = ds.idx >= 0 && ds.idx < a.vocab && load_one<__nv_bfloat16>(rowq, ds.idx) == ds.ml;
                sh.stat_ok = ok;
                sh.x_ml[1] = ds.ml; sh.x_sx[1] = ds.sx; sh.x_idx[1] = ok ? ds.idx : 0;
            } else {
                sh.x_ml[1] = Qs.ml; sh.x_sx[1] = Qs.sx; sh.x_idx[1] = Qs.idx;
            }
        }
    }
    __syncthreads();
    RowStat P, Q;
    merge_slices<1>(sh, 0, k, P);
    merge_slices<1>(sh, 1, k, Q);
    float Zp = P.sx + P.own;
    const float Zq = Q.sx + Q.own;
    float cP = P.C, invZp = 1.f / Zp;
    const float cQ = Q.C, invZq = 1.f / Zq;
    float rho = __fdiv_rn(Zp, Zq);
    if (STATS && !sh.stat_ok) {
        for (int m = 0; m < 3; ++m) o[m].status = SPECHUB_ST_STATS;
        finish();
        return;
    }
    auto prob_p = [&](int y) { return prob_of(load_one<__nv_bfloat16>(rowp, y), k, cP, invZp); };
    auto prob_q = [&](int y) { return prob_of(load_one<__nv_bfloat16>(rowq, y), k, cQ, invZq); };
    auto draw_from_p = [&]() { return lean_sample_row<1>(g, rowp, k, P, 0, -1, ures, 0, sh); };

    if (!(P.ml > neg_inf()) || !(P.ml < pinf) || !finite_pos(Zp)) {
        for (int m = 0; m < 3; ++m) o[m].status = SPECHUB_ST_NONFINITE;
        finish();
        return;
    }
    if (!(Q.ml > neg_inf()) || !(Q.ml < pinf) || !finite_pos(Zq)) {
        for (int m = 0; m < 3; ++m) o[m].status = SPECHUB_ST_NONFINITE;
        finish();
        return;
    }
    // ---- per-method draft tokens ----
    const int hubtok = Q.idx;
    const int sx1 = A.tok[0][2 * r], sx2 = A.tok[0][2 * r + 1];
    const bool pair_xa = (sx2 == hubtok && sx1 != hubtok), pair_ax = (sx1 == hubtok && sx2 != hubtok);
    const int x = pair_xa ? sx1 : sx2;
    const bool ok_s = (pair_xa || pair_ax) && x >= 0 && x < a.vocab;
    int rx1[2], rx2[2];
    bool ok_r[2];
    for (int m = 0; m < 2; ++m) {
        rx1[m] = A.tok[1 + m][2 * r]; rx2[m] = A.tok[1 + m][2 * r + 1];
        ok_r[m] = rx1[m] >= 0 && rx1[m] < a.vocab && rx2[m] >= 0 && rx2[m] < a.vocab;
    }
    o[0].hub = hubtok;
    if (!ok_s) o[0].status = SPECHUB_ST_TOKEN_RANGE;
    if (!ok_r[0]) o[1].status = SPECHUB_ST_TOKEN_RANGE;
    if (!ok_r[1]) o[2].status = SPECHUB_ST_TOKEN_RANGE;
    const bool degenerate = !(Q.sx > 0.f);
    const float c = degenerate ? 0.f : Q.own / Q.sx;
    float crho = c * rho;
    const float qa = Q.own * invZq, rest = Q.sx * invZq;
    const int hubvec = hubtok >> 3, hubel = hubtok & 7;
    const int wx1 = ok_r[1] ? rx1[1] : -1;            // RRSw's first draft (left out of its renormaliser)
    const int wvec = wx1 >> 3, wel = wx1 & 7;

    // ---- pass B (backwards): SpecHub S1, S2, R; A1; RRSw's sum of q outside its x1 ----
    float s1a, s2a, ra, s1b, s2b, rb, a1a, a1b, dna, dnb;
    unsigned diff = 0;
    auto pass_b = [&]() {
    // (packed as in lean_verify_kernel: the low lane of a pair takes the even ids of a vector, the high lane the
    // odd ones; every sum keeps the association of the per-method kernels)
    F2 s1 = f2_make(0.f, 0.f), s2 = s1, rr = s1, a1 = s1;
    dna = dnb = 0.f;
    const F2 k2 = f2_make(k, k), ncp2 = f2_make(-cP, -cP), ncq2 = f2_make(-cQ, -cQ);
    const F2 nrho2 = f2_make(-rho, -rho), ncrho2 = f2_make(-crho, -crho);
#pragma unroll 2
    for (int vi = last_vi; vi >= lo; vi -= 32) {
        const uint4 rawp = vp[vi], rawq = vq[vi];
        if (STATS) diff |= (rawp.x ^ rawq.x) | (rawp.y ^ rawq.y) | (rawp.z ^ rawq.z) | (rawp.w ^ rawq.w);
        const unsigned wps[4] = {rawp.x, rawp.y, rawp.z, rawp.w}, wqs[4] = {rawq.x, rawq.y, rawq.z, rawq.w};
        float qw[8];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const F2 ep = f2_exp_word(wps[i], k2, ncp2);
            F2 eq = f2_exp_word(wqs[i], k2, ncq2);
            if (!STATS) f2_get(eq, qw[2 * i], qw[2 * i + 1]);
            F2 d = f2_fma(nrho2, eq, ep);              // Z_p (p - q)
            F2 m = f2_max0(d);
            a1 = f2_add(a1, m);                         // RRS / RRSw: over every id
            if (vi == hubvec && i == (hubel >> 1)) {    // SpecHub's sums run over ids != a: that lane adds 0
                float d0, d1, q0, q1;
                f2_get(d, d0, d1);
                f2_get(eq, q0, q1);
                if (hubel & 1) { d1 = 0.f; q1 = 0.f; } else { d0 = 0.f; q0 = 0.f; }
                d = f2_make(d0, d1);
                eq = f2_make(q0, q1);
                m = f2_max0(d);
            }
            const F2 t = f2_fma(ncrho2, eq, m);         // Z_p (max(p - q, 0) - c q)
            const F2 w = f2_max0(t);
            s1 = f2_add(s1, f2_sub(m, d));              // max(-d, 0) = max(d, 0) - d, exactly
            s2 = f2_add(s2, f2_sub(w, t));
            rr = f2_add(rr, w);
        }
        if (!STATS) {   // RRSw's renormaliser leaves its x1 out (from draft statistics: sum_without, below)
            if (vi == wvec) {
#pragma unroll
                for (int i = 0; i < 8; ++i)
                    if (i == wel) qw[i] = 0.f;
            }
            dna += (qw[0] + qw[1]) + (qw[2] + qw[3]);
            dnb += (qw[4] + qw[5]) + (qw[6] + qw[7]);
        }
    }
    f2_get(s1, s1a, s1b);
    f2_get(s2, s2a, s2b);
    f2_get(rr, ra, rb);
    f2_get(a1, a1a, a1b);
    };
    pass_b();
    if (STATS && !__syncthreads_or(diff != 0)) {   // the target row is the draft row: Z_p = Z_q exactly
        Zp = Zq; invZp = invZq; cP = cQ; rho = 1.f; crho = c;
        pass_b();
    }
    float accB[5] = {s1a + s1b, s2a + s2b, ra + rb, a1a + a1b, dna + dnb};
    lean_block_sums<5, 0>(accB, sh);   // per-warp R stays in sh.acc[2]
    if (STATS) accB[4] = wx1 >= 0 ? sum_without(Q, rowq, wx1, k) : 0.f;
    const float Rraw = accB[2];
    const float S1 = accB[0] * invZp, S2 = degenerate ? qa : accB[1] * invZp, R = Rraw * invZp;
    const float A1 = accB[3] * invZp, den = accB[4] * invZq;

    // ---- pass C (forwards): second-stage residual masses of RRS and RRSw ----
    const bool q1_zero = !(den > 0.f);
    const float A1g[2] = {A1, A1 * (q1_zero ? 0.f : 1.f / den)};
    const float A1grho[2] = {A1g[0] * rho, A1g[1] * rho};
    float w0a, w0b, w1a, w1b;
    {
        F2 w0 = f2_make(0.f, 0.f), w1 = w0;
        const F2 k2 = f2_make(k, k), ncp2 = f2_make(-cP, -cP), ncq2 = f2_make(-cQ, -cQ), nrho2 = f2_make(-rho, -rho);
        const F2 nsc0 = f2_make(-A1grho[0], -A1grho[0]), nsc1 = f2_make(-A1grho[1], -A1grho[1]);
        uint64_t polf;   // the rows' last use: L2 may let these lines go first
        asm("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(polf));
#pragma unroll 2
        for (int vi = lo + lane; vi < hi; vi += 32) {
            const uint4 rawp = ld_l2_hint(vp + vi, polf), rawq = ld_l2_hint(vq + vi, polf);
            const unsigned wps[4] = {rawp.x, rawp.y, rawp.z, rawp.w}, wqs[4] = {rawq.x, rawq.y, rawq.z, rawq.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                F2 nsc = nsc1;
                if (vi == wvec && i == (wel >> 1)) nsc = (wel & 1) ? f2_make(-A1grho[1], 0.f) : f2_make(0.f, -A1grho[1]);
                const F2 eq = f2_exp_word(wqs[i], k2, ncq2);
                const F2 m = f2_max0(f2_fma(nrho2, eq, f2_exp_word(wps[i], k2, ncp2)));
                w0 = f2_add(w0, f2_max0(f2_fma(nsc0, eq, m)));
                w1 = f2_add(w1, f2_max0(f2_fma(nsc, eq, m)));
            }
        }
        f2_get(w0, w0a, w0b);
        f2_get(w1, w1a, w1b);
    }
    float accC[2] = {w0a + w0b, w1a + w1b};
    lean_block_sums<2, 5>(accC, sh);   // per-warp W2 stay in sh.acc[5], sh.acc[6]
    __syncthreads();

    // ---- SpecHub decisions (Algorithm 3) ----
    if (ok_s) {
        NodeResult &s = o[0];
        const float pa = prob_p(hubtok);
        const float hub_left = fmaxf(pa - S2, 0.f);
        s.rate[0] = fmaxf(rest - S1, 0.f) + fminf(pa, S2);
        s.rate[1] = (degenerate ? 0.f : fmaxf(qa - S2, 0.f)) + fminf(hub_left, S1);
        s.rate[2] = R;
        if (degenerate) s.status |= SPECHUB_ST_DEGENERATE_Q;
        const float px = prob_p(x), qx = prob_q(x);
        bool acc1, acc2;
        if (pair_xa) {
            acc1 = accept_test(r1, px, qx, s.beta[0], true, s.status);
            if (acc1) { s.accept_idx = 0; s.token = x; }
            acc2 = accept_test(r2, hub_left, S1, s.beta[1], !acc1, s.status);
            if (!acc1 && acc2) { s.accept_idx = 1; s.token = hubtok; }
        } else {
            acc1 = accept_test(r1, fmaxf(__fsub_rn(px, qx), 0.f), c * qx, s.beta[0], true, s.status);
            if (acc1) { s.accept_idx = 1; s.token = x; }
            acc2 = accept_test(r2, pa, S2, s.beta[1], !acc1, s.status);
            if (!acc1 && acc2) { s.accept_idx = 0; s.token = hubtok; }
        }
        if (!(acc1 || acc2)) {
            s.accept_idx = -1;
            int tok;
            if (Rraw > 0.f) {
                if (threadIdx.x < g.nwarps) sh.mass[threadIdx.x] = sh.acc[2][threadIdx.x];
                __syncthreads();
                auto wf = [&](int vi, float(&w)[8]) {
                    float fp[8], fq[8];
                    unpack_bf16x8(vp[vi], fp);
                    unpack_bf16x8(vq[vi], fq);
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        float d, t;
                        lean_terms(lean_exp(fp[i], k, cP), lean_exp(fq[i], k, cQ), rho, crho, d, t);
                        w[i] = (vi * 8 + i == hubtok) ? 0.f : fmaxf(t, 0.f);
                    }
                };
                tok = block_sample3(g, wf, sh, ures * Rraw);
            } else {
                s.status |= SPECHUB_ST_ZERO_RESIDUAL;
                tok = draw_from_p();
            }
            s.token = tok;
        }
    }
    // ---- RRS / RRSw decisions (Algorithm 1) ----
#pragma unroll
    for (int m = 0; m < 2; ++m) {
        if (!ok_r[m]) continue;
        NodeResult &s = o[1 + m];
        const bool wo = (m == 1);
        const float W2raw = accC[m], W2 = W2raw * invZp;
        const int x1 = rx1[m], x2 = rx2[m];
        s.rate[0] = fmaxf(1.f - A1, 0.f);
        s.rate[1] = fmaxf(A1 - W2, 0.f);
        s.rate[2] = W2;
        const float px1 = prob_p(x1), qx1 = prob_q(x1), px2 = prob_p(x2), qx2 = prob_q(x2);
        const bool acc1 = accept_test(r1, px1, qx1, s.beta[0], true, s.status);
        if (acc1) { s.accept_idx = 0; s.token = x1; }
        if (!acc1 && wo && q1_zero) s.status |= SPECHUB_ST_DEGENERATE_Q;
        bool acc2 = false;
        if (A1 > 0.f) {
            const float q1x2 = (wo && x2 == x1) ? 0.f : A1g[m] * qx2;
            acc2 = accept_test(r2, fmaxf(__fsub_rn(px2, qx2), 0.f), q1x2, s.beta[1], !acc1, s.status);
        }
        if (!acc1 && acc2) { s.accept_idx = 1; s.token = x2; }
        if (!(acc1 || acc2)) {
            s.accept_idx = -1;
            int tok;
            if (A1 > 0.f && W2raw > 0.f) {
                if (threadIdx.x < g.nwarps) sh.mass[threadIdx.x] = sh.acc[5 + m][threadIdx.x];
                __syncthreads();
                const float coef = A1grho[m];
                auto wf = [&](int vi, float(&w)[8]) {
                    float fp[8], fq[8];
                    unpack_bf16x8(vp[vi], fp);
                    unpack_bf16x8(vq[vi], fq);
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        float d, t;
                        const float sc = (wo && vi * 8 + i == x1) ? 0.f : coef;
                        lean_terms(lean_exp(fp[i], k, cP), lean_exp(fq[i], k, cQ), rho, sc, d, t);
                        w[i] = fmaxf(t, 0.f);
                    }
                };
                tok = block_sample3(g, wf, sh, ures * W2raw);
            } else {
                s.status |= SPECHUB_ST_ZERO_RESIDUAL;
                tok = draw_from_p();
            }
            s.token = tok;
        }
    }
    finish();
}

// Draft step of the three methods from one read of q (the checkpointed pass A and sampler of
// lean_draft_ck_kernel).  x1 ~ q is the same draw for all three: they share u_d1.
template <int THREADS>
__global__ void __launch_bounds__(THREADS, 1024 / THREADS) fused_draft_kernel(FusedArgs A, int32_t *hub_out,
                                                                            float *draft_prob) {
    __shared__ LeanCkShared sh;
    const RowArgs &a = A.r;
    const long long r = blockIdx.x;
    const int b = static_cast<int>(r / a.nodes), n = static_cast<int>(r % a.nodes);
    const __nv_bfloat16 *rowq = static_cast<const __nv_bfloat16 *>(a.draft) + b * a.stride_seq + n * a.stride_node;
    const uint4 *vq = reinterpret_cast<const uint4 *>(rowq);
    const Geo g = make_geo(a.vocab, 8);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int lo = g.seg_lo(warp), hi = g.seg_hi(warp);
    const float k = kLog2e / temperature_of(a, b);
    const float u1 = a.uniforms[r * 5 + 0], u2 = a.uniforms[r * 5 + 1];
    const bool t0 = threadIdx.x == 0;
    const int CK = lean_ck_interval(g);

    LeanAcc tq, unused;
    unused.m2 = 0xff80ff80u; unused.s = 0.f; unused.c = 0.f;
    lean_pass_a_ck(vq, lo, hi, lane, k, CK, tq, sh.cks[warp], sh.ckc[warp]);
    {
        ArgMaxSum q, unusedq;
        lean_reduce2<false>(tq, unused, vq, vq, lo, hi, k, sh, q, unusedq);
        if (t0) { sh.x_ml[0] = q.ml; sh.x_sx[0] = q.sx; sh.x_idx[0] = q.idx; }
    }
    __syncthreads();
    RowStat Q;
    merge_slices<1>(sh, 0, k, Q);
    const float Zq = Q.sx + Q.own;
    if (t0 && a.draft_stats_out) {   // the record lean_draft_ck_kernel leaves, bit for bit
        DraftStat ds;
        ds.ml = Q.ml; ds.sx = Q.sx; ds.idx = Q.idx; ds.tag = kDraftStatTag ^ __float_as_uint(k);
        static_cast<DraftStat *>(a.draft_stats_out)[r] = ds;
    }
    if (!(Q.ml > neg_inf()) || !finite_pos(Zq) || !(Q.ml < -neg_inf())) {
        if (t0) {
            for (int m = 0; m < 3; ++m) {
                A.tok_out[m][2 * r] = -1; A.tok_out[m][2 * r + 1] = -1;
                if (A.dstatus[m]) A.dstatus[m][r] = SPECHUB_ST_NONFINITE;
            }
            if (hub_out) hub_out[r] = -1;
            if (draft_prob) { draft_prob[2 * r] = 0.f; draft_prob[2 * r + 1] = 0.f; }
        }
        return;
    }
    const int hubtok = Q.idx;
    const int x1 = lean_ck_sample(g, rowq, k, Q.C, CK, -1, u1, sh);
    uint32_t st[3] = {0, 0, 0};
    int x2[3];
    // SpecHub (Section 4)
    const float prob0 = Q.own / Zq;
    float prob1 = 0.f;
    if (x1 != hubtok) {
        x2[0] = hubtok;
        prob1 = ex2(fmaf(load_one<__nv_bfloat16>(rowq, x1), k, -Q.C)) / Zq;
    } else if (!(Q.sx > 0.f)) {
        x2[0] = (hubtok == 0) ? 1 : 0;
        st[0] |= SPECHUB_ST_DEGENERATE_Q;
    } else {
        x2[0] = lean_ck_sample(g, rowq, k, Q.C, CK, hubtok, u2, sh);
        prob1 = prob0 * ex2(fmaf(load_one<__nv_bfloat16>(rowq, x2[0]), k, -Q.C)) / Q.sx;
    }
    // RRS: an independent second draw
    x2[1] = lean_ck_sample(g, rowq, k, Q.C, CK, -1, u2, sh);
    // RRSw: q with q(x1) set to 0
    x2[2] = lean_ck_sample(g, rowq, k, Q.C, CK, x1, u2, sh);
    if (x2[2] < 0) {
        x2[2] = (x1 == 0) ? 1 : 0;
        st[2] |= SPECHUB_ST_DEGENERATE_Q;
    }
    if (t0) {
        for (int m = 0; m < 3; ++m) {
            A.tok_out[m][2 * r] = x1;
            A.tok_out[m][2 * r + 1] = x2[m];
            if (A.dstatus[m]) A.dstatus[m][r] = st[m];
        }
        if (hub_out) hub_out[r] = hubtok;
        if (draft_prob) { draft_prob[2 * r] = prob0; draft_prob[2 * r + 1] = prob1; }
    }
}

}  // namespace spechub
