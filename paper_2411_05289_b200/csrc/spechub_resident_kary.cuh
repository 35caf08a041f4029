// Algorithm 1 with k > 2 drafts per node on the exponentials kept on chip (see spechub_resident.cuh
// for the storage: e_p in tensor memory, e_q in shared memory and registers, one integer exponent
// reference per thread and row, a row spread over the CS CTAs of a cluster).
//
// Unnormalised form of Algorithm 1, in units of 1 / Z_p:  P_0 = E_p,  m_0 = 1 and for stage j = 1..k
//   q_j = q (RRS), or q with q(x_1..x_{j-1}) zeroed, over den_j = its remaining mass (RRSw)
//   test j:  accept x_j  iff  r_j m_{j-1} q_j(x_j) < P_{j-1}(x_j) / Z_p
//   P_j = max(P_{j-1} - m_{j-1} g_j rho E_q, 0),   m_j = sum_y P_j(y) / Z_p,   g_j = 1 / den_j
// m_j needs m_{j-1}, so every stage is one pass -- over tensor / shared memory, not over HBM: the
// row pair is read once, the stored P is updated in place, and each stage costs one FMA and one
// maximum per id (the streaming kernel re-reads the row and recomputes two exponentials per id and
// stage).  After a stage every warp writes its sum into every CTA of the row, and every warp adds
// the records up by itself, in the same order: no CTA waits for one warp to broadcast.
#pragma once

#include "spechub_kary.cuh"
#include "spechub_resident.cuh"

namespace spechub {

struct __align__(16) ResKaryShared {
    float recA[kResMaxParts][8];      // c_p, s_p, c_q, s_q, s_q without the drafts x_1..x_{k-1}
    float recS[2][kResMaxParts][8];   // a stage's sum of P_j; [4..8): per batch.  Two buffers, by stage parity
    float bc[8];
    int bi[8];
    uint32_t tmem_base;
};

template <int CS>
__global__ void __launch_bounds__(kResThreads, 2) resident_kary_kernel(KaryArgs A, int NB, uint32_t tmem_cols) {
    constexpr int W = CS * kResWarps;
    extern __shared__ float4 eq_store[];
    __shared__ ResKaryShared sh;

    const RowArgs &a = A.r;
    const int K = A.k;
    const bool wo = A.without_replacement != 0;
    const int me = RowGroup<CS>::rank();
    const long long r = blockIdx.x / CS;
    const int b = static_cast<int>(r / a.nodes), n = static_cast<int>(r % a.nodes);
    const bool leaf = a.node_kind && a.node_kind[n] == SPECHUB_NODE_LEAF;   // the bonus token: a draw from p
    res_arrive<CS>();   // [0] "this CTA runs"

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (warp == 0) tmem_alloc(res_smem_addr(&sh.tmem_base), tmem_cols);

    const __nv_bfloat16 *rowp = static_cast<const __nv_bfloat16 *>(a.target) + b * a.stride_seq + n * a.stride_node;
    const __nv_bfloat16 *rowq = static_cast<const __nv_bfloat16 *>(a.draft) + b * a.stride_seq + n * a.stride_node;
    const uint4 *vp = reinterpret_cast<const uint4 *>(rowp), *vq = reinterpret_cast<const uint4 *>(rowq);
    const int V = a.vocab, nvec = V >> 3;
    const int g = me * kResWarps + warp;
    const int seg = (((nvec + W - 1) / W) + 7) & ~7;
    const int lo = min(g * seg, nvec), hi = min(lo + seg, nvec);
    const float k = kLog2e / temperature_of(a, b);
    const V2 k2 = v2_make(k, k);
    const float *un = a.uniforms + r * (2 * K + 1);
    const bool writer = (me == 0 && threadIdx.x == 0);
    const int LB = NB - 1;

    // drafts and the logits at them
    int x[kMaxK];
    float lpx[kMaxK], lqx[kMaxK];
    bool bad_tok = false;
    for (int i = 0; i < K; ++i) {
        x[i] = leaf ? 0 : a.draft_tokens_in[K * r + i];
        const bool ok = x[i] >= 0 && x[i] < V;
        bad_tok |= !ok;
        lpx[i] = load_one<__nv_bfloat16>(rowp, ok ? x[i] : 0);
        lqx[i] = load_one<__nv_bfloat16>(rowq, ok ? x[i] : 0);
    }
    // RRSw takes the drafts out of q stage by stage.  Where a draft lies in what this lane stores:
    // one bit per stored exponential of a batch (bit = 8 * vector of the batch + element).
    bool tok_warp = false;           // this warp's range holds one of x_1..x_{k-1}
    auto tok_bit = [&](int i, int &bt) -> unsigned {   // draft i in this lane's storage: its batch and bit, or 0
        const int v = x[i] >> 3;
        if (!(x[i] >= 0 && v >= lo && v < hi && ((v - lo) & 31) == lane)) return 0u;
        const int slot = (v - lo) >> 5;
        bt = slot >> 2;
        return 1u << ((slot & 3) * 8 + (x[i] & 7));
    };
    auto mask_of = [&](const unsigned (&mk)[4], int bt) {
        return bt == 0 ? mk[0] : bt == 1 ? mk[1] : bt == 2 ? mk[2] : mk[3];
    };
    unsigned mask_all[4] = {0u, 0u, 0u, 0u};   // x_1..x_{k-1}: left out of the sum that gives the renormalisers
    unsigned mask_cum[4] = {0u, 0u, 0u, 0u};   // the drafts drawn before the current stage
    if (wo && !leaf) {
        for (int i = 0; i < K - 1; ++i) {
            const int v = x[i] >> 3;
            tok_warp |= (x[i] >= 0 && v >= lo && v < hi);
            int bt = 0;
            const unsigned bit = tok_bit(i, bt);
#pragma unroll
            for (int b4 = 0; b4 < 4; ++b4)
                if (b4 == bt) mask_all[b4] |= bit;
        }
    }

    const uint32_t lane_field = static_cast<uint32_t>((warp & 3) * 32) << 16;
    const uint32_t col0 = static_cast<uint32_t>((warp >> 2) * (32 * NB));
    auto eq_ptr = [&](int slot) { return eq_store + (2 * slot) * kResThreads + threadIdx.x; };
    auto load_eq_batch = [&](int bt, float (&e)[32]) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float4 *src = eq_ptr(4 * bt + j);
            const float4 u = src[0], w = src[kResThreads];
            e[8 * j + 0] = u.x; e[8 * j + 1] = u.y; e[8 * j + 2] = u.z; e[8 * j + 3] = u.w;
            e[8 * j + 4] = w.x; e[8 * j + 5] = w.y; e[8 * j + 6] = w.z; e[8 * j + 7] = w.w;
        }
    };

    // ---- pass A: the only read of the row pair (as in resident_verify_kernel) ----------------------
    float c_pt = kNoRef, c_qt = kNoRef;
    V2 pacc[4], qacc[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) pacc[i] = qacc[i] = v2_make(0.f, 0.f);
    uint32_t taddr = 0;
    float eqk[32];
    auto rescale_stored = [&](int upto, float fp, float fq) {
        tmem_wait_st();
        for (int b2 = 0; b2 < upto; ++b2) {
            float t[32];
            tmem_ld32(taddr + 32 * b2, t);
#pragma unroll
            for (int i = 0; i < 32; ++i) t[i] = mul_ftz(t[i], fp);
            tmem_st32(taddr + 32 * b2, t);
            if (b2 < LB) {
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    float4 *ptr = eq_ptr(4 * b2 + j);
                    float4 u = ptr[0], w = ptr[kResThreads];
                    u.x = mul_ftz(u.x, fq); u.y = mul_ftz(u.y, fq); u.z = mul_ftz(u.z, fq); u.w = mul_ftz(u.w, fq);
                    w.x = mul_ftz(w.x, fq); w.y = mul_ftz(w.y, fq); w.z = mul_ftz(w.z, fq); w.w = mul_ftz(w.w, fq);
                    ptr[0] = u; ptr[kResThreads] = w;
                }
            }
        }
        tmem_wait_st();
    };
#pragma unroll 1
    for (int bt = 0; bt < NB; ++bt) {
        ResRaw R;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int vi = lo + lane + 32 * (4 * bt + j);
            R.p[j] = R.q[j] = make_uint4(0xff80ff80u, 0xff80ff80u, 0xff80ff80u, 0xff80ff80u);
            if (vi < hi) {
                R.p[j] = ld_stream(vp + vi);
                if (!leaf) R.q[j] = ld_stream(vq + vi);
            }
        }
        const float rpb = res_ref(res_max4(R.p), k), rqb = res_ref(res_max4(R.q), k);
        if (bt == 0) {
            c_pt = rpb; c_qt = rqb;
            tmem_fence_before();
            __syncthreads();
            tmem_fence_after();
            taddr = sh.tmem_base + lane_field + col0;
        } else {
            const bool mvp = rpb > c_pt + kRefSlack, mvq = rqb > c_qt + kRefSlack;
            if (__any_sync(kFull, mvp || mvq)) {
                const float fp = mvp ? res_pow2(c_pt - rpb) : 1.f, fq = mvq ? res_pow2(c_qt - rqb) : 1.f;
                rescale_stored(bt, fp, fq);
                const V2 fp2 = v2_make(fp, fp), fq2 = v2_make(fq, fq), z2 = v2_make(0.f, 0.f);
#pragma unroll
                for (int i = 0; i < 4; ++i) { pacc[i] = v2_fma(pacc[i], fp2, z2); qacc[i] = v2_fma(qacc[i], fq2, z2); }
                if (mvp) c_pt = rpb;
                if (mvq) c_qt = rqb;
            }
        }
        const V2 ncp2 = v2_make(-c_pt, -c_pt), ncq2 = v2_make(-c_qt, -c_qt);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            float e[8];
            res_exp8(R.p[j], k2, ncp2, e, pacc);
            tmem_st8(taddr + 8 * (4 * bt + j), e);
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            float e[8];
            res_exp8(R.q[j], k2, ncq2, e, qacc);
            if (bt == LB) {
#pragma unroll
                for (int i = 0; i < 8; ++i) eqk[8 * j + i] = e[i];
            } else {
                float4 *dst = eq_ptr(4 * bt + j);
                dst[0] = make_float4(e[0], e[1], e[2], e[3]);
                dst[kResThreads] = make_float4(e[4], e[5], e[6], e[7]);
            }
        }
    }
    tmem_wait_st();
    {
        const float sp_t = res_total(pacc), sq_t = res_total(qacc);
        const float cpw = warp_max(c_pt), cqw = warp_max(c_qt);
        const float fpw = res_pow2(c_pt - cpw), fqw = res_pow2(c_qt - cqw);
        const float spw = warp_sum(__fmul_rn(sp_t, fpw)), sqw = warp_sum(__fmul_rn(sq_t, fqw));
        float sxw = sqw;
        if (tok_warp) {   // this warp's e_q without the drafts x_1..x_{k-1}, term by term
            float s0 = 0.f;
            for (int bt = 0; bt < NB; ++bt) {
                float e[32];
                if (bt < LB) {
                    load_eq_batch(bt, e);
                } else {
#pragma unroll
                    for (int i = 0; i < 32; ++i) e[i] = eqk[i];
                }
                const unsigned mk = mask_of(mask_all, bt);
#pragma unroll
                for (int i = 0; i < 32; ++i) s0 += ((mk >> i) & 1u) ? 0.f : e[i];
            }
            sxw = warp_sum(__fmul_rn(s0, fqw));
        }
        const float4 rec[2] = {make_float4(cpw, spw, cqw, sqw), make_float4(sxw, 0.f, 0.f, 0.f)};
        if (CS > 1) res_wait<CS>();   // [0]
        res_push<CS, 2>(sh.recA[g], rec, lane);
    }
    res_arrive<CS>();
    res_wait<CS>();   // [1] pass-A records exchanged
    // every warp merges the records by itself (same order, same result everywhere)
    float Cp, Cq, Zp, Zq, Zex;
    {
        const int g0 = 2 * lane, g1 = 2 * lane + 1;
        float c0 = kNoRef, s0 = 0.f, d0 = kNoRef, q0 = 0.f, y0 = 0.f, c1 = kNoRef, s1 = 0.f, d1 = kNoRef, q1 = 0.f, y1 = 0.f;
        if (g0 < W) { const float *rc = sh.recA[g0]; c0 = rc[0]; s0 = rc[1]; d0 = rc[2]; q0 = rc[3]; y0 = rc[4]; }
        if (g1 < W) { const float *rc = sh.recA[g1]; c1 = rc[0]; s1 = rc[1]; d1 = rc[2]; q1 = rc[3]; y1 = rc[4]; }
        Cp = warp_max(fmaxf(c0, c1));
        Cq = warp_max(fmaxf(d0, d1));
        const float f0 = res_pow2(c0 - Cp), f1 = res_pow2(c1 - Cp), h0 = res_pow2(d0 - Cq), h1 = res_pow2(d1 - Cq);
        Zp = warp_sum(__fadd_rn(__fmul_rn(s0, f0), __fmul_rn(s1, f1)));
        Zq = warp_sum(__fadd_rn(__fmul_rn(q0, h0), __fmul_rn(q1, h1)));
        Zex = warp_sum(__fadd_rn(__fmul_rn(y0, h0), __fmul_rn(y1, h1)));
    }
    const float invZp = 1.f / Zp, invZq = 1.f / Zq, rho = __fdiv_rn(Zp, Zq);
    const float ures = un[2 * K];

    int accept_idx = -1, token = -1;
    uint32_t status = 0;
    float beta[kMaxK], rate[kMaxK + 1];
    for (int i = 0; i < K; ++i) beta[i] = 0.f;
    for (int i = 0; i <= K; ++i) rate[i] = 0.f;
    bool token_elsewhere = false;
    // 0: nothing to draw, 1: from the stored P (the residual after k rejections), 2: from p
    int drawkind = 0;
    float m[kMaxK + 1], coef[kMaxK], den[kMaxK], px[kMaxK], qx[kMaxK];
    m[0] = 1.f;

    const bool bad_p = !finite_pos(Zp), bad_q = !leaf && !finite_pos(Zq);
    const bool run = !(bad_p || bad_q || leaf || bad_tok);
    if (bad_p || bad_q) status = SPECHUB_ST_NONFINITE;
    else if (leaf) { drawkind = 2; rate[K] = 1.f; token_elsewhere = true; }
    else if (bad_tok) status = SPECHUB_ST_TOKEN_RANGE;

    // this thread's scales (see resident_verify_kernel)
    float np = (c_pt == kNoRef) ? 0.f : c_pt - Cp, nq = (c_qt == kNoRef) ? 0.f : c_qt - Cq;
    if (run) {
        const bool far = np < -kRefFar || nq < -kRefFar;
        if (__any_sync(kFull, far)) {
            const float fp = far ? res_pow2(np) : 1.f, fq = far ? res_pow2(nq) : 1.f;
            rescale_stored(NB, fp, fq);
#pragma unroll
            for (int i = 0; i < 32; ++i) eqk[i] = mul_ftz(eqk[i], fq);
            if (far) { np = 0.f; nq = 0.f; }
        }
    }
    const float F = res_pow2(np), sc = res_pow2(nq - np);

    if (run) {
        for (int i = 0; i < K; ++i) {
            px[i] = prob_of(lpx[i], k, Cp, invZp);
            qx[i] = prob_of(lqx[i], k, Cq, invZq);
            den[i] = 1.f;
        }
        if (wo) {
            // den[l] = (q outside x[0..K-1)) + q of the distinct tokens among x[l..K-1) not in x[0..l)
            const float base = Zex * invZq;
            for (int l = 1; l < K; ++l) {
                float d = base;
                for (int t = l; t < K - 1; ++t)
                    if (!in_set(x, l, x[t]) && !in_set(x + l, t - l, x[t])) d += qx[t];
                den[l] = d;
            }
        }
        // ---- the k stages, each a pass over the stored P and e_q ----------------------------------------
        for (int j = 1; j <= K; ++j) {
            const float gj = wo ? (den[j - 1] > 0.f ? 1.f / den[j - 1] : 0.f) : 1.f;
            coef[j - 1] = m[j - 1] * gj;
            const float ct = __fmul_rn(__fmul_rn(coef[j - 1], rho), sc);   // per unit of e_q on this thread's scale
            const V2 nc2 = v2_make(-ct, -ct);
            float Mw = 0.f;
            float *recs = sh.recS[j & 1][g];
            if (tok_warp && j > 1) {   // x_{j-1} leaves q from this stage on
                int btk = 0;
                const unsigned bit = tok_bit(j - 2, btk);
#pragma unroll
                for (int b4 = 0; b4 < 4; ++b4)
                    if (b4 == btk) mask_cum[b4] |= bit;
            }
            for (int bt = 0; bt < NB; ++bt) {
                float P[32], eq[32];
                tmem_ld32(taddr + 32 * bt, P);
                if (bt < LB) {
                    load_eq_batch(bt, eq);
                } else {
#pragma unroll
                    for (int i = 0; i < 32; ++i) eq[i] = eqk[i];
                }
                V2 acc = v2_make(0.f, 0.f);
                if (tok_warp && j > 1) {   // RRSw: drafts drawn before this stage carry no draft mass in it
                    const unsigned mk = mask_of(mask_cum, bt);
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        if ((mk >> i) & 1u) eq[i] = 0.f;
                }
#pragma unroll
                for (int i = 0; i < 32; i += 2) {
                    const V2 pn = v2_max0(v2_fma(nc2, v2_make(eq[i], eq[i + 1]), v2_make(P[i], P[i + 1])));
                    v2_get(pn, P[i], P[i + 1]);
                    acc = v2_add(acc, pn);
                }
                tmem_st32(taddr + 32 * bt, P);
                const float sb = warp_sum(mul_ftz(v2_sum(acc), F));
                if (lane < CS) {
                    float *dst = recs + 4 + bt;
                    if (CS > 1) dst = cooperative_groups::this_cluster().map_shared_rank(dst, lane);
                    *dst = sb;
                }
                Mw += sb;
            }
            tmem_wait_st();
            if (lane < CS) {
                float *dst = recs;
                if (CS > 1) dst = cooperative_groups::this_cluster().map_shared_rank(dst, lane);
                *dst = Mw;
            }
            res_arrive<CS>();
            res_wait<CS>();   // stage j exchanged
            const int g0 = 2 * lane, g1 = 2 * lane + 1;
            const float Mj = warp_sum((g0 < W ? sh.recS[j & 1][g0][0] : 0.f) + (g1 < W ? sh.recS[j & 1][g1][0] : 0.f));
            m[j] = Mj * invZp;
        }
        // ---- the tests (every warp alike) ---------------------------------------------------------------
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
            token_elsewhere = true;
            if (m[K] > 0.f) drawkind = 1;
            else { status |= SPECHUB_ST_ZERO_RESIDUAL; drawkind = 2; }
        }
    }
    if (writer) {
        a.accept_idx[r] = accept_idx;
        if (!token_elsewhere) a.token[r] = token;
        if (a.hub) a.hub[r] = -1;
        if (a.beta) for (int i = 0; i < K; ++i) a.beta[K * r + i] = beta[i];
        if (a.rate) for (int i = 0; i <= K; ++i) a.rate[(K + 1) * r + i] = rate[i];
        if (a.status) a.status[r] = status;
    }

    // ---- the draw -------------------------------------------------------------------------------------
    if (drawkind == 1) {
        // the (warp, batch) part that holds the target, from the last stage's records; that warp walks it
        float mm[8], base = 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int gg = 2 * lane + (i >> 2), bt = i & 3;
            mm[i] = (gg < W && bt < NB) ? sh.recS[K & 1][gg][4 + bt] : 0.f;
        }
        float tot = 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i) tot += mm[i];
        tot = warp_sum(tot);
        const int part = res_pick8(mm, ures * tot, lane, base);
        if (part < 0) {
            if (writer) a.token[r] = -1;
        } else if ((part >> 2) == g) {
            const int bt = part & 3;
            const float tt = ures * tot - base;
            float P[32];
            tmem_ld32(taddr + 32 * bt, P);
            float prefix = 0.f;
            int found = -1, lastpos = -1;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                if (found < 0) {
                    const int vi = lo + lane + 32 * (4 * bt + j);
                    float w[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) w[i] = mul_ftz(P[8 * j + i], F);
                    res_scan_step(w, vi, lane, tt, prefix, found, lastpos);
                }
            }
            if (found < 0) found = lastpos;
            if (lane == 0) a.token[r] = found;
        }
    } else if (drawkind == 2) {
        // a draw from p: the bonus token of a leaf, or the fallback when the residual has no mass.  The
        // stored P has been consumed by the stages, so the picked warp reads its range of the row again.
        const int g0 = 2 * lane, g1 = 2 * lane + 1;
        float mm[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f}, base = 0.f;
        if (g0 < W) mm[0] = __fmul_rn(sh.recA[g0][1], res_pow2(sh.recA[g0][0] - Cp));
        if (g1 < W) mm[4] = __fmul_rn(sh.recA[g1][1], res_pow2(sh.recA[g1][0] - Cp));
        const float tot = warp_sum(mm[0] + mm[4]);
        const int part = res_pick8(mm, ures * tot, lane, base);
        if (part < 0) {
            if (writer) a.token[r] = -1;
        } else if ((part >> 2) == g) {
            const float tt = ures * tot - base;
            float prefix = 0.f;
            int found = -1, lastpos = -1;
            for (int v0 = lo; v0 < hi && found < 0; v0 += 32) {
                const int vi = v0 + lane;
                float w[8];
                if (vi < hi) {
                    float v[8];
                    unpack_bf16x8(vp[vi], v);
#pragma unroll
                    for (int i = 0; i < 8; ++i) w[i] = ex2(__fmaf_rn(v[i], k, -Cp));
                } else {
#pragma unroll
                    for (int i = 0; i < 8; ++i) w[i] = 0.f;
                }
                res_scan_step(w, vi, lane, tt, prefix, found, lastpos);
            }
            if (found < 0) found = lastpos;
            if (lane == 0) a.token[r] = found;
        }
    }

    tmem_fence_before();
    __syncthreads();
    if (warp == 0) {
        tmem_fence_after();
        tmem_dealloc(sh.tmem_base, tmem_cols);
    }
}

}  // namespace spechub
