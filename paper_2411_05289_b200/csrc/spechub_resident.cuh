// Register-resident kernels for bf16 rows that fit on chip (sm_100a).
//
// One thread-block cluster owns one (sequence, node) row at a time and loops
// over rows (persistent, one CTA per SM).  CTA r of the cluster owns the
// contiguous slice [r*Lc, (r+1)*Lc) of the vocabulary.  Per row:
//
//   load   the two bf16 slices arrive in shared memory through bulk async copies
//          (TMA, completion on an mbarrier), double buffered: the copy of the
//          row after next is issued as soon as a buffer is free, so HBM is kept
//          busy while the current row is being worked on;
//   pass A each thread reads its NV vectors once, takes its local maximum with
//          packed bf16 max, and computes e(y) = 2^(k l(y) - c_thread) ONCE, into
//          registers; these 16*NV exponentials per thread are all later passes
//          read (the special-function pipe, 16 ex2/clk/SM, is the scarcest
//          resource on this path, so nothing is exponentiated twice);
//   reduce (max, argmax, sum without the argmax) per warp -> CTA -> cluster; the
//          cluster level goes through distributed shared memory and a hardware
//          cluster barrier;
//   pass B the closed-form transport sums from the cached exponentials;
//   decide accept / reject on scalars; on rejection the CTA whose slice holds the
//          target mass draws the residual token from its registers.
//
// Only hardware barriers and one bounded mbarrier wait (the copy's completion)
// are waited on.  If that wait expires the row is flagged SPECHUB_ST_INTERNAL,
// and the cluster barriers are still executed by every thread.
#pragma once

#include <cooperative_groups.h>

#include "spechub.h"
#include "spechub_common.cuh"
#include "spechub_stream.cuh"

namespace spechub {
namespace cg = cooperative_groups;

constexpr int kResThreads = 512;
constexpr int kResWarps = kResThreads / 32;
constexpr int kMaxCluster = 8;
constexpr uint32_t kWaitLimit = 1u << 22;  // try_wait rounds before giving up on a copy

// ---- PTX helpers ----------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_addr(const void *p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(unsigned long long *bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(unsigned long long *bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(unsigned long long *bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_addr(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bulk async copy global -> this CTA's shared memory.  Addresses and size are multiples of 16.
__device__ __forceinline__ void bulk_load(void *dst_smem, const void *src, uint32_t bytes,
                                          unsigned long long *bar) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
            smem_addr(dst_smem)),
        "l"(src), "r"(bytes), "r"(smem_addr(bar))
        : "memory");
}

// ---- shared-memory control block ------------------------------------------------------------------
struct LeafX {  // what one CTA tells the cluster after pass A
    float p_ml, p_sx, q_ml, q_sx;
    int p_idx, q_idx;
    float lx[4];  // raw logits lp[x1], lq[x1], lp[x2], lq[x2] when the token lies in this slice
    int failed;   // this CTA's copy did not complete within the wait limit
};
struct SumX {  // ... and after pass B
    float s[4];
    float lpa;  // raw target logit of the hub when it lies in this slice
};
struct ResShared {
    unsigned long long full[2];
    LeafX xa;
    SumX xb;
    float wml[2][kResWarps];   // per-warp max logit (0: target, 1: draft)
    float wsx[2][kResWarps];   // per-warp sum of exponentials relative to the warp max
    int cand[2];               // lowest index attaining the CTA maximum
    float wacc[4][kResWarps];  // per-warp pass-B sums
    float mass[kResWarps];
    float bc[24];              // broadcast scalars
    int bi[8];
    int tok;
    int failed;
};

struct ResArgs {
    RowArgs r;
    int rows;   // batch * nodes
    int Lc;     // slice length in elements (multiple of 8)
};

// vector lv (local) of thread: warp*32*NV + j*32 + lane
template <int NV>
__device__ __forceinline__ int local_vec(int warp, int lane, int j) {
    return warp * (32 * NV) + j * 32 + lane;
}

__device__ __forceinline__ void unpack8(const uint4 &v, float (&o)[8]) {
    o[0] = __uint_as_float(v.x << 16); o[1] = __uint_as_float(v.x & 0xffff0000u);
    o[2] = __uint_as_float(v.y << 16); o[3] = __uint_as_float(v.y & 0xffff0000u);
    o[4] = __uint_as_float(v.z << 16); o[5] = __uint_as_float(v.z & 0xffff0000u);
    o[6] = __uint_as_float(v.w << 16); o[7] = __uint_as_float(v.w & 0xffff0000u);
}

__device__ __forceinline__ unsigned bfmax2(unsigned a, unsigned b) {
    unsigned d;
    asm("max.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}

// Pass A of one slice for one thread: local max logit and e[] relative to it.
// Vectors past the slice read as -inf.  Returns the plain sum of e[].
template <int NV>
__device__ __forceinline__ float pass_a_thread(const __nv_bfloat16 *slice, int len, int warp, int lane,
                                               float k, float (&e)[NV * 8], float &ml, float &c) {
    uint4 raw[NV];
    const unsigned ninf2 = 0xff80ff80u;
#pragma unroll
    for (int j = 0; j < NV; ++j) {
        const int lv = local_vec<NV>(warp, lane, j);
        if (lv * 8 < len) raw[j] = *reinterpret_cast<const uint4 *>(slice + lv * 8);
        else raw[j] = make_uint4(ninf2, ninf2, ninf2, ninf2);
    }
    unsigned m2 = ninf2;
#pragma unroll
    for (int j = 0; j < NV; ++j) {
        m2 = bfmax2(m2, bfmax2(bfmax2(raw[j].x, raw[j].y), bfmax2(raw[j].z, raw[j].w)));
    }
    ml = fmaxf(__uint_as_float(m2 << 16), __uint_as_float(m2 & 0xffff0000u));
    c = shift_of(ml, k);
    float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
    for (int j = 0; j < NV; ++j) {
        float v[8];
        unpack8(raw[j], v);
#pragma unroll
        for (int i = 0; i < 8; ++i) e[j * 8 + i] = ex2(__fmaf_rn(v[i], k, -c));
        s0 += e[j * 8 + 0] + e[j * 8 + 4];
        s1 += e[j * 8 + 1] + e[j * 8 + 5];
        s2 += e[j * 8 + 2] + e[j * 8 + 6];
        s3 += e[j * 8 + 3] + e[j * 8 + 7];
    }
    return (s0 + s1) + (s2 + s3);
}

// Sum of e[] without element `skip` (same association as pass_a_thread's sum).
template <int NV>
__device__ __forceinline__ float sum_without(const float (&e)[NV * 8], int skip) {
    float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
    for (int j = 0; j < NV; ++j) {
#define E_(t) ((j * 8 + (t)) == skip ? 0.f : e[j * 8 + (t)])
        s0 += E_(0) + E_(4);
        s1 += E_(1) + E_(5);
        s2 += E_(2) + E_(6);
        s3 += E_(3) + E_(7);
#undef E_
    }
    return (s0 + s1) + (s2 + s3);
}

// First position (0 .. NV*8-1, in the thread's own order) whose raw logit equals `val`; -1 if none.
template <int NV>
__device__ __forceinline__ int first_equal(const __nv_bfloat16 *slice, int len, int warp, int lane,
                                           float val) {
    int pos = -1;
    for (int j = NV - 1; j >= 0; --j) {
        const int lv = local_vec<NV>(warp, lane, j);
        if (lv * 8 >= len) continue;
        const uint4 raw = *reinterpret_cast<const uint4 *>(slice + lv * 8);
        float v[8];
        unpack8(raw, v);
#pragma unroll
        for (int i = 7; i >= 0; --i) pos = (v[i] == val) ? j * 8 + i : pos;
    }
    return pos;
}

// Token id of position `pos` of this thread.
template <int NV>
__device__ __forceinline__ int token_of(int slice_base, int warp, int lane, int pos) {
    return slice_base + local_vec<NV>(warp, lane, pos >> 3) * 8 + (pos & 7);
}

// CTA-wide inverse-CDF draw over weights held in registers.  w[] are this thread's weights in
// its own order; mass[warp] (shared) the per-warp totals computed with the same arithmetic.
// tt = target within this CTA's slice.  Returns the token to every thread (-1 if the slice has
// no mass).  Called by all threads of the CTA.
template <int NV>
__device__ int resident_sample(const float (&w)[NV * 8], const float *mass, float tt, int slice_base,
                               int *sh_tok) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    int wsel = -1, lastw = -1;
    float base = 0.f, lastbase = 0.f, run = 0.f;
    for (int x = 0; x < kResWarps; ++x) {
        const float m = mass[x];
        if (m > 0.f) {
            lastw = x;
            lastbase = run;
            if (wsel < 0 && run + m > tt) { wsel = x; base = run; }
        }
        run += m;
    }
    if (wsel < 0) { wsel = lastw; base = lastbase; }
    if (lastw < 0) return -1;
    if (warp == wsel) {
        const float t2 = tt - base;
        float prefix = 0.f;
        int found = -1, lastpos = -1;
#pragma unroll
        for (int j = 0; j < NV; ++j) {
            if (found < 0) {
                float lsum = 0.f;
                int lp = -1;
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    lsum += w[j * 8 + i];
                    if (w[j * 8 + i] > 0.f) lp = j * 8 + i;
                }
                float incl = lsum;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const float up = __shfl_up_sync(kFull, incl, o);
                    if (lane >= o) incl += up;
                }
                const float tot = __shfl_sync(kFull, incl, 31);
                const unsigned hit = __ballot_sync(kFull, lsum > 0.f && prefix + incl > t2);
                if (hit) {
                    const int L = __ffs(hit) - 1;
                    int cand = -1;
                    if (lane == L) {
                        float acc = prefix + (incl - lsum);
                        int lastin = -1;
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            acc += w[j * 8 + i];
                            if (w[j * 8 + i] > 0.f) {
                                lastin = j * 8 + i;
                                if (cand < 0 && acc > t2) cand = lastin;
                            }
                        }
                        if (cand < 0) cand = lastin;
                        cand = token_of<NV>(slice_base, warp, lane, cand);
                    }
                    found = __shfl_sync(kFull, cand, L);
                } else {
                    int lt = (lp >= 0) ? token_of<NV>(slice_base, warp, lane, lp) : -1;
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) lt = max(lt, __shfl_xor_sync(kFull, lt, o));
                    lastpos = max(lastpos, lt);
                    prefix += tot;
                }
            }
        }
        if (found < 0) found = lastpos;
        if (lane == 0) *sh_tok = found;
    }
    __syncthreads();
    const int tok = *sh_tok;
    __syncthreads();
    return tok;
}

// ------------------------------------------------------------------------------------------------
// SpecHub verification, resident.
// ------------------------------------------------------------------------------------------------
template <int NV>
__global__ void __launch_bounds__(kResThreads, 1) resident_spechub_kernel(ResArgs A) {
    extern __shared__ __align__(128) unsigned char dyn_smem[];
    ResShared &sh = *reinterpret_cast<ResShared *>(dyn_smem);
    constexpr int kCtl = (sizeof(ResShared) + 127) / 128 * 128;
    const RowArgs &a = A.r;
    const int Lc = A.Lc;
    __nv_bfloat16 *buf = reinterpret_cast<__nv_bfloat16 *>(dyn_smem + kCtl);  // [2][2][Lc]

    cg::cluster_group cluster = cg::this_cluster();
    const int C = static_cast<int>(cluster.num_blocks());
    const int rank = static_cast<int>(cluster.block_rank());
    const int cid = blockIdx.x / C, ncl = gridDim.x / C;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int V = a.vocab;
    const int slice_base = rank * Lc;
    const int len = max(0, min(Lc, V - slice_base));
    const __nv_bfloat16 *gp = static_cast<const __nv_bfloat16 *>(a.target);
    const __nv_bfloat16 *gq = static_cast<const __nv_bfloat16 *>(a.draft);
    const float pinf = -neg_inf();

    auto is_leaf = [&](int row) { return a.node_kind && a.node_kind[row % a.nodes] == SPECHUB_NODE_LEAF; };
    auto issue = [&](int it) {  // thread 0 only
        const int row = cid + it * ncl;
        if (row >= A.rows || len == 0) return;
        const int b = it & 1;
        const long long off = static_cast<long long>(row / a.nodes) * a.stride_seq +
                              static_cast<long long>(row % a.nodes) * a.stride_node + slice_base;
        const uint32_t bytes = static_cast<uint32_t>(len) * 2u;
        const bool leaf = is_leaf(row);
        mbar_expect_tx(&sh.full[b], leaf ? bytes : 2u * bytes);
        bulk_load(buf + (b * 2 + 0) * Lc, gp + off, bytes, &sh.full[b]);
        if (!leaf) bulk_load(buf + (b * 2 + 1) * Lc, gq + off, bytes, &sh.full[b]);
    };

    if (tid == 0) {
        mbar_init(&sh.full[0], 1);
        mbar_init(&sh.full[1], 1);
        mbar_fence_init();
        sh.failed = 0;
    }
    __syncthreads();
    if (tid == 0) { issue(0); issue(1); }

    for (int it = 0;; ++it) {
        const int row = cid + it * ncl;
        if (row >= A.rows) break;
        const int b = it & 1;
        const uint32_t parity = static_cast<uint32_t>((it >> 1) & 1);
        const int bseq = row / a.nodes;
        const bool leaf = is_leaf(row);
        const float k = kLog2e / temperature_of(a, bseq);
        const int x1 = a.draft_tokens_in[2 * row], x2 = a.draft_tokens_in[2 * row + 1];
        const float r1 = a.uniforms[row * 5 + 2], r2 = a.uniforms[row * 5 + 3], ures = a.uniforms[row * 5 + 4];
        const __nv_bfloat16 *sp = buf + (b * 2 + 0) * Lc, *sq = buf + (b * 2 + 1) * Lc;

        // ---- wait for the slices (bounded) ----
        if (len > 0) {
            uint32_t spins = 0;
            while (!mbar_try_wait(&sh.full[b], parity)) {
                if (++spins > kWaitLimit) { sh.failed = 1; break; }
            }
        }
        if (tid == 0) { sh.cand[0] = 0x7fffffff; sh.cand[1] = 0x7fffffff; }

        // ---- pass A: exponentials into registers ----
        float ep[NV * 8], eq[NV * 8];
        float mlp, cp, mlq = neg_inf(), cq = 0.f;
        float sp_t = pass_a_thread<NV>(sp, len, warp, lane, k, ep, mlp, cp);
        float sq_t = 0.f;
        if (!leaf) sq_t = pass_a_thread<NV>(sq, len, warp, lane, k, eq, mlq, cq);
        else {
#pragma unroll
            for (int i = 0; i < NV * 8; ++i) eq[i] = 0.f;
        }
        // warp maxima
        float wmp = mlp, wmq = mlq;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            wmp = fmaxf(wmp, __shfl_xor_sync(kFull, wmp, o));
            wmq = fmaxf(wmq, __shfl_xor_sync(kFull, wmq, o));
        }
        if (lane == 0) { sh.wml[0][warp] = wmp; sh.wml[1][warp] = wmq; }
        __syncthreads();  // (1)
        float cmp = sh.wml[0][0], cmq = sh.wml[1][0];
#pragma unroll
        for (int w = 1; w < kResWarps; ++w) { cmp = fmaxf(cmp, sh.wml[0][w]); cmq = fmaxf(cmq, sh.wml[1][w]); }
        // candidates for the CTA argmax find their first matching element
        int posp = -1, posq = -1;
        if (mlp == cmp && cmp > neg_inf()) {
            posp = first_equal<NV>(sp, len, warp, lane, cmp);
            atomicMin(&sh.cand[0], token_of<NV>(slice_base, warp, lane, posp));
        }
        if (!leaf && mlq == cmq && cmq > neg_inf()) {
            posq = first_equal<NV>(sq, len, warp, lane, cmq);
            atomicMin(&sh.cand[1], token_of<NV>(slice_base, warp, lane, posq));
        }
        __syncthreads();  // (2)
        const int idxp = sh.cand[0], idxq = sh.cand[1];
        const bool own_p = posp >= 0 && token_of<NV>(slice_base, warp, lane, posp) == idxp;
        const bool own_q = posq >= 0 && token_of<NV>(slice_base, warp, lane, posq) == idxq;
        // the owner's sum leaves its maximum out (1 - q(a) must be a direct sum)
        if (own_p) sp_t = sum_without<NV>(ep, posp);
        if (own_q) sq_t = sum_without<NV>(eq, posq);
        {
            const float cwp = shift_of(wmp, k), cwq = shift_of(wmq, k);
            float vp = sp_t * rescale(mlp, cp, cwp), vq = sq_t * rescale(mlq, cq, cwq);
            vp = warp_sum(vp);
            vq = warp_sum(vq);
            if (lane == 0) { sh.wsx[0][warp] = vp; sh.wsx[1][warp] = vq; }
        }
        __syncthreads();  // (3)
        const float ccp = shift_of(cmp, k), ccq = shift_of(cmq, k);
        if (warp == 0) {
            float vp = 0.f, vq = 0.f;
            if (lane < kResWarps) {
                const float a0 = sh.wml[0][lane], a1 = sh.wml[1][lane];
                vp = sh.wsx[0][lane] * rescale(a0, shift_of(a0, k), ccp);
                vq = sh.wsx[1][lane] * rescale(a1, shift_of(a1, k), ccq);
            }
            vp = warp_sum(vp);
            vq = warp_sum(vq);
            if (lane == 0) {
                sh.xa.p_ml = cmp; sh.xa.p_sx = vp; sh.xa.p_idx = idxp;
                sh.xa.q_ml = cmq; sh.xa.q_sx = vq; sh.xa.q_idx = idxq;
                const bool in1 = x1 >= slice_base && x1 < slice_base + len;
                const bool in2 = x2 >= slice_base && x2 < slice_base + len;
                sh.xa.lx[0] = in1 ? load_one<__nv_bfloat16>(sp, x1 - slice_base) : 0.f;
                sh.xa.lx[1] = (in1 && !leaf) ? load_one<__nv_bfloat16>(sq, x1 - slice_base) : 0.f;
                sh.xa.lx[2] = in2 ? load_one<__nv_bfloat16>(sp, x2 - slice_base) : 0.f;
                sh.xa.lx[3] = (in2 && !leaf) ? load_one<__nv_bfloat16>(sq, x2 - slice_base) : 0.f;
                sh.xa.failed = sh.failed;
            }
        }
        cluster.sync();  // [A]
        // ---- merge the CTA leaves (warp 0), broadcast ----
        if (warp == 0) {
            ArgMaxSum P, Q;
            P.init(); Q.init();
            int fail = 0;
            if (lane < C) {
                const LeafX *px = cluster.map_shared_rank(&sh.xa, lane);
                P.ml = px->p_ml; P.c = shift_of(P.ml, k); P.sx = px->p_sx; P.idx = px->p_idx;
                Q.ml = px->q_ml; Q.c = shift_of(Q.ml, k); Q.sx = px->q_sx; Q.idx = px->q_idx;
                fail = px->failed;
            }
            P = argmaxsum_warp(P);
            Q = argmaxsum_warp(Q);
            fail = __any_sync(kFull, fail != 0);
            if (lane == 0) {
                sh.bc[0] = P.ml; sh.bc[1] = P.sx; sh.bc[2] = Q.ml; sh.bc[3] = Q.sx;
                sh.bi[0] = P.idx; sh.bi[1] = Q.idx; sh.bi[2] = fail;
                const int o1 = (x1 >= 0 && x1 < V) ? x1 / Lc : 0, o2 = (x2 >= 0 && x2 < V) ? x2 / Lc : 0;
                const LeafX *l1 = cluster.map_shared_rank(&sh.xa, o1), *l2 = cluster.map_shared_rank(&sh.xa, o2);
                sh.bc[4] = l1->lx[0]; sh.bc[5] = l1->lx[1]; sh.bc[6] = l2->lx[2]; sh.bc[7] = l2->lx[3];
            }
        }
        __syncthreads();  // (4)
        const float Pml = sh.bc[0], Psx = sh.bc[1], Qml = sh.bc[2], Qsx = sh.bc[3];
        const int hubtok = sh.bi[1];
        const bool failed = sh.bi[2] != 0;
        const float Zp = Psx + 1.f, Zq = Qsx + 1.f;
        const float CP = shift_of(Pml, k), CQ = shift_of(Qml, k);

        NodeResult o;
        o.accept_idx = -1; o.token = -1; o.hub = -1; o.status = 0;
        o.beta[0] = o.beta[1] = 0.f; o.rate[0] = o.rate[1] = o.rate[2] = 0.f;
        bool done = false;        // output complete without pass B
        bool need_sample = false; // a residual / leaf draw is required
        int sample_kind = 0;      // 0: residual, 1: from p
        if (failed) {
            o.status = SPECHUB_ST_INTERNAL; done = true;
        } else if (!(Pml > neg_inf()) || !(Pml < pinf) || !finite_pos(Zp)) {
            o.status = SPECHUB_ST_NONFINITE; done = true;
        } else if (!leaf && (!(Qml > neg_inf()) || !(Qml < pinf) || !finite_pos(Zq))) {
            o.status = SPECHUB_ST_NONFINITE; done = true;
        }
        const float invZp = 1.f / Zp, invZq = 1.f / Zq;
        const float fp_t = rescale(mlp, cp, CP) * invZp;   // e -> probability, this thread's elements
        const float fq_t = rescale(mlq, cq, CQ) * invZq;
        bool pair_xa = false, pair_ax = false;
        int x = -1;
        if (!done && !leaf) {
            o.hub = hubtok;
            pair_xa = (x2 == hubtok && x1 != hubtok);
            pair_ax = (x1 == hubtok && x2 != hubtok);
            x = pair_xa ? x1 : x2;
            if (!(pair_xa || pair_ax) || x < 0 || x >= V) { o.status = SPECHUB_ST_TOKEN_RANGE; done = true; }
        }
        const bool degenerate = !(Qsx > 0.f);
        const float c = degenerate ? 0.f : 1.f / Qsx;
        float S1 = 0.f, S2 = 0.f, R = 0.f, pa = 0.f;
        const bool run_b = !done && !leaf;   // cluster-uniform
        if (run_b) {
            // the hub's pair carries no mass in the sums below: zero it in the owning thread
            if (own_q && idxq == hubtok) {
#pragma unroll
                for (int i = 0; i < NV * 8; ++i) {
                    if (i == posq) { ep[i] = 0.f; eq[i] = 0.f; }
                }
            }
            // ---- pass B: transport sums over ids != a (Section 4, Appendix B.1) ----
            float a0 = 0.f, a1 = 0.f, a2 = 0.f, b0 = 0.f, b1 = 0.f, b2 = 0.f;
#pragma unroll
            for (int i = 0; i < NV * 8; i += 2) {
                float d, t;
                transport_terms(__fmul_rn(ep[i], fp_t), __fmul_rn(eq[i], fq_t), c, d, t);
                a0 += fmaxf(-d, 0.f); a1 += fmaxf(-t, 0.f); a2 += fmaxf(t, 0.f);
                transport_terms(__fmul_rn(ep[i + 1], fp_t), __fmul_rn(eq[i + 1], fq_t), c, d, t);
                b0 += fmaxf(-d, 0.f); b1 += fmaxf(-t, 0.f); b2 += fmaxf(t, 0.f);
            }
            const float s1 = warp_sum(a0 + b0), s2 = warp_sum(a1 + b1), s3 = warp_sum(a2 + b2);
            if (lane == 0) { sh.wacc[0][warp] = s1; sh.wacc[1][warp] = s2; sh.wacc[2][warp] = s3; }
        }
        __syncthreads();  // (5)
        if (warp == 0) {
            float v0 = 0.f, v1 = 0.f, v2 = 0.f;
            if (run_b && lane < kResWarps) { v0 = sh.wacc[0][lane]; v1 = sh.wacc[1][lane]; v2 = sh.wacc[2][lane]; }
            v0 = warp_sum(v0); v1 = warp_sum(v1); v2 = warp_sum(v2);
            if (lane == 0) {
                sh.xb.s[0] = v0; sh.xb.s[1] = v1; sh.xb.s[2] = v2;
                // per-CTA mass of p for a draw from p (leaf, or empty residual)
                sh.xb.s[3] = (sh.xa.p_sx + (sh.xa.p_ml > neg_inf() ? 1.f : 0.f)) *
                             rescale(sh.xa.p_ml, shift_of(sh.xa.p_ml, k), CP);
                const bool hub_here = run_b && hubtok >= slice_base && hubtok < slice_base + len;
                sh.xb.lpa = hub_here ? load_one<__nv_bfloat16>(sp, hubtok - slice_base) : 0.f;
            }
        }
        cluster.sync();  // [B]
        if (warp == 0) {
            float v[4] = {0.f, 0.f, 0.f, 0.f};
            if (lane < C) {
                const SumX *px = cluster.map_shared_rank(&sh.xb, lane);
#pragma unroll
                for (int i = 0; i < 4; ++i) v[i] = px->s[i];
            }
            // ordered totals (rank order) and each rank's residual / target mass for the draw
            float t0 = 0.f, t1 = 0.f, t2 = 0.f, t3 = 0.f;
            for (int rr = 0; rr < C; ++rr) {
                t0 += __shfl_sync(kFull, v[0], rr);
                t1 += __shfl_sync(kFull, v[1], rr);
                const float m2 = __shfl_sync(kFull, v[2], rr), m3 = __shfl_sync(kFull, v[3], rr);
                if (lane == 0) { sh.bc[12 + rr] = m2; sh.wacc[3][rr] = m3; }
                t2 += m2; t3 += m3;
            }
            if (lane == 0) {
                sh.bc[8] = t0; sh.bc[9] = t1; sh.bc[10] = t2; sh.bc[20] = t3;
                const int oh = (hubtok >= 0 && hubtok < V) ? hubtok / Lc : 0;
                sh.bc[11] = cluster.map_shared_rank(&sh.xb, oh)->lpa;
            }
        }
        __syncthreads();  // (6)
        if (run_b) {
            S1 = sh.bc[8]; S2 = degenerate ? invZq : sh.bc[9]; R = sh.bc[10];
            const float qa = invZq, rest = Qsx * invZq;
            pa = prob_of(sh.bc[11], k, CP, invZp);
            const float hub_left = fmaxf(pa - S2, 0.f);
            o.rate[0] = fmaxf(rest - S1, 0.f) + fminf(pa, S2);
            o.rate[1] = (degenerate ? 0.f : fmaxf(qa - S2, 0.f)) + fminf(hub_left, S1);
            o.rate[2] = R;
            if (degenerate) o.status |= SPECHUB_ST_DEGENERATE_Q;
            const float px = prob_of(pair_xa ? sh.bc[4] : sh.bc[6], k, CP, invZp);
            const float qx = prob_of(pair_xa ? sh.bc[5] : sh.bc[7], k, CQ, invZq);
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
                need_sample = true;
                if (!(R > 0.f)) { sample_kind = 1; o.status |= SPECHUB_ST_ZERO_RESIDUAL; }
            }
        } else if (!done && leaf) {
            need_sample = true; sample_kind = 1; o.rate[2] = 1.f;
        }
        if (need_sample) {
            // which CTA's slice holds the target mass (rank order = ascending token ids)
            const float *cm = (sample_kind == 0) ? &sh.bc[12] : &sh.wacc[3][0];
            float total = 0.f;
            for (int rr = 0; rr < C; ++rr) total += cm[rr];
            const float t = ures * total;
            int osel = -1, lasto = -1;
            float base = 0.f, lastbase = 0.f, run = 0.f;
            for (int rr = 0; rr < C; ++rr) {
                const float m = cm[rr];
                if (m > 0.f) {
                    lasto = rr; lastbase = run;
                    if (osel < 0 && run + m > t) { osel = rr; base = run; }
                }
                run += m;
            }
            if (osel < 0) { osel = lasto; base = lastbase; }
            if (rank == osel) {
                if (sample_kind == 1) {
                    // weights: p's exponentials on the common scale (all ids, the hub included)
                    const float fs = rescale(mlp, cp, CP);
                    float wp[NV * 8];
                    if (run_b) {
                        // ep was zeroed at the hub for pass B: this path (empty residual) needs it back
                        const float e_hub = ex2(__fmaf_rn(sh.bc[11], k, -cp));
#pragma unroll
                        for (int i = 0; i < NV * 8; ++i)
                            wp[i] = ((own_q && idxq == hubtok && i == posq) ? e_hub : ep[i]) * fs;
                    } else {
#pragma unroll
                        for (int i = 0; i < NV * 8; ++i) wp[i] = ep[i] * fs;
                    }
                    float ws = 0.f;
#pragma unroll
                    for (int i = 0; i < NV * 8; ++i) ws += wp[i];
                    ws = warp_sum(ws);
                    if (lane == 0) sh.mass[warp] = ws;
                    __syncthreads();
                    const int tok = resident_sample<NV>(wp, sh.mass, t - base, slice_base, &sh.tok);
                    if (tid == 0) a.token[row] = tok;
                } else {
                    // residual weights p''(y), recomputed with pass B's arithmetic
                    float w[NV * 8];
#pragma unroll
                    for (int i = 0; i < NV * 8; ++i) {
                        float d, tt;
                        transport_terms(__fmul_rn(ep[i], fp_t), __fmul_rn(eq[i], fq_t), c, d, tt);
                        w[i] = fmaxf(tt, 0.f);
                    }
                    if (tid < kResWarps) sh.mass[tid] = sh.wacc[2][tid];
                    __syncthreads();
                    const int tok = resident_sample<NV>(w, sh.mass, t - base, slice_base, &sh.tok);
                    if (tid == 0) a.token[row] = tok;
                }
            }
        }
        if (rank == 0 && tid == 0) {
            a.accept_idx[row] = o.accept_idx;
            if (!need_sample) a.token[row] = o.token;
            if (a.hub) a.hub[row] = o.hub;
            if (a.beta) { a.beta[2 * row] = o.beta[0]; a.beta[2 * row + 1] = o.beta[1]; }
            if (a.rate) { a.rate[3 * row] = o.rate[0]; a.rate[3 * row + 1] = o.rate[1]; a.rate[3 * row + 2] = o.rate[2]; }
            if (a.status) a.status[row] = o.status;
        }
        __syncthreads();  // (7) every reader of this buffer and of the control block is done
        if (tid == 0) issue(it + 2);
    }
    cluster.sync();  // no CTA leaves while a peer may still read its shared memory
}

}  // namespace spechub
