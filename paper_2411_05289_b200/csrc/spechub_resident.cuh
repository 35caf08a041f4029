// Verification with the exponentials resident on chip: every row is read from HBM exactly once.
//
// The transport sums of Section 4 / Appendix B.1 (and the residual masses of Algorithm 1) need
// Z_p, Z_q, the hub a and c = q(a) / (1 - q(a)), which are known only when the whole row has been
// seen.  Instead of reading the logits a second time, pass A keeps what it computed from them, as
// fp32, relative to one integer exponent reference per thread and row (c = rint(k * the maximum of
// the thread's first batch), so every later rescaling is an exact power of two):
//
//   e_p(y) = 2^(k l_p(y) - c_p)   in tensor memory (tcgen05.st / tcgen05.ld, 32x32b shape: lane i of
//                                 a warp owns TMEM lane i, 32 columns per batch of four vectors),
//   e_q(y) = 2^(k l_q(y) - c_q)   in shared memory, the thread's last batch in registers.
//
// A row of V ids takes 8 V bytes on chip.  It is spread over the CS CTAs of a thread-block cluster
// (CS = 1 up to V = 32768, 2, 4, 8 beyond), 8 warps each, up to four batches per lane.  At four
// batches a CTA holds 128 KB in tensor memory (256 columns), 96 KB in shared memory and 32
// registers per thread, so two CTAs of different rows share an SM and one row's exchanges overlap
// the other row's streaming.
//
// Warp g of a row (g = 8 * cluster rank + warp) owns a contiguous range of vectors, hence of token
// ids; after each pass it writes one small record into the shared memory of every CTA of its row
// (distributed shared memory), a cluster barrier follows, and warp 0 of each CTA merges the
// records in a fixed order and takes the row's decisions.  Every CTA thus computes bit-identical
// row values.  Passes B and C and the residual draw read tensor / shared memory only: 2 ex2 per
// vocabulary pair in all.  The arithmetic of the passes is packed two fp32 lanes per instruction
// (fma / add / sub .f32x2), which halves their issue slots.
//
// One kernel template serves SpecHub, RRS, RRSw and the three together (MASK): the per-method
// results of the combined kernel are, by construction, those of the separate ones bit for bit.
//
// Tensor memory is allocated by warp 0 (tcgen05.alloc) and released before the CTA ends on every
// path.  The CTAs that fit an SM by their shared memory and registers never ask for more than its
// 512 columns, so the allocation never waits for a CTA of this kernel.
#pragma once

#include <cooperative_groups.h>

#include <type_traits>

#include "spechub.h"
#include "spechub_common.cuh"
#include "spechub_stream.cuh"
#include "spechub_tmem.cuh"
#include "spechub_lean.cuh"
#include "spechub_fused.cuh"

namespace spechub {

constexpr int kResThreads = 256;
constexpr int kResWarps = 8;
constexpr int kResMaxParts = 64;     // warps per row: 8 CTAs x 8 warps at most
constexpr int kResMaxBatches = 4;    // batches of four 16-byte vectors per lane
constexpr float kNoRef = -1.0e30f;   // exponent reference of a thread that has seen no finite logit
constexpr int kNoIdx = 0x7fffffff;
constexpr float kRefSlack = 32.f;    // a thread's exponentials stay below 2^32 on its own scale
constexpr float kRefFar = 50.f;      // references farther than this below the row's are brought to it

enum { kMaskSpecHub = 1, kMaskRRS = 2, kMaskRRSw = 4 };

struct __align__(16) ResShared {
    // per-part records, one slot per warp of the row, written by that warp into every CTA's copy
    float recA[kResMaxParts][12];  // c_p, s_p, c_q, s_q, max l_q, first id of the candidate hub logit,
                                   // s_q without exclusion candidate 0, 1, 2
    float recB[kResMaxParts][8];   // S1, S2, R (SpecHub), A1 (RRS / RRSw); R of each of the warp's batches
    float recC[kResMaxParts][12];  // W2 of RRS, W2 of RRSw, -, -; W2 of RRS per batch; W2 of RRSw per batch
    int recH[kResMaxParts];        // first id of the row maximum (rows whose pair lacks the hub)
    float bc[24];                  // row values from warp 0 to the CTA
    int bi[12];
    uint32_t tmem_base;
};

// ---- PTX wrappers (tensor memory: spechub_tmem.cuh) ---------------------------------------------
__device__ __forceinline__ uint4 ld_stream(const uint4 *p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}
__device__ __forceinline__ float mul_ftz(float a, float b) {
    float d;
    asm("mul.rn.ftz.f32 %0, %1, %2;" : "=f"(d) : "f"(a), "f"(b));
    return d;
}

// Two fp32 lanes in one 64-bit register pair, one instruction for both (fma / add / sub .f32x2).
// Subnormal results are flushed, as ex2.approx.ftz does for the exponentials themselves.
struct V2 {
    unsigned long long v;
};
__device__ __forceinline__ V2 v2_make(float lo, float hi) {
    V2 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r.v) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void v2_get(V2 a, float &lo, float &hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(a.v));
}
__device__ __forceinline__ V2 v2_fma(V2 a, V2 b, V2 c) {
    V2 d;
    asm("fma.rn.ftz.f32x2 %0, %1, %2, %3;" : "=l"(d.v) : "l"(a.v), "l"(b.v), "l"(c.v));
    return d;
}
__device__ __forceinline__ V2 v2_add(V2 a, V2 b) {
    V2 d;
    asm("add.rn.ftz.f32x2 %0, %1, %2;" : "=l"(d.v) : "l"(a.v), "l"(b.v));
    return d;
}
__device__ __forceinline__ V2 v2_sub(V2 a, V2 b) {
    V2 d;
    asm("sub.rn.ftz.f32x2 %0, %1, %2;" : "=l"(d.v) : "l"(a.v), "l"(b.v));
    return d;
}
__device__ __forceinline__ V2 v2_max0(V2 a) {   // lane-wise max(a, 0)
    float lo, hi;
    v2_get(a, lo, hi);
    return v2_make(fmaxf(lo, 0.f), fmaxf(hi, 0.f));
}
__device__ __forceinline__ float v2_sum(V2 a) {
    float lo, hi;
    v2_get(a, lo, hi);
    return lo + hi;
}

template <int CS>
__device__ __forceinline__ void res_arrive() {
    if (CS > 1) asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
}
// Completes an exchange: every record written before the matching arrive is visible afterwards.
template <int CS>
__device__ __forceinline__ void res_wait() {
    if (CS > 1) asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
    else __syncthreads();
}
// Lanes 0..CS-1 of a warp store its record into the copy of CTA `lane` of the row.
template <int CS, int NF4>
__device__ __forceinline__ void res_push(float *slot, const float4 (&v)[NF4], int lane) {
    if (lane < CS) {
        float *dst = slot;
        if (CS > 1) dst = cooperative_groups::this_cluster().map_shared_rank(slot, lane);
#pragma unroll
        for (int i = 0; i < NF4; ++i) reinterpret_cast<float4 *>(dst)[i] = v[i];
    }
}

// ---- exponent references -------------------------------------------------------------------------
// Integer reference for a largest logit m: rint(k m).  Monotone in m.
__device__ __forceinline__ float res_ref(float m, float k) { return m > neg_inf() ? rintf(__fmul_rn(m, k)) : kNoRef; }
// 2^n for an integer-valued n (exact); 0 below the normal range and for NaN
__device__ __forceinline__ float res_pow2(float n) {
    return n >= -126.f ? __int_as_float((__float2int_rn(fminf(n, 127.f)) + 127) << 23) : 0.f;
}
__device__ __forceinline__ float warp_max(float x) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x = fmaxf(x, __shfl_xor_sync(kFull, x, o));
    return x;
}
__device__ __forceinline__ int warp_min_int(int x) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x = min(x, __shfl_xor_sync(kFull, x, o));
    return x;
}
__device__ __forceinline__ float res_max4(const uint4 (&r)[4]) {
    unsigned m2 = bf2max(bf2max(r[0].x, r[0].y), bf2max(r[0].z, r[0].w));
#pragma unroll
    for (int j = 1; j < 4; ++j) m2 = bf2max(m2, bf2max(bf2max(r[j].x, r[j].y), bf2max(r[j].z, r[j].w)));
    return bf2_hmax(m2);
}
// The eight exponentials of one vector, 2^(k l - c), and their packed accumulation by position.
__device__ __forceinline__ void res_exp8(const uint4 &raw, V2 k2, V2 nc2, float (&e)[8], V2 (&acc)[4]) {
    const unsigned w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const V2 x = v2_fma(v2_make(__uint_as_float(w[i] << 16), __uint_as_float(w[i] & 0xffff0000u)), k2, nc2);
        float x0, x1;
        v2_get(x, x0, x1);
        e[2 * i] = ex2(x0);
        e[2 * i + 1] = ex2(x1);
        acc[i] = v2_add(acc[i], v2_make(e[2 * i], e[2 * i + 1]));
    }
}
__device__ __forceinline__ float res_total(const V2 (&acc)[4]) {
    return (v2_sum(acc[0]) + v2_sum(acc[1])) + (v2_sum(acc[2]) + v2_sum(acc[3]));
}

// Inverse-CDF pick over the parts of a row (ascending token ranges), by one warp: lane l holds the
// masses m[0..8) of eight consecutive parts (parts 8l .. 8l+7).  The first part with mass whose
// inclusive prefix exceeds t, else the last part with mass; -1 when nothing has mass.  `base` = the
// mass before the picked part.
__device__ __forceinline__ int res_pick8(const float (&m)[8], float t, int lane, float &base) {
    float ls = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) ls += m[i];
    float incl = ls;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const float up = __shfl_up_sync(kFull, incl, o);
        if (lane >= o) incl += up;
    }
    const float excl = incl - ls;
    const unsigned pos = __ballot_sync(kFull, ls > 0.f);
    const unsigned hit = __ballot_sync(kFull, ls > 0.f && incl > t);
    if (!pos) { base = 0.f; return -1; }
    const int L = hit ? (__ffs(hit) - 1) : (31 - __clz(pos));
    int sel = -1, last = -1;
    float bs = 0.f, lastbs = 0.f, run = excl;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        if (m[i] > 0.f) {
            last = 8 * lane + i;
            lastbs = run;
            if (sel < 0 && run + m[i] > t) { sel = last; bs = run; }
        }
        run += m[i];
    }
    if (sel < 0) { sel = last; bs = lastbs; }
    base = __shfl_sync(kFull, bs, L);
    return __shfl_sync(kFull, sel, L);
}

// One step of a warp-wide inverse-CDF walk: the lanes hold the weights w[8] of 32 consecutive
// vectors (lane order = id order).  Updates (prefix, found, lastpos); all uniform across the warp.
__device__ __forceinline__ void res_scan_step(const float (&w)[8], int vi, int lane, float tt, float &prefix,
                                              int &found, int &lastpos) {
    float lsum = 0.f;
    int lp = -1;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        lsum += w[i];
        if (w[i] > 0.f) lp = vi * 8 + i;
    }
    float incl = lsum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const float up = __shfl_up_sync(kFull, incl, o);
        if (lane >= o) incl += up;
    }
    const float tot = __shfl_sync(kFull, incl, 31);
    const unsigned hit = __ballot_sync(kFull, lsum > 0.f && prefix + incl > tt);
    if (hit) {
        const int L = __ffs(hit) - 1;
        int cand = -1;
        if (lane == L) {
            float acc = prefix + (incl - lsum);
            int lastin = -1;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                acc += w[i];
                if (w[i] > 0.f) {
                    lastin = vi * 8 + i;
                    if (cand < 0 && acc > tt) cand = lastin;
                }
            }
            if (cand < 0) cand = lastin;
        }
        found = __shfl_sync(kFull, cand, L);
    } else {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) lp = max(lp, __shfl_xor_sync(kFull, lp, o));
        lastpos = max(lastpos, lp);
        prefix += tot;
    }
}

// Weight kinds of the residual draws
enum { kDrawP = 0, kDrawSpecHub = 1, kDrawAlg1 = 2 };

// ------------------------------------------------------------------------------------------------
// Verification: SpecHub (Algorithm 3 with the closed form of Section 4 / Appendix B.1), RRS and
// RRSw (Algorithm 1), any subset of the three (MASK) on the same rows.  NB = batches per lane.
// ------------------------------------------------------------------------------------------------
struct ResRaw {   // one batch of a lane: four 16-byte vectors of each row, as loaded
    uint4 p[4], q[4];
};

template <int MASK, int CS>
__global__ void __launch_bounds__(kResThreads, 2) resident_verify_kernel(FusedArgs A, int NB, uint32_t tmem_cols) {
    constexpr int W = CS * kResWarps;   // warps per row
    constexpr bool kSH = (MASK & kMaskSpecHub) != 0, kR = (MASK & kMaskRRS) != 0, kRW = (MASK & kMaskRRSw) != 0;
    constexpr bool kAlg1 = kR || kRW;
    extern __shared__ float4 eq_store[];   // e_q of the batches but the last: [slot][half][thread] as float4
    __shared__ ResShared sh;

    const RowArgs &a = A.r;
    const int me = RowGroup<CS>::rank();
    const long long r = blockIdx.x / CS;
    const int b = static_cast<int>(r / a.nodes), n = static_cast<int>(r % a.nodes);
    // leaf rows belong to lean_leaf_kernel (every CTA of the row leaves, before any barrier)
    if (a.node_kind && a.node_kind[n] == SPECHUB_NODE_LEAF) return;
    res_arrive<CS>();   // [0] "this CTA runs": awaited before the first remote write

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (warp == 0) tmem_alloc(res_smem_addr(&sh.tmem_base), tmem_cols);

    const __nv_bfloat16 *rowp = static_cast<const __nv_bfloat16 *>(a.target) + b * a.stride_seq + n * a.stride_node;
    const __nv_bfloat16 *rowq = static_cast<const __nv_bfloat16 *>(a.draft) + b * a.stride_seq + n * a.stride_node;
    const uint4 *vp = reinterpret_cast<const uint4 *>(rowp), *vq = reinterpret_cast<const uint4 *>(rowq);
    const int V = a.vocab, nvec = V >> 3;
    const int g = me * kResWarps + warp;
    const int seg = (((nvec + W - 1) / W) + 7) & ~7;   // vectors per warp (host: seg <= 128 NB)
    const int lo = min(g * seg, nvec), hi = min(lo + seg, nvec);
    const bool writer = (me == 0 && threadIdx.x == 0);
    const int LB = NB - 1;   // the batch whose e_q stays in registers

    // the draft tokens first: the logits at them are gathered below, behind the first vector loads
    int x1[3], x2[3];
    bool ok1[3], ok2[3];
#pragma unroll
    for (int m = 0; m < 3; ++m) {
        x1[m] = x2[m] = -1;
        if (MASK & (1 << m)) { x1[m] = A.tok[m][2 * r]; x2[m] = A.tok[m][2 * r + 1]; }
    }
    auto load_raw = [&](int bt, ResRaw &R) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int vi = lo + lane + 32 * (4 * bt + j);
            R.p[j] = R.q[j] = make_uint4(0xff80ff80u, 0xff80ff80u, 0xff80ff80u, 0xff80ff80u);   // -inf
            if (vi < hi) { R.p[j] = ld_stream(vp + vi); R.q[j] = ld_stream(vq + vi); }
        }
    };
    ResRaw X, Y;   // two batches in flight: one is consumed while the other arrives
    load_raw(0, X);
    if (NB > 1) load_raw(1, Y);
    else Y = X;

    const float k = kLog2e / temperature_of(a, b);
    const V2 k2 = v2_make(k, k);
    float lp1[3], lp2[3], lq1[3], lq2[3];
#pragma unroll
    for (int m = 0; m < 3; ++m) {
        ok1[m] = ok2[m] = false;
        lp1[m] = lp2[m] = lq1[m] = lq2[m] = 0.f;
        if (MASK & (1 << m)) {
            ok1[m] = x1[m] >= 0 && x1[m] < V; ok2[m] = x2[m] >= 0 && x2[m] < V;
            const int i1 = ok1[m] ? x1[m] : 0, i2 = ok2[m] ? x2[m] : 0;
            if (warp == 0) {   // only warp 0 takes the decisions
                lp1[m] = load_one<__nv_bfloat16>(rowp, i1); lp2[m] = load_one<__nv_bfloat16>(rowp, i2);
            }
            lq1[m] = load_one<__nv_bfloat16>(rowq, i1); lq2[m] = load_one<__nv_bfloat16>(rowq, i2);
        }
    }
    // Exclusion candidates: ids whose term must be left out of a sum of q directly, because
    // subtracting it afterwards cancels on a peaked row.  0, 1: SpecHub's two drafts (one of them is
    // the hub of a well-formed pair; 1 - q(a) = sum over y != a).  2: RRSw's first draft (1 - q(x1)).
    const int cand[3] = {kSH && ok1[0] ? x1[0] : -1, kSH && ok2[0] ? x2[0] : -1, kRW && ok1[2] ? x1[2] : -1};
    int cslot[3];       // slot of this lane that holds the candidate (-1: none)
    bool cwarp[3];      // the candidate lies in this warp's range
#pragma unroll
    for (int c = 0; c < 3; ++c) {
        const int cv = cand[c] >> 3;
        cwarp[c] = cand[c] >= 0 && cv >= lo && cv < hi;
        cslot[c] = (cwarp[c] && ((cv - lo) & 31) == lane) ? (cv - lo) >> 5 : -1;
    }
    // The hub is the first id that attains the maximum draft logit.  For a well-formed pair that
    // logit is the larger of the two drafts' logits, Lc: pass A records the first id equal to Lc.
    float Lc = __int_as_float(0x7fc00000);   // NaN: equal to nothing
    if (kSH) {
        if (ok1[0] && ok2[0]) Lc = fmaxf(lq1[0], lq2[0]);
        else if (ok1[0]) Lc = lq1[0];
        else if (ok2[0]) Lc = lq2[0];
    }

    // ---- storage --------------------------------------------------------------------------------------
    const uint32_t lane_field = static_cast<uint32_t>((warp & 3) * 32) << 16;
    const uint32_t col0 = static_cast<uint32_t>((warp >> 2) * (32 * NB));
    auto eq_ptr = [&](int slot) { return eq_store + (2 * slot) * kResThreads + threadIdx.x; };
    auto store_eq = [&](int slot, const float (&e)[8]) {
        float4 *dst = eq_ptr(slot);
        dst[0] = make_float4(e[0], e[1], e[2], e[3]);
        dst[kResThreads] = make_float4(e[4], e[5], e[6], e[7]);
    };
    auto load_eq_batch = [&](int bt, float (&e)[32]) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float4 *src = eq_ptr(4 * bt + j);
            const float4 u = src[0], w = src[kResThreads];
            e[8 * j + 0] = u.x; e[8 * j + 1] = u.y; e[8 * j + 2] = u.z; e[8 * j + 3] = u.w;
            e[8 * j + 4] = w.x; e[8 * j + 5] = w.y; e[8 * j + 6] = w.z; e[8 * j + 7] = w.w;
        }
    };

    // ---- pass A: the only read of the row pair -------------------------------------------------
    float c_pt = kNoRef, c_qt = kNoRef;   // this thread's exponent references
    V2 pacc[4], qacc[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) pacc[i] = qacc[i] = v2_make(0.f, 0.f);
    float mq_t = neg_inf();
    int ieq_t = kNoIdx;
    uint32_t taddr = 0;
    // Multiply what this thread has stored of batches [0, upto) by the powers of two fp, fq (the
    // whole warp calls it: tensor-memory accesses are warp-wide).
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
    // References of a batch, before its exponentials are taken.
    auto batch_refs = [&](int bt, const ResRaw &R) {
        const float mpb = res_max4(R.p), mqb = res_max4(R.q);
        mq_t = fmaxf(mq_t, mqb);
        if (kSH && mqb == Lc) {   // rare: this batch holds an id with the candidate hub logit
#pragma unroll
            for (int j = 3; j >= 0; --j) {
                float v[8];
                unpack_bf16x8(R.q[j], v);
                const int vi = lo + lane + 32 * (4 * bt + j);
#pragma unroll
                for (int i = 7; i >= 0; --i)
                    if (v[i] == Lc) ieq_t = min(ieq_t, vi * 8 + i);
            }
        }
        const float rpb = res_ref(mpb, k), rqb = res_ref(mqb, k);
        if (bt == 0) {
            c_pt = rpb; c_qt = rqb;
            // first use of tensor memory: the allocation must have been published
            tmem_fence_before();
            __syncthreads();
            tmem_fence_after();
            taddr = sh.tmem_base + lane_field + col0;
        } else {
            // a batch far above the thread's reference moves it (what is stored is rescaled)
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
    };
    // One batch but the last: exponentials to tensor / shared memory, sums.
    auto pass_a_batch = [&](int bt, const ResRaw &R) {
        batch_refs(bt, R);
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
            store_eq(4 * bt + j, e);
        }
    };
    // the next batch but one is requested as soon as a buffer is free
#pragma unroll 1
    for (int bt = 0; bt < LB; bt += 2) {
        pass_a_batch(bt, X);
        if (bt + 2 <= LB) load_raw(bt + 2, X);
        if (bt + 1 < LB) {
            pass_a_batch(bt + 1, Y);
            if (bt + 3 <= LB) load_raw(bt + 3, Y);
        }
    }
    float eqk[32];   // e_q of the last batch stays in registers
    {
        ResRaw L;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            L.p[j] = (LB & 1) ? Y.p[j] : X.p[j];
            L.q[j] = (LB & 1) ? Y.q[j] : X.q[j];
        }
        batch_refs(LB, L);
        const V2 ncp2 = v2_make(-c_pt, -c_pt), ncq2 = v2_make(-c_qt, -c_qt);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            float e[8];
            res_exp8(L.p[j], k2, ncp2, e, pacc);
            tmem_st8(taddr + 8 * (4 * LB + j), e);
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            float e[8];
            res_exp8(L.q[j], k2, ncq2, e, qacc);
#pragma unroll
            for (int i = 0; i < 8; ++i) eqk[8 * j + i] = e[i];
        }
    }
    tmem_wait_st();
    const float sp_t = res_total(pacc), sq_t = res_total(qacc);

    {   // this warp's record
        const float cpw = warp_max(c_pt), cqw = warp_max(c_qt);
        const float fpw = res_pow2(c_pt - cpw), fqw = res_pow2(c_qt - cqw);
        const float spw = warp_sum(__fmul_rn(sp_t, fpw)), sqw = warp_sum(__fmul_rn(sq_t, fqw));
        float sxw[3] = {sqw, sqw, sqw};
#pragma unroll
        for (int c = 0; c < 3; ++c) {
            if (cwarp[c]) {   // warp-uniform: the sum of this warp's e_q without the candidate, term by term
                const int sk = cslot[c], el = cand[c] & 7;
                float s0 = 0.f, s1 = 0.f;
                for (int bt = 0; bt < LB; ++bt) {
                    float e[32];
                    load_eq_batch(bt, e);
#pragma unroll
                    for (int i = 0; i < 32; i += 2) {
                        s0 += (sk == 4 * bt + (i >> 3) && el == (i & 7)) ? 0.f : e[i];
                        s1 += (sk == 4 * bt + (i >> 3) && el == ((i + 1) & 7)) ? 0.f : e[i + 1];
                    }
                }
#pragma unroll
                for (int i = 0; i < 32; i += 2) {
                    s0 += (sk == 4 * LB + (i >> 3) && el == (i & 7)) ? 0.f : eqk[i];
                    s1 += (sk == 4 * LB + (i >> 3) && el == ((i + 1) & 7)) ? 0.f : eqk[i + 1];
                }
                sxw[c] = warp_sum(__fmul_rn(s0 + s1, fqw));
            }
        }
        const float mqw = warp_max(mq_t);
        const int ieqw = kSH ? warp_min_int(ieq_t) : kNoIdx;
        const float4 rec[3] = {make_float4(cpw, spw, cqw, sqw),
                               make_float4(mqw, __int_as_float(ieqw), sxw[0], sxw[1]),
                               make_float4(sxw[2], 0.f, 0.f, 0.f)};
        if (CS > 1) res_wait<CS>();   // [0] every CTA of the row runs
        res_push<CS, 3>(sh.recA[g], rec, lane);
    }
    res_arrive<CS>();
    res_wait<CS>();   // [1] pass-A records exchanged

    // ---- row values and decisions: warp 0 of every CTA, all lanes alike ----------------------------
    const float r1 = a.uniforms[r * 5 + 2], r2 = a.uniforms[r * 5 + 3], ures = a.uniforms[r * 5 + 4];
    float Cp = 0.f, Cq = 0.f, Zp = 0.f, Zq = 0.f, invZp = 0.f, invZq = 0.f, rho = 0.f, mq = 0.f;
    float Zx[3] = {0.f, 0.f, 0.f};
    NodeResult o[3];
    bool live[3] = {false, false, false}, need[3] = {false, false, false}, elsewhere[3] = {false, false, false};
    int hubtok = -1, xs = -1;
    bool pair_xa = false, degenerate = false;
    float c = 0.f, crho = 0.f, qa = 0.f, rest = 0.f, pxs = 0.f, qxs = 0.f, pa = 0.f;
#pragma unroll
    for (int m = 0; m < 3; ++m) {
        o[m].accept_idx = -1; o[m].token = -1; o[m].hub = -1; o[m].status = 0;
        o[m].beta[0] = o[m].beta[1] = 0.f; o[m].rate[0] = o[m].rate[1] = o[m].rate[2] = 0.f;
    }
    auto prob_p = [&](float l) { return prob_of(l, k, Cp, invZp); };
    auto prob_q = [&](float l) { return prob_of(l, k, Cq, invZq); };
    // SpecHub's pair logic once the hub is known; then which methods need the passes
    auto after_hub = [&]() {
        if (kSH && live[0]) {
            o[0].hub = hubtok;
            pair_xa = (x2[0] == hubtok && x1[0] != hubtok);
            const bool pair_ax = (x1[0] == hubtok && x2[0] != hubtok);
            xs = pair_xa ? x1[0] : x2[0];
            if (!(pair_xa || pair_ax) || xs < 0 || xs >= V) {
                o[0].status = SPECHUB_ST_TOKEN_RANGE;
                live[0] = false;
            } else {
                const float own = ex2(__fmaf_rn(mq, k, -Cq));     // the hub's own term on the row's scale
                const float Zrest = pair_xa ? Zx[1] : Zx[0];      // sum over y != a, summed directly
                degenerate = !(Zrest > 0.f);
                c = degenerate ? 0.f : own / Zrest;
                crho = c * rho;
                qa = own * invZq;
                rest = Zrest * invZq;
                pxs = prob_p(pair_xa ? lp1[0] : lp2[0]);
                qxs = prob_q(pair_xa ? lq1[0] : lq2[0]);
                pa = prob_p(pair_xa ? lp2[0] : lp1[0]);
            }
        }
        if (kR && live[1] && !(ok1[1] && ok2[1])) { o[1].status = SPECHUB_ST_TOKEN_RANGE; live[1] = false; }
        if (kRW && live[2] && !(ok1[2] && ok2[2])) { o[2].status = SPECHUB_ST_TOKEN_RANGE; live[2] = false; }
        // No probability asked for: a row whose first test accepts needs no sum at all.
#pragma unroll
        for (int m = 0; m < 3; ++m) {
            need[m] = live[m];
            if (live[m] && !A.out[m].beta && !A.out[m].rate) {
                bool acc1;
                if (m == 0) {
                    acc1 = pair_xa ? accept_test(r1, pxs, qxs, o[0].beta[0], true, o[0].status)
                                   : accept_test(r1, fmaxf(__fsub_rn(pxs, qxs), 0.f), c * qxs, o[0].beta[0], true,
                                                 o[0].status);
                    if (acc1) {
                        o[0].accept_idx = pair_xa ? 0 : 1;
                        o[0].token = xs;
                        if (degenerate) o[0].status |= SPECHUB_ST_DEGENERATE_Q;
                    }
                } else {
                    acc1 = accept_test(r1, prob_p(lp1[m]), prob_q(lq1[m]), o[m].beta[0], true, o[m].status);
                    if (acc1) { o[m].accept_idx = 0; o[m].token = x1[m]; }
                }
                if (acc1) need[m] = false;
                else o[m].status = 0;   // the full path sets the flags again
            }
        }
        if (lane == 0) {
            sh.bc[2] = rho; sh.bc[3] = crho;
            sh.bi[0] = hubtok;
            sh.bi[1] = (need[0] ? 1 : 0) | (need[1] ? 2 : 0) | (need[2] ? 4 : 0);
            sh.bi[2] = (kSH && need[0]) ? (pair_xa ? 1 : 0) : -1;   // which exclusion candidate is the hub
        }
    };
    if (warp == 0) {
        const int g0 = 2 * lane, g1 = 2 * lane + 1;
        float c0 = kNoRef, s0 = 0.f, d0 = kNoRef, q0 = 0.f, m0 = neg_inf(), y0[3] = {0.f, 0.f, 0.f};
        float c1 = kNoRef, s1 = 0.f, d1 = kNoRef, q1 = 0.f, m1 = neg_inf(), y1[3] = {0.f, 0.f, 0.f};
        int i0 = kNoIdx, i1 = kNoIdx;
        if (g0 < W) {
            const float *rc = sh.recA[g0];
            c0 = rc[0]; s0 = rc[1]; d0 = rc[2]; q0 = rc[3]; m0 = rc[4]; i0 = __float_as_int(rc[5]);
            y0[0] = rc[6]; y0[1] = rc[7]; y0[2] = rc[8];
        }
        if (g1 < W) {
            const float *rc = sh.recA[g1];
            c1 = rc[0]; s1 = rc[1]; d1 = rc[2]; q1 = rc[3]; m1 = rc[4]; i1 = __float_as_int(rc[5]);
            y1[0] = rc[6]; y1[1] = rc[7]; y1[2] = rc[8];
        }
        Cp = warp_max(fmaxf(c0, c1));
        Cq = warp_max(fmaxf(d0, d1));
        const float f0 = res_pow2(c0 - Cp), f1 = res_pow2(c1 - Cp), h0 = res_pow2(d0 - Cq), h1 = res_pow2(d1 - Cq);
        // pinned roundings: the target and the draft row go through the same arithmetic, so
        // identical rows give identical normalisers
        Zp = warp_sum(__fadd_rn(__fmul_rn(s0, f0), __fmul_rn(s1, f1)));
        Zq = warp_sum(__fadd_rn(__fmul_rn(q0, h0), __fmul_rn(q1, h1)));
#pragma unroll
        for (int cnd = 0; cnd < 3; ++cnd) Zx[cnd] = warp_sum(__fadd_rn(__fmul_rn(y0[cnd], h0), __fmul_rn(y1[cnd], h1)));
        mq = warp_max(fmaxf(m0, m1));
        const int ieq = warp_min_int(min(i0, i1));
        invZp = 1.f / Zp; invZq = 1.f / Zq;
        rho = __fdiv_rn(Zp, Zq);
        const bool bad = !finite_pos(Zp) || !finite_pos(Zq) || !(mq > neg_inf()) || !(mq < -neg_inf());
#pragma unroll
        for (int m = 0; m < 3; ++m) {
            live[m] = (MASK & (1 << m)) != 0;
            if (live[m] && bad) { o[m].status = SPECHUB_ST_NONFINITE; live[m] = false; }
        }
        const bool cold = kSH && live[0] && !(mq == Lc);
        if (lane == 0) {
            sh.bc[0] = Cp; sh.bc[1] = Cq; sh.bc[4] = mq;
            sh.bi[3] = cold ? 1 : 0;
        }
        if (!cold) {
            hubtok = ieq;
            after_hub();
        }
    }
    __syncthreads();
    if (kSH && sh.bi[3]) {
        // The pair does not hold the hub (a malformed pair).  The hub is still reported: the first
        // id of the row maximum, found by a rescan of the draft row (a cold path that every CTA of
        // the row takes together).
        const float mrow = sh.bc[4];
        int fi = kNoIdx;
        for (int vi = lo + lane; vi < hi; vi += 32) {
            float v[8];
            unpack_bf16x8(vq[vi], v);
#pragma unroll
            for (int i = 7; i >= 0; --i)
                if (v[i] == mrow) fi = min(fi, vi * 8 + i);
        }
        fi = warp_min_int(fi);
        if (lane < CS) {
            int *dst = &sh.recH[g];
            if (CS > 1) dst = cooperative_groups::this_cluster().map_shared_rank(dst, lane);
            *dst = fi;
        }
        res_arrive<CS>();
        res_wait<CS>();
        if (warp == 0) {
            const int g0 = 2 * lane, g1 = 2 * lane + 1;
            hubtok = warp_min_int(min(g0 < W ? sh.recH[g0] : kNoIdx, g1 < W ? sh.recH[g1] : kNoIdx));
            after_hub();
        }
        __syncthreads();
    }
    // what every thread needs for the passes over its stored exponentials
    Cp = sh.bc[0]; Cq = sh.bc[1];
    const float rho_b = sh.bc[2], crho_b = sh.bc[3];
    const int needmask = sh.bi[1];
    const int hubc = sh.bi[2];
    const bool needB = needmask != 0;
    const bool needC = (kR && (needmask & 2)) || (kRW && (needmask & 4));

    // This thread's scales: E = e * 2^(c_t - C).  The passes work on the thread's own scale,
    //   d' = e_p - rho' e_q,  rho' = rho 2^(nq - np),  and multiply their sums by F = 2^np;
    // references far below the row's are first brought to it, so that rho' stays in range.
    float np = (c_pt == kNoRef) ? 0.f : c_pt - Cp, nq = (c_qt == kNoRef) ? 0.f : c_qt - Cq;
    if (needB) {
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
    const float rho_t = __fmul_rn(rho_b, sc), crho_t = __fmul_rn(crho_b, sc);
    const V2 nrq2 = v2_make(-rho_t, -rho_t), nsq2 = v2_make(-crho_t, -crho_t);
    // the slot of this lane that holds the hub (-1: none)
    const int hub_slot = (kSH && hubc >= 0) ? cslot[hubc] : -1;
    const bool hub_warp = kSH && hubc >= 0 && cwarp[hubc];
    const int hub_el = (kSH && hubc >= 0) ? (cand[hubc] & 7) : 0;
    // a per-batch partial of this warp, to every CTA of the row
    auto push_scalar = [&](float *slot, float v) {
        if (lane < CS) {
            float *dst = slot;
            if (CS > 1) dst = cooperative_groups::this_cluster().map_shared_rank(slot, lane);
            *dst = v;
        }
    };

    // ---- pass B over the stored exponentials: S1, S2, R (ids != a) and A1 (all ids) -----------------
    //   d = e_p - rho' e_q   (Z_p (p - q) on the thread's scale),   t = max(d, 0) - c rho' e_q;
    //   S1 += max(-d, 0) = max(d, 0) - d,  S2 += max(-t, 0) = max(t, 0) - t,  R += max(t, 0),  A1 += max(d, 0).
    // R is also kept per batch: the residual draw then walks one batch of one warp.
    if (needB) {
        V2 s1 = v2_make(0.f, 0.f), s2 = s1, a1 = s1;
        float Rw = 0.f;
        auto pass_b_batch = [&](int bt, const float (&ep)[32], const float (&eq)[32]) {
            const bool special = hub_warp && (hub_slot >> 2) == bt && hub_slot >= 0;
            const bool any_special = hub_warp && __any_sync(kFull, special);
            V2 rr = v2_make(0.f, 0.f);
            if (!any_special) {
#pragma unroll
                for (int i = 0; i < 32; i += 2) {
                    const V2 e_q = v2_make(eq[i], eq[i + 1]);
                    const V2 d = v2_fma(nrq2, e_q, v2_make(ep[i], ep[i + 1]));
                    const V2 m = v2_max0(d);
                    if (kAlg1) a1 = v2_add(a1, m);
                    if (kSH) {
                        const V2 t = v2_fma(nsq2, e_q, m);
                        const V2 w = v2_max0(t);
                        s1 = v2_add(s1, v2_sub(m, d));
                        s2 = v2_add(s2, v2_sub(w, t));
                        rr = v2_add(rr, w);
                    }
                }
            } else {   // the batch of one lane of this warp holds the hub: its pair is not part of the sums over y != a
#pragma unroll
                for (int i = 0; i < 32; i += 2) {
                    const V2 e_q = v2_make(eq[i], eq[i + 1]);
                    const V2 d = v2_fma(nrq2, e_q, v2_make(ep[i], ep[i + 1]));
                    const V2 m = v2_max0(d);
                    if (kAlg1) a1 = v2_add(a1, m);
                    if (kSH) {
                        const V2 t = v2_fma(nsq2, e_q, m);
                        const V2 w = v2_max0(t);
                        float u0, u1, v0, v1, w0, w1;
                        v2_get(v2_sub(m, d), u0, u1);
                        v2_get(v2_sub(w, t), v0, v1);
                        v2_get(w, w0, w1);
                        const bool hv = special && (hub_slot & 3) == (i >> 3);
                        if (hv && hub_el == (i & 7)) { u0 = 0.f; v0 = 0.f; w0 = 0.f; }
                        if (hv && hub_el == ((i + 1) & 7)) { u1 = 0.f; v1 = 0.f; w1 = 0.f; }
                        s1 = v2_add(s1, v2_make(u0, u1));
                        s2 = v2_add(s2, v2_make(v0, v1));
                        rr = v2_add(rr, v2_make(w0, w1));
                    }
                }
            }
            if (kSH) {
                const float rb = warp_sum(mul_ftz(v2_sum(rr), F));
                push_scalar(&sh.recB[g][4 + bt], rb);
                Rw += rb;
            }
        };
#pragma unroll 1
        for (int bt = 0; bt < LB; ++bt) {
            float ep[32], eq[32];
            tmem_ld32(taddr + 32 * bt, ep);
            load_eq_batch(bt, eq);
            pass_b_batch(bt, ep, eq);
        }
        {
            float ep[32];
            tmem_ld32(taddr + 32 * LB, ep);
            pass_b_batch(LB, ep, eqk);
        }
        const float4 rec[1] = {make_float4(kSH ? warp_sum(mul_ftz(v2_sum(s1), F)) : 0.f,
                                           kSH ? warp_sum(mul_ftz(v2_sum(s2), F)) : 0.f, Rw,
                                           kAlg1 ? warp_sum(mul_ftz(v2_sum(a1), F)) : 0.f)};
        res_push<CS, 1>(sh.recB[g], rec, lane);
        res_arrive<CS>();
        res_wait<CS>();   // [2] pass-B records exchanged
    }
    // The masses of the (warp, batch) parts 8 lane .. 8 lane + 7 of a row, in id order (NB <= 4 per warp).
    auto parts_of = [&](const float *rec0, int stride, int off, float (&m)[8]) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int gg = 2 * lane + (i >> 2), bt = i & 3;
            m[i] = (gg < W && bt < NB) ? rec0[gg * stride + off + bt] : 0.f;
        }
    };

    // ---- warp 0: SpecHub's tests (Algorithm 3); scalars of Algorithm 1's second stage ---------------
    float A1 = 0.f, A1g[3] = {0.f, 0.f, 0.f}, A1grho[3] = {0.f, 0.f, 0.f};
    bool q1_zero = false;
    if (warp == 0) {
        float tot[4] = {0.f, 0.f, 0.f, 0.f};
        int selB = -1;
        float ttB = 0.f;
        if (needB) {
            const int g0 = 2 * lane, g1 = 2 * lane + 1;
            float x0[4] = {0.f, 0.f, 0.f, 0.f}, y0[4] = {0.f, 0.f, 0.f, 0.f};
            if (g0 < W) { x0[0] = sh.recB[g0][0]; x0[1] = sh.recB[g0][1]; x0[2] = sh.recB[g0][2]; x0[3] = sh.recB[g0][3]; }
            if (g1 < W) { y0[0] = sh.recB[g1][0]; y0[1] = sh.recB[g1][1]; y0[2] = sh.recB[g1][2]; y0[3] = sh.recB[g1][3]; }
#pragma unroll
            for (int i = 0; i < 4; ++i) tot[i] = warp_sum(x0[i] + y0[i]);
            if (kSH) {
                float m[8], base = 0.f;
                parts_of(&sh.recB[0][0], 8, 4, m);
                selB = res_pick8(m, ures * tot[2], lane, base);
                ttB = ures * tot[2] - base;
            }
        }
        int drawkind[3] = {-1, -1, -1};   // what each method still has to draw (-1: nothing)
        if (kSH && need[0]) {
            NodeResult &os = o[0];
            const float S1 = tot[0] * invZp, Rraw = tot[2];
            const float S2 = degenerate ? qa : tot[1] * invZp;
            const float R = Rraw * invZp;
            const float hub_left = fmaxf(pa - S2, 0.f);
            os.rate[0] = fmaxf(rest - S1, 0.f) + fminf(pa, S2);
            os.rate[1] = (degenerate ? 0.f : fmaxf(qa - S2, 0.f)) + fminf(hub_left, S1);
            os.rate[2] = R;
            if (degenerate) os.status |= SPECHUB_ST_DEGENERATE_Q;
            bool acc1, acc2;
            if (pair_xa) {
                acc1 = accept_test(r1, pxs, qxs, os.beta[0], true, os.status);
                if (acc1) { os.accept_idx = 0; os.token = xs; }
                acc2 = accept_test(r2, hub_left, S1, os.beta[1], !acc1, os.status);
                if (!acc1 && acc2) { os.accept_idx = 1; os.token = hubtok; }
            } else {
                acc1 = accept_test(r1, fmaxf(__fsub_rn(pxs, qxs), 0.f), c * qxs, os.beta[0], true, os.status);
                if (acc1) { os.accept_idx = 1; os.token = xs; }
                acc2 = accept_test(r2, pa, S2, os.beta[1], !acc1, os.status);
                if (!acc1 && acc2) { os.accept_idx = 0; os.token = hubtok; }
            }
            if (!(acc1 || acc2)) {
                os.accept_idx = -1;
                elsewhere[0] = true;
                if (!(Rraw > 0.f) || selB < 0) { os.status |= SPECHUB_ST_ZERO_RESIDUAL; drawkind[0] = kDrawP; }
                else drawkind[0] = kDrawSpecHub;
            }
        }
        if (kAlg1) {
            A1 = tot[3] * invZp;
            const float den = Zx[2] * invZq;   // 1 - q(x1) of RRSw, summed directly
            q1_zero = kRW && !(den > 0.f);
            const float gq[3] = {0.f, 1.f, q1_zero ? 0.f : 1.f / den};   // q1 = gq * q off x1
#pragma unroll
            for (int m = 1; m < 3; ++m) { A1g[m] = A1 * gq[m]; A1grho[m] = A1g[m] * rho; }
        }
        if (lane == 0) {
            sh.bi[4] = drawkind[0]; sh.bi[5] = selB; sh.bc[5] = ttB;
            sh.bc[6] = A1grho[1]; sh.bc[7] = A1grho[2];
        }
    }
    __syncthreads();

    // ---- pass C (Algorithm 1): mass of the residual after two rejections ---------------------------
    //   on the thread's scale:  t = max(d, 0) - (A1 g rho') e_q,  W2 += max(t, 0)
    const float sr_t = kAlg1 ? __fmul_rn(sh.bc[6], sc) : 0.f, sw_t = kAlg1 ? __fmul_rn(sh.bc[7], sc) : 0.f;
    const int x1w_slot = kRW ? cslot[2] : -1;
    const bool x1w_warp = kRW && cwarp[2];
    const int x1w_el = cand[2] & 7;
    if (kAlg1 && needC) {
        const V2 nsr2 = v2_make(-sr_t, -sr_t), nsw2 = v2_make(-sw_t, -sw_t);
        float Wr = 0.f, Ww = 0.f;
        auto pass_c_batch = [&](int bt, const float (&ep)[32], const float (&eq)[32]) {
            const bool special = x1w_warp && x1w_slot >= 0 && (x1w_slot >> 2) == bt;
            const bool any_special = x1w_warp && __any_sync(kFull, special);
            V2 wr = v2_make(0.f, 0.f), ww = wr;
#pragma unroll
            for (int i = 0; i < 32; i += 2) {
                const V2 e_q = v2_make(eq[i], eq[i + 1]);
                const V2 m = v2_max0(v2_fma(nrq2, e_q, v2_make(ep[i], ep[i + 1])));
                if (kR) wr = v2_add(wr, v2_max0(v2_fma(nsr2, e_q, m)));
                if (kRW) {
                    V2 s = nsw2;
                    if (any_special) {   // q1(x1) = 0
                        const bool xv = special && (x1w_slot & 3) == (i >> 3);
                        s = v2_make((xv && x1w_el == (i & 7)) ? 0.f : -sw_t, (xv && x1w_el == ((i + 1) & 7)) ? 0.f : -sw_t);
                    }
                    ww = v2_add(ww, v2_max0(v2_fma(s, e_q, m)));
                }
            }
            if (kR) {
                const float v = warp_sum(mul_ftz(v2_sum(wr), F));
                push_scalar(&sh.recC[g][4 + bt], v);
                Wr += v;
            }
            if (kRW) {
                const float v = warp_sum(mul_ftz(v2_sum(ww), F));
                push_scalar(&sh.recC[g][8 + bt], v);
                Ww += v;
            }
        };
#pragma unroll 1
        for (int bt = 0; bt < LB; ++bt) {
            float ep[32], eq[32];
            tmem_ld32(taddr + 32 * bt, ep);
            load_eq_batch(bt, eq);
            pass_c_batch(bt, ep, eq);
        }
        {
            float ep[32];
            tmem_ld32(taddr + 32 * LB, ep);
            pass_c_batch(LB, ep, eqk);
        }
        const float4 rec[1] = {make_float4(Wr, Ww, 0.f, 0.f)};
        res_push<CS, 1>(sh.recC[g], rec, lane);
        res_arrive<CS>();
        res_wait<CS>();   // [3] pass-C records exchanged
    }
    // ---- warp 0: the tests of Algorithm 1 -----------------------------------------------------------
    if (kAlg1) {
        if (warp == 0) {
            float W2raw[3] = {0.f, 0.f, 0.f}, ttC[3] = {0.f, 0.f, 0.f};
            int selC[3] = {-1, -1, -1};
            if (needC) {
                const int g0 = 2 * lane, g1 = 2 * lane + 1;
#pragma unroll
                for (int i = 0; i < 2; ++i) {
                    if (!((i == 0 && kR) || (i == 1 && kRW))) continue;
                    const float tt = warp_sum((g0 < W ? sh.recC[g0][i] : 0.f) + (g1 < W ? sh.recC[g1][i] : 0.f));
                    float m[8], base = 0.f;
                    parts_of(&sh.recC[0][0], 12, 4 + 4 * i, m);
                    selC[1 + i] = res_pick8(m, ures * tt, lane, base);
                    W2raw[1 + i] = tt;
                    ttC[1 + i] = ures * tt - base;
                }
            }
#pragma unroll
            for (int m = 1; m < 3; ++m) {
                int dk = -1;
                if ((MASK & (1 << m)) && need[m]) {
                    NodeResult &om = o[m];
                    const bool wo = (m == 2);
                    const float W2 = W2raw[m] * invZp;
                    om.rate[0] = fmaxf(1.f - A1, 0.f);
                    om.rate[1] = fmaxf(A1 - W2, 0.f);
                    om.rate[2] = W2;
                    const float px1 = prob_p(lp1[m]), qx1 = prob_q(lq1[m]), px2 = prob_p(lp2[m]), qx2 = prob_q(lq2[m]);
                    const bool acc1 = accept_test(r1, px1, qx1, om.beta[0], true, om.status);
                    if (acc1) { om.accept_idx = 0; om.token = x1[m]; }
                    if (wo && !acc1 && q1_zero) om.status |= SPECHUB_ST_DEGENERATE_Q;
                    bool acc2 = false;
                    if (A1 > 0.f) {
                        const float q1x2 = (wo && x2[m] == x1[m]) ? 0.f : A1g[m] * qx2;
                        acc2 = accept_test(r2, fmaxf(__fsub_rn(px2, qx2), 0.f), q1x2, om.beta[1], !acc1, om.status);
                    }
                    if (!acc1 && acc2) { om.accept_idx = 1; om.token = x2[m]; }
                    if (!(acc1 || acc2)) {
                        om.accept_idx = -1;
                        elsewhere[m] = true;
                        if (!(A1 > 0.f) || !(W2raw[m] > 0.f) || selC[m] < 0) { om.status |= SPECHUB_ST_ZERO_RESIDUAL; dk = kDrawP; }
                        else dk = kDrawAlg1;
                    }
                }
                if (lane == 0) { sh.bi[4 + 2 * m] = dk; sh.bi[5 + 2 * m] = selC[m]; sh.bc[5 + 3 * m] = ttC[m]; }
            }
        }
        __syncthreads();
    }
    if (writer) {
#pragma unroll
        for (int m = 0; m < 3; ++m)
            if (MASK & (1 << m)) write_node3(A.out[m], r, o[m], elsewhere[m]);
    }

    // ---- residual draws: the warp whose range holds the target walks one batch of its stored exponentials
    // kind: what the weights are.  nscale: -(second-stage scale) on the thread's scale; xex: id whose second-
    // stage scale is 0 (RRSw's first draft), hubx: id without weight (the hub).  part = 4 * warp + batch.
    auto draw = [&](int kind, int part, float tt, float nscale, int xex, int hubx, int32_t *token_out) {
        if (kind == kDrawP) {   // residual mass 0 on a rejection: the token is a draw from p (whole warp ranges)
            if (warp == 0) {
                const int g0 = 2 * lane, g1 = 2 * lane + 1;
                float m[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
                if (g0 < W) m[0] = __fmul_rn(sh.recA[g0][1], res_pow2(sh.recA[g0][0] - Cp));
                if (g1 < W) m[4] = __fmul_rn(sh.recA[g1][1], res_pow2(sh.recA[g1][0] - Cp));
                const float Ztot = warp_sum(m[0] + m[4]);
                float base;
                const int s = res_pick8(m, ures * Ztot, lane, base);
                if (lane == 0) { sh.bi[10] = s; sh.bc[20] = ures * Ztot - base; }
            }
            __syncthreads();
            part = sh.bi[10] < 0 ? -1 : (sh.bi[10] & ~3);   // batch 0 of the picked warp; the walk goes on
            tt = sh.bc[20];
            __syncthreads();
        }
        if (part < 0 || (part >> 2) != g) return;
        const int bt0 = part & 3, bt1 = (kind == kDrawP) ? NB : bt0 + 1;
        float prefix = 0.f;
        int found = -1, lastpos = -1;
        const V2 ns2 = v2_make(nscale, nscale);
        auto walk = [&](int bt, const float (&ep)[32], const float (&eq)[32]) {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                if (found < 0) {
                    const int vi = lo + lane + 32 * (4 * bt + j);
                    float w[8];
#pragma unroll
                    for (int i = 0; i < 8; i += 2) {
                        float w0, w1;
                        if (kind == kDrawP) {
                            w0 = ep[8 * j + i]; w1 = ep[8 * j + i + 1];
                        } else {
                            const V2 e_q = v2_make(eq[8 * j + i], eq[8 * j + i + 1]);
                            const V2 m = v2_max0(v2_fma(nrq2, e_q, v2_make(ep[8 * j + i], ep[8 * j + i + 1])));
                            V2 s = ns2;
                            if (xex >= 0) s = v2_make(vi * 8 + i == xex ? 0.f : nscale, vi * 8 + i + 1 == xex ? 0.f : nscale);
                            v2_get(v2_max0(v2_fma(s, e_q, m)), w0, w1);
                            if (vi * 8 + i == hubx) w0 = 0.f;
                            if (vi * 8 + i + 1 == hubx) w1 = 0.f;
                        }
                        w[i] = mul_ftz(w0, F); w[i + 1] = mul_ftz(w1, F);
                    }
                    res_scan_step(w, vi, lane, tt, prefix, found, lastpos);
                }
            }
        };
#pragma unroll 1
        for (int bt = bt0; bt < bt1 && bt < LB && found < 0; ++bt) {
            float ep[32], eq[32];
            tmem_ld32(taddr + 32 * bt, ep);
            load_eq_batch(bt, eq);
            walk(bt, ep, eq);
        }
        if (found < 0 && bt1 > LB) {
            float ep[32];
            tmem_ld32(taddr + 32 * LB, ep);
            walk(LB, ep, eqk);
        }
        if (found < 0) found = lastpos;
        if (lane == 0) *token_out = found;
    };
    if (kSH && sh.bi[4] >= 0) draw(sh.bi[4], sh.bi[5], sh.bc[5], -crho_t, -1, sh.bi[0], &A.out[0].token[r]);
    if (kR && sh.bi[6] >= 0) draw(sh.bi[6], sh.bi[7], sh.bc[8], -sr_t, -1, -1, &A.out[1].token[r]);
    if (kRW && sh.bi[8] >= 0) draw(sh.bi[8], sh.bi[9], sh.bc[11], -sw_t, x1[2], -1, &A.out[2].token[r]);

    // release the tensor memory: every warp is done with it
    tmem_fence_before();
    __syncthreads();
    if (warp == 0) {
        tmem_fence_after();
        tmem_dealloc(sh.tmem_base, tmem_cols);
    }
}

}  // namespace spechub
