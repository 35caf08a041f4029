// Lean streaming kernels for bf16 rows with 16-byte aligned starts and V % 8 == 0
// (the shapes of the large-vocabulary workloads).  A (sequence, node) row is
// worked on by a cluster of CS CTAs (CS = 1, 2 or 4), each owning a contiguous
// slice of the vocabulary; several CTAs of different rows share an SM so that one
// row's reductions overlap another row's streaming.  Splitting a row keeps the
// number of rows in flight -- and with it the bytes between a row's first and
// second read -- small enough that pass B hits L2 instead of HBM, without giving
// up the thread count that hides latency.  The CTAs of a row meet at two or three
// hardware cluster barriers and read each other's few partial results through
// distributed shared memory.  Compared with the general kernels in
// spechub_stream.cuh the inner loops are branch-free and carry no index
// bookkeeping:
//
//   pass A  per 16-byte vector: a packed bf16 max tree (4 ops), 8 x (unpack, FMA,
//           ex2, add).  The exponent reference c of a thread is the maximum of the
//           first vector it reads, not a running maximum: 2^(k l - c) is exact in
//           floating point for any c within 2^+-100 of the true one, so c only
//           moves if a partial sum leaves that range (checked once per vector).
//   argmax  only threads whose maximum equals the row maximum rescan their own
//           elements (L2 hits) for the first index; the one owner also re-sums its
//           elements without the maximum, so 1 - q(a) is a direct sum.
//   pass B  re-reads the row (L2), recomputes the probabilities and the transport
//           sums; the hub's pair is removed in the one iteration that holds it.
//
// The special-function pipe (16 ex2/clk/SM) bounds both passes: 4 ex2 per
// vocabulary pair per row.
#pragma once

#include <cooperative_groups.h>

#include "spechub.h"
#include "spechub_common.cuh"
#include "spechub_stream.cuh"
#include "spechub_ring.cuh"

namespace spechub {
namespace cg = cooperative_groups;

constexpr int kLeanMaxWarps = 32;
constexpr int kLeanCk = 8;        // checkpoints per warp in the draft step's pass A
constexpr float kHuge = 1.0e30f;  // ~2^100: partial sums beyond this move the reference

struct LeanShared {
    float wml[2][kLeanMaxWarps];    // per-warp max logit (0 target, 1 draft)
    float wmass[2][kLeanMaxWarps];  // per-warp sum of exponentials on the row's scale, argmax left out
    int cand[2];                    // lowest index attaining the row maximum
    float acc[8][kLeanMaxWarps];
    float mass[kLeanMaxWarps];
    float part[1024];  // sampler: per-thread block sums of the selected warp range
    float tt2;
    int blk;
    int tok;
    // what this CTA tells the other CTAs of its row (read through distributed shared memory)
    float x_ml[2], x_sx[2];  // slice (max logit, sum without the slice argmax), 0 target / 1 draft
    int x_idx[2];            // slice argmax
    float x_sum[4];          // pass-B / pass-C sums of the slice
    float x_mass;            // slice mass for a draw from q without a given token
    int x_tok;               // a token drawn by this CTA
    int stat_ok;             // verification from draft statistics: the row's record was accepted
};
// draft step and leaf rows: also the checkpoint sums of pass A (per warp, every CK lane-iterations), their
// exponent references, and the masses of those sub-blocks on the row's scale
struct LeanCkShared : LeanShared {
    float cks[kLeanMaxWarps][kLeanCk], ckc[kLeanMaxWarps][kLeanCk];
    float ckm[kLeanMaxWarps * kLeanCk];
};

// The CTAs of one row.  CS = 1 compiles to no cluster instruction at all.
template <int CS>
struct RowGroup {
    __device__ __forceinline__ static int rank() {
        if (CS == 1) return 0;
        return static_cast<int>(cg::this_cluster().block_rank());
    }
    __device__ __forceinline__ static void sync() {
        if (CS == 1) __syncthreads();
        else cg::this_cluster().sync();
    }
    template <class T>
    __device__ __forceinline__ static const T *peer(const T *local, int r) {
        if (CS == 1) return local;
        return cg::this_cluster().map_shared_rank(local, r);
    }
};

__device__ __forceinline__ unsigned bf2max(unsigned a, unsigned b) {
    unsigned d;
    asm("max.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
__device__ __forceinline__ float bf2_hmax(unsigned m2) {
    return fmaxf(__uint_as_float(m2 << 16), __uint_as_float(m2 & 0xffff0000u));
}
__device__ __forceinline__ void unpack_bf16x8(const uint4 &v, float (&o)[8]) {
    o[0] = __uint_as_float(v.x << 16); o[1] = __uint_as_float(v.x & 0xffff0000u);
    o[2] = __uint_as_float(v.y << 16); o[3] = __uint_as_float(v.y & 0xffff0000u);
    o[4] = __uint_as_float(v.z << 16); o[5] = __uint_as_float(v.z & 0xffff0000u);
    o[6] = __uint_as_float(v.w << 16); o[7] = __uint_as_float(v.w & 0xffff0000u);
}

// Two fp32 lanes per instruction (fma / add / sub .f32x2): half the issue slots of the scalar forms,
// the same roundings (round to nearest, subnormals kept), so results do not depend on which form is used.
struct F2 {
    unsigned long long v;
};
__device__ __forceinline__ F2 f2_make(float lo, float hi) {
    F2 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r.v) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void f2_get(F2 a, float &lo, float &hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(a.v));
}
__device__ __forceinline__ F2 f2_fma(F2 a, F2 b, F2 c) {
    F2 d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d.v) : "l"(a.v), "l"(b.v), "l"(c.v));
    return d;
}
__device__ __forceinline__ F2 f2_add(F2 a, F2 b) {
    F2 d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d.v) : "l"(a.v), "l"(b.v));
    return d;
}
__device__ __forceinline__ F2 f2_sub(F2 a, F2 b) {
    F2 d;
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(d.v) : "l"(a.v), "l"(b.v));
    return d;
}
__device__ __forceinline__ F2 f2_max0(F2 a) {
    float lo, hi;
    f2_get(a, lo, hi);
    return f2_make(fmaxf(lo, 0.f), fmaxf(hi, 0.f));
}
__device__ __forceinline__ float f2_sum(F2 a) {
    float lo, hi;
    f2_get(a, lo, hi);
    return lo + hi;
}
// the exponentials 2^(k l - c) of one 32-bit word (two bf16 logits), as a pair
__device__ __forceinline__ F2 f2_exp_word(unsigned w, F2 k2, F2 nc2) {
    const F2 x = f2_fma(f2_make(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u)), k2, nc2);
    float x0, x1;
    f2_get(x, x0, x1);
    return f2_make(ex2(x0), ex2(x1));
}

// a 16-byte load with an L2 eviction policy (createpolicy)
__device__ __forceinline__ uint4 ld_l2_hint(const uint4 *p, uint64_t pol) {
    uint4 v;
    asm volatile("ld.global.L2::cache_hint.v4.u32 {%0, %1, %2, %3}, [%4], %5;"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p), "l"(pol));
    return v;
}

struct LeanAcc {  // one thread's pass-A state for one row
    unsigned m2;  // packed running maximum
    float c;      // exponent reference (k * some logit of this thread, or 0)
    float s;      // sum of 2^(k l - c)
};

__device__ __forceinline__ void lean_push(LeanAcc &st, const uint4 &raw, float k) {
    const unsigned vm = bf2max(bf2max(raw.x, raw.y), bf2max(raw.z, raw.w));
    st.m2 = bf2max(st.m2, vm);
    const F2 k2 = f2_make(k, k);
    F2 nc2 = f2_make(-st.c, -st.c);
    // the vector's sum, two lanes at a time: (e0 + e2) + (e4 + e6) and (e1 + e3) + (e5 + e7)
    float a = f2_sum(f2_add(f2_add(f2_exp_word(raw.x, k2, nc2), f2_exp_word(raw.y, k2, nc2)),
                            f2_add(f2_exp_word(raw.z, k2, nc2), f2_exp_word(raw.w, k2, nc2))));
    if (!(a < kHuge)) {  // out of range (or NaN / +inf input): move the reference to this vector's max
        const float vmax = bf2_hmax(vm);
        const float cn = shift_of(vmax, k);
        st.s *= ex2(st.c - cn);
        st.c = cn;
        nc2 = f2_make(-st.c, -st.c);
        a = f2_sum(f2_add(f2_add(f2_exp_word(raw.x, k2, nc2), f2_exp_word(raw.y, k2, nc2)),
                          f2_add(f2_exp_word(raw.z, k2, nc2), f2_exp_word(raw.w, k2, nc2))));
    }
    st.s += a;
}

// Pass A over this warp's range of one or two rows.
// AHEAD: the next vector pair is requested before the current one is consumed (measured per
// method: it pays for RRS, 1.92 -> 1.82 ms on V = 128256, and costs SpecHub 2 %).
template <bool BOTH, bool AHEAD = false>
__device__ __forceinline__ void lean_pass_a(const uint4 *rp, const uint4 *rq, int lo, int hi, int lane,
                                            float k, LeanAcc &P, LeanAcc &Q) {
    P.m2 = 0xff80ff80u; P.s = 0.f; P.c = 0.f;
    Q.m2 = 0xff80ff80u; Q.s = 0.f; Q.c = 0.f;
    int vi = lo + lane;
    // the reference comes from the thread's first vector that holds a finite logit
    for (int vr = vi; vr < hi; vr += 32) {
        const uint4 a = rp[vr];
        const float m0 = bf2_hmax(bf2max(bf2max(a.x, a.y), bf2max(a.z, a.w)));
        if (m0 > neg_inf()) { P.c = shift_of(m0, k); break; }
    }
    if (BOTH) {
        for (int vr = vi; vr < hi; vr += 32) {
            const uint4 b = rq[vr];
            const float m0 = bf2_hmax(bf2max(bf2max(b.x, b.y), bf2max(b.z, b.w)));
            if (m0 > neg_inf()) { Q.c = shift_of(m0, k); break; }
        }
    }
    if (BOTH && AHEAD) {
        uint4 na = make_uint4(0, 0, 0, 0), nb = na;
        if (vi < hi) { na = rp[vi]; nb = rq[vi]; }
#pragma unroll 1
        for (; vi < hi; vi += 32) {
            const uint4 a = na, b = nb;
            if (vi + 32 < hi) { na = rp[vi + 32]; nb = rq[vi + 32]; }
            lean_push(P, a, k);
            lean_push(Q, b, k);
        }
    } else {
#pragma unroll 2
        for (; vi < hi; vi += 32) {
            const uint4 a = rp[vi];
            uint4 b;
            if (BOTH) b = rq[vi];
            lean_push(P, a, k);
            if (BOTH) lean_push(Q, b, k);
        }
    }
}

// Pass A over one row with four vectors per lane in flight: the next four are requested before the current
// four are consumed.  Same vectors in the same order as lean_pass_a<false>, so the same sums.
__device__ __forceinline__ void lean_pass_a_deep(const uint4 *rp, int lo, int hi, int lane, float k, LeanAcc &P) {
    uint64_t pol;   // the row is read again by pass B: L2 is asked to keep it
    asm("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
    P.m2 = 0xff80ff80u; P.s = 0.f; P.c = 0.f;
    for (int vr = lo + lane; vr < hi; vr += 32) {
        const uint4 a = rp[vr];
        const float m0 = bf2_hmax(bf2max(bf2max(a.x, a.y), bf2max(a.z, a.w)));
        if (m0 > neg_inf()) { P.c = shift_of(m0, k); break; }
    }
    const int n = (hi - lo - lane + 31) >> 5;   // this lane's vectors (<= 0: none)
    const uint4 *p = rp + lo + lane;
    int it = 0;
    uint4 n0 = make_uint4(0, 0, 0, 0), n1 = n0, n2 = n0, n3 = n0;
    if (4 <= n) { n0 = ld_l2_hint(p, pol); n1 = ld_l2_hint(p + 32, pol); n2 = ld_l2_hint(p + 64, pol); n3 = ld_l2_hint(p + 96, pol); }
#pragma unroll 1
    for (; it + 4 <= n; it += 4) {
        const uint4 a0 = n0, a1 = n1, a2 = n2, a3 = n3;
        if (it + 8 <= n) {
            n0 = ld_l2_hint(p + 32 * (it + 4), pol); n1 = ld_l2_hint(p + 32 * (it + 5), pol);
            n2 = ld_l2_hint(p + 32 * (it + 6), pol); n3 = ld_l2_hint(p + 32 * (it + 7), pol);
        }
        lean_push(P, a0, k);
        lean_push(P, a1, k);
        lean_push(P, a2, k);
        lean_push(P, a3, k);
    }
    for (; it < n; ++it) lean_push(P, p[32 * it], k);
}

// Pass A over both rows with the vectors coming from the warp's ring (the first pass of its stream, forwards).
__device__ __forceinline__ void lean_pass_a_ring(WarpRing &R, int lane, float k, LeanAcc &P, LeanAcc &Q) {
    P.m2 = 0xff80ff80u; P.s = 0.f; P.c = 0.f;
    Q.m2 = 0xff80ff80u; Q.s = 0.f; Q.c = 0.f;
    const int vi0 = R.lo + lane;
    if (R.nc > 0) {
        // the reference comes from the thread's first vector that holds a finite logit: nearly always the
        // very first one, which the first chunk holds; otherwise look further in global memory
        ring_wait(R);
        if (vi0 < R.hi) {
            uint4 a, b;
            ring_load(R, 0, lane, a, b);
            float m0 = bf2_hmax(bf2max(bf2max(a.x, a.y), bf2max(a.z, a.w)));
            if (m0 > neg_inf()) P.c = shift_of(m0, k);
            else {
                for (int vr = vi0 + 32; vr < R.hi; vr += 32) {
                    const uint4 a2 = R.vp[vr];
                    m0 = bf2_hmax(bf2max(bf2max(a2.x, a2.y), bf2max(a2.z, a2.w)));
                    if (m0 > neg_inf()) { P.c = shift_of(m0, k); break; }
                }
            }
            m0 = bf2_hmax(bf2max(bf2max(b.x, b.y), bf2max(b.z, b.w)));
            if (m0 > neg_inf()) Q.c = shift_of(m0, k);
            else {
                for (int vr = vi0 + 32; vr < R.hi; vr += 32) {
                    const uint4 b2 = R.vq[vr];
                    m0 = bf2_hmax(bf2max(bf2max(b2.x, b2.y), bf2max(b2.z, b2.w)));
                    if (m0 > neg_inf()) { Q.c = shift_of(m0, k); break; }
                }
            }
        }
    }
#pragma unroll 1
    for (int c = 0; c < R.nc; ++c) {
        ring_wait(R);
        const int v0 = vi0 + c * kRingChunkVecs;
#pragma unroll
        for (int j = 0; j < kRingCh; ++j) {
            uint4 x, y;
            ring_load(R, j, lane, x, y);
            if (j == kRingCh - 1) ring_release(R, lane);
            if (v0 + j * 32 < R.hi) {
                lean_push(P, x, k);
                lean_push(Q, y, k);
            }
        }
    }
}

// The lanes of a warp rescan, together, the elements of its lane `src` (whose maximum equals the
// row maximum `val`): lane j takes the j-th vector of that thread, so the rescan costs one load
// round trip instead of one per vector.  Returns (to every lane) the first index of val among
// those elements and the sum of 2^(k l - c) over them without that index.
__device__ __forceinline__ void lean_rescan_warp(const uint4 *row, int lo, int hi, int lane, int src,
                                                 float val, float k, float c, int &first_idx,
                                                 float &s_excl) {
    int fi = 0x7fffffff;
    // pass 1: first index
    for (int vj = lo + src + 32 * lane; vj < hi; vj += 32 * 32) {
        float v[8];
        unpack_bf16x8(row[vj], v);
#pragma unroll
        for (int i = 7; i >= 0; --i)
            if (v[i] == val) fi = min(fi, vj * 8 + i);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) fi = min(fi, __shfl_xor_sync(kFull, fi, o));
    // pass 2: the sum without it (the vectors are L1/L2 hits now)
    float s = 0.f;
    for (int vj = lo + src + 32 * lane; vj < hi; vj += 32 * 32) {
        float v[8];
        unpack_bf16x8(row[vj], v);
        float e[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) e[i] = (vj * 8 + i == fi) ? 0.f : ex2(__fmaf_rn(v[i], k, -c));
        s += ((e[0] + e[1]) + (e[2] + e[3])) + ((e[4] + e[5]) + (e[6] + e[7]));
    }
    s_excl = warp_sum(s);
    first_idx = fi;
}

// Row-level (max, argmax, sum without the argmax) of the target (r = 0) and, if BOTH, the draft
// (r = 1) from the per-thread pass-A states.  Leaves the per-warp masses (row scale, argmax left
// out) in sh.wmass[r] for the samplers.  All threads call it.
template <bool BOTH>
__device__ void lean_reduce2(const LeanAcc &tp, const LeanAcc &tq, const uint4 *vp, const uint4 *vq, int lo,
                             int hi, float k, LeanShared &sh, ArgMaxSum &P, ArgMaxSum &Q) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
    const float mlp = bf2_hmax(tp.m2), mlq = BOTH ? bf2_hmax(tq.m2) : neg_inf();
    float wp = mlp, wq = mlq;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        wp = fmaxf(wp, __shfl_xor_sync(kFull, wp, o));
        if (BOTH) wq = fmaxf(wq, __shfl_xor_sync(kFull, wq, o));
    }
    if (lane == 0) { sh.wml[0][warp] = wp; sh.wml[1][warp] = wq; }
    if (threadIdx.x == 0) { sh.cand[0] = 0x7fffffff; sh.cand[1] = 0x7fffffff; }
    __syncthreads();
    float rmp = sh.wml[0][0], rmq = sh.wml[1][0];
    for (int w = 1; w < nwarps; ++w) { rmp = fmaxf(rmp, sh.wml[0][w]); rmq = fmaxf(rmq, sh.wml[1][w]); }
    const float pinf = -neg_inf();
    int idxp_mine = 0x7fffffff, idxq_mine = 0x7fffffff;
    float sxp = 0.f, sxq = 0.f;
    {
        const bool cand = (mlp == rmp) && rmp > neg_inf() && rmp < pinf;
        unsigned cm = __ballot_sync(kFull, cand);
        while (cm) {
            const int src = __ffs(cm) - 1;
            cm &= cm - 1;
            int fi; float sx;
            lean_rescan_warp(vp, lo, hi, lane, src, rmp, k, __shfl_sync(kFull, tp.c, src), fi, sx);
            if (lane == src) { idxp_mine = fi; sxp = sx; atomicMin(&sh.cand[0], fi); }
        }
    }
    if (BOTH) {
        const bool cand = (mlq == rmq) && rmq > neg_inf() && rmq < pinf;
        unsigned cm = __ballot_sync(kFull, cand);
        while (cm) {
            const int src = __ffs(cm) - 1;
            cm &= cm - 1;
            int fi; float sx;
            lean_rescan_warp(vq, lo, hi, lane, src, rmq, k, __shfl_sync(kFull, tq.c, src), fi, sx);
            if (lane == src) { idxq_mine = fi; sxq = sx; atomicMin(&sh.cand[1], fi); }
        }
    }
    __syncthreads();
    const int idxp = sh.cand[0], idxq = sh.cand[1];
    const float Cp = shift_of(rmp, k), Cq = shift_of(rmq, k);
    {
        const float mine = (idxp_mine != 0x7fffffff && idxp_mine == idxp) ? sxp : tp.s;
        float v = (mlp > neg_inf()) ? mine * ex2(tp.c - Cp) : 0.f;
        v = warp_sum(v);
        if (lane == 0) sh.wmass[0][warp] = v;
    }
    if (BOTH) {
        const float mine = (idxq_mine != 0x7fffffff && idxq_mine == idxq) ? sxq : tq.s;
        float v = (mlq > neg_inf()) ? mine * ex2(tq.c - Cq) : 0.f;
        v = warp_sum(v);
        if (lane == 0) sh.wmass[1][warp] = v;
    }
    __syncthreads();
    float t0 = 0.f, t1 = 0.f;
    for (int w = 0; w < nwarps; ++w) { t0 += sh.wmass[0][w]; if (BOTH) t1 += sh.wmass[1][w]; }
    P.ml = rmp; P.c = Cp; P.idx = idxp; P.sx = t0;
    Q.ml = rmq; Q.c = Cq; Q.idx = idxq; Q.sx = t1;
}

// CTA-wide inverse-CDF draw over this CTA's part of a row.  sh.mass[w] = total weight of warp w's
// range (the coarse CDF); weights(vi, w[8]) the weights of vector vi; t = target prefix within
// this part.  Every thread knows the selected warp range; pass 1 cuts it into one contiguous
// block of vectors per thread of the CTA and sums the blocks in parallel, warp 0 scans the block
// sums; pass 2 spreads the chosen block's vectors over the lanes of warp 0.  Two load round trips
// in all.  Returns to every thread the lowest id whose inclusive prefix exceeds t; when rounding
// leaves none inside the selected range, the last id with positive weight there; -1 when this
// part has no mass.  Called by all threads of the CTA.
// The two passes of the CTA-wide draw over the vectors [lo, hi): tt = target prefix within the
// range.  Called by all threads of the CTA; returns the id to every thread (-1: no mass in range).
template <class WF>
__device__ int range_sample3(int lo, int hi, WF weights, LeanShared &sh, float tt) {
    const int lane = threadIdx.x & 31, nth = blockDim.x;
    const int Bv = (hi - lo + nth - 1) / nth;  // vectors per thread block
    {   // pass 1
        const int b0 = lo + threadIdx.x * Bv, b1 = min(hi, b0 + Bv);
        float tot = 0.f;
#pragma unroll 4
        for (int vi = b0; vi < b1; ++vi) {
            float w[8];
            weights(vi, w);
            tot += ((w[0] + w[1]) + (w[2] + w[3])) + ((w[4] + w[5]) + (w[6] + w[7]));
        }
        sh.part[threadIdx.x] = tot;
    }
    __syncthreads();
    if (threadIdx.x < 32) {
        const int per = nth >> 5;  // block sums per lane
        float ls = 0.f;
        for (int i = 0; i < per; ++i) ls += sh.part[lane * per + i];
        float incl = ls;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const float up = __shfl_up_sync(kFull, incl, o);
            if (lane >= o) incl += up;
        }
        const unsigned pos = __ballot_sync(kFull, ls > 0.f);
        const unsigned hit = __ballot_sync(kFull, ls > 0.f && incl > tt);
        int blk = -1;
        float tt2 = 0.f;
        if (pos) {
            const int L = hit ? (__ffs(hit) - 1) : (31 - __clz(pos));
            if (lane == L) {
                float acc = incl - ls;
                int lastb = -1;
                float lastacc = 0.f;
                for (int i = 0; i < per; ++i) {
                    const float m = sh.part[lane * per + i];
                    if (m > 0.f) {
                        lastb = lane * per + i;
                        lastacc = acc;
                        if (blk < 0 && acc + m > tt) { blk = lastb; tt2 = tt - acc; }
                    }
                    acc += m;
                }
                if (blk < 0) { blk = lastb; tt2 = tt - lastacc; }
                sh.blk = blk;
                sh.tt2 = tt2;
            }
        } else if (lane == 0) {
            sh.blk = -1;
        }
        __syncwarp();
        blk = sh.blk;
        tt2 = sh.tt2;
        int found = -1;
        if (blk >= 0) {   // pass 2: the block's vectors over the lanes
            const int c0 = lo + blk * Bv, c1 = min(hi, c0 + Bv);
            float prefix = 0.f;
            int lastpos = -1;
            for (int v0 = c0; v0 < c1 && found < 0; v0 += 32) {
                const int vi = v0 + lane;
                float w[8];
                if (vi < c1) {
                    weights(vi, w);
                } else {
#pragma unroll
                    for (int i = 0; i < 8; ++i) w[i] = 0.f;
                }
                float lsum = 0.f;
                int lp = -1;
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    lsum += w[i];
                    if (w[i] > 0.f) lp = vi * 8 + i;
                }
                float in2 = lsum;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const float up = __shfl_up_sync(kFull, in2, o);
                    if (lane >= o) in2 += up;
                }
                const float tot2 = __shfl_sync(kFull, in2, 31);
                const unsigned hit2 = __ballot_sync(kFull, lsum > 0.f && prefix + in2 > tt2);
                if (hit2) {
                    const int M = __ffs(hit2) - 1;
                    int cand = -1;
                    if (lane == M) {
                        float acc = prefix + (in2 - lsum);
                        int lastin = -1;
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            acc += w[i];
                            if (w[i] > 0.f) {
                                lastin = vi * 8 + i;
                                if (cand < 0 && acc > tt2) cand = lastin;
                            }
                        }
                        if (cand < 0) cand = lastin;
                    }
                    found = __shfl_sync(kFull, cand, M);
                } else {
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) lp = max(lp, __shfl_xor_sync(kFull, lp, o));
                    lastpos = max(lastpos, lp);
                    prefix += tot2;
                }
            }
            if (found < 0) found = lastpos;
        }
        if (lane == 0) sh.tok = found;
    }
    __syncthreads();
    const int tok = sh.tok;
    __syncthreads();
    return tok;
}

template <class WF>
__device__ int block_sample3(const Geo &g, WF weights, LeanShared &sh, float t) {
    int wsel = -1, lastw = -1;
    float base = 0.f, lastbase = 0.f, run = 0.f;
    for (int w = 0; w < g.nwarps; ++w) {
        const float m = sh.mass[w];
        if (m > 0.f) {
            lastw = w;
            lastbase = run;
            if (wsel < 0 && run + m > t) { wsel = w; base = run; }
        }
        run += m;
    }
    if (lastw < 0) return -1;
    if (wsel < 0) { wsel = lastw; base = lastbase; }
    return range_sample3(g.seg_lo(wsel), g.seg_hi(wsel), weights, sh, t - base);
}

// Pick the CTA of a row whose part holds the target t of an inverse-CDF draw over per-CTA masses
// m[0..n) (ascending token ranges).  Returns the rank (-1 if no mass) and the mass before it.
__device__ __forceinline__ int pick_part(const float *m, int n, float t, float &base) {
    int sel = -1, last = -1;
    float lastbase = 0.f, run = 0.f;
    base = 0.f;
    for (int r = 0; r < n; ++r) {
        if (m[r] > 0.f) {
            last = r;
            lastbase = run;
            if (sel < 0 && run + m[r] > t) { sel = r; base = run; }
        }
        run += m[r];
    }
    if (sel < 0) { sel = last; base = lastbase; }
    return sel;
}

// What every CTA of a row knows about one of its rows after the slices were merged.
struct RowStat {
    float ml, C, sx;  // row max logit, its shift, sum without the row argmax
    float own;        // the row argmax's own term 2^(k ml - C) (1 up to the rounding of C)
    int idx;          // row argmax
};

// Merge the slices' (max, argmax, sum without argmax) in rank order (Section 4: a = argmax q).
template <int CS>
__device__ __forceinline__ void merge_slices(const LeanShared &sh, int r, float k, RowStat &st) {
    ArgMaxSum tot;
    tot.init();
#pragma unroll
    for (int c = 0; c < CS; ++c) {
        const LeanShared *ps = RowGroup<CS>::peer(&sh, c);
        ArgMaxSum o;
        o.ml = ps->x_ml[r]; o.c = shift_of(o.ml, k); o.sx = ps->x_sx[r]; o.idx = ps->x_idx[r];
        tot = argmaxsum_merge(tot, o, k);
    }
    st.ml = tot.ml; st.C = tot.c; st.sx = tot.sx; st.idx = tot.idx; st.own = tot.own(k);
}

// Mass of slice c of a row (row scale) for a draw from softmax(row) without token `excl`
// (excl < 0: none; only a slice's own argmax can be left out here).  The slices' published
// partials stay valid until the kernel ends.
template <int CS>
__device__ __forceinline__ float slice_mass(const LeanShared &sh, int r, const RowStat &st, int c, int excl,
                                            float k) {
    const LeanShared *ps = RowGroup<CS>::peer(&sh, c);
    const float ml = ps->x_ml[r];
    const float own = (ps->x_idx[r] != excl) ? own_term(ml, k) : 0.f;
    return (ps->x_sx[r] + own) * rescale(ml, shift_of(ml, k), st.C);
}

// Draw inside this CTA's slice from softmax(row) without token `excl`, target t (row scale,
// relative to the start of the slice).  sh.wmass[r] holds the per-warp sums of the slice on the
// slice's own scale with the slice argmax left out.
__device__ int lean_sample_slice(const Geo &g, const __nv_bfloat16 *row, float k, const RowStat &st,
                                 int excl, float t, int r, LeanShared &sh) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int locarg = sh.x_idx[r];
    const float lml = sh.x_ml[r];
    const float f = rescale(lml, shift_of(lml, k), st.C);
    const float C = st.C;
    if (threadIdx.x < g.nwarps) {
        const int w = threadIdx.x;
        const int lv = locarg >> 3;
        const bool holds = lml > neg_inf() && lv >= g.seg_lo(w) && lv < g.seg_hi(w);
        sh.mass[w] = (sh.wmass[r][w] + ((holds && excl != locarg) ? own_term(lml, k) : 0.f)) * f;
    }
    __syncthreads();
    if (excl >= 0 && excl != locarg && g.holds_vec(excl >> 3)) {
        // an arbitrary token of this slice is removed: its warp re-sums its range
        const int wex = g.warp_of_vec(excl >> 3);
        if (warp == wex) {
            float s = 0.f;
            for (int vi = g.seg_lo(warp) + lane; vi < g.seg_hi(warp); vi += 32) {
                float v[8];
                load_vec<__nv_bfloat16, true>(row, vi, g.V, v);
#pragma unroll
                for (int i = 0; i < 8; ++i) s += (vi * 8 + i == excl) ? 0.f : ex2(__fmaf_rn(v[i], k, -C));
            }
            s = warp_sum(s);
            if (lane == 0) sh.mass[warp] = s;
        }
        __syncthreads();
    }
    auto wf = [&](int vi, float(&w)[8]) {
        float v[8];
        load_vec<__nv_bfloat16, true>(row, vi, g.V, v);
#pragma unroll
        for (int i = 0; i < 8; ++i) w[i] = (vi * 8 + i == excl) ? 0.f : ex2(__fmaf_rn(v[i], k, -C));
    };
    return block_sample3(g, wf, sh, t);
}

// Draw from softmax(row) without `excl` (the row argmax, a slice argmax, or nothing) over the
// whole row: every CTA of the row calls it; the CTA whose slice holds the target draws and
// returns the token, the others return -2.  -1: no mass.
template <int CS>
__device__ int lean_sample_row(const Geo &g, const __nv_bfloat16 *row, float k, const RowStat &st, int me,
                               int excl, float u, int r, LeanShared &sh) {
    float m[CS];
    float total = 0.f;
#pragma unroll
    for (int c = 0; c < CS; ++c) { m[c] = slice_mass<CS>(sh, r, st, c, excl, k); total += m[c]; }
    if (!(total > 0.f)) return -1;
    float base;
    const int sel = pick_part(m, CS, u * total, base);
    if (sel != me) return -2;
    return lean_sample_slice(g, row, k, st, excl, u * total - base, r, sh);
}

// CTA sums of NACC per-thread accumulators; the per-warp sums stay in sh.acc[OFF + i][w].
template <int NACC, int OFF = 0>
__device__ __forceinline__ void lean_block_sums(float (&x)[NACC], LeanShared &sh) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
#pragma unroll
    for (int i = 0; i < NACC; ++i) {
        const float s = warp_sum(x[i]);
        if (lane == 0) sh.acc[OFF + i][warp] = s;
    }
    __syncthreads();
    const int nwarps = blockDim.x >> 5;
#pragma unroll
    for (int i = 0; i < NACC; ++i) {
        float t = 0.f;
        for (int w = 0; w < nwarps; ++w) t += sh.acc[OFF + i][w];
        x[i] = t;
    }
}

// Sum NACC per-thread accumulators over the whole row: CTA sums, then the slices in rank order.
// part[i][c] receives slice c's sum of accumulator i; sh.acc[i][w] keeps this CTA's per-warp sums.
// Contains one row-group barrier.  OFF: first exchange slot used (a second call in the same
// kernel takes other slots, so no CTA overwrites what a slower one has not read yet).
template <int CS, int NACC, int OFF>
__device__ __forceinline__ void lean_row_sums(float (&x)[NACC], float (&part)[NACC][CS], LeanShared &sh) {
    lean_block_sums<NACC>(x, sh);
    if (CS == 1) {
#pragma unroll
        for (int i = 0; i < NACC; ++i) part[i][0] = x[i];
        __syncthreads();  // sh.acc may be rewritten by a later sum only after all have read it
        return;
    }
    if (threadIdx.x == 0) {
#pragma unroll
        for (int i = 0; i < NACC; ++i) sh.x_sum[OFF + i] = x[i];
    }
    RowGroup<CS>::sync();
#pragma unroll
    for (int i = 0; i < NACC; ++i) {
        float t = 0.f;
#pragma unroll
        for (int c = 0; c < CS; ++c) {
            part[i][c] = RowGroup<CS>::peer(&sh, c)->x_sum[OFF + i];
            t += part[i][c];
        }
        x[i] = t;
    }
}

// ------------------------------------------------------------------------------------------------
// Draft step, one CTA per row, with a finer coarse CDF.  Pass A records, every CK lane-iterations,
// the warp's sum since its previous checkpoint: sub-blocks of 32 * CK consecutive vectors, at most
// kLeanCk per warp.  A draw then picks a sub-block from those sums and rescans only that (a few KB
// instead of a warp's whole range), which is what the two-pass sampler costs most.
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ int lean_ck_interval(const Geo &g) {
    const int iters = (g.seg + 31) >> 5;
    return 4 * max(1, (iters + 4 * kLeanCk - 1) / (4 * kLeanCk));   // a multiple of the unroll of pass A
}

__device__ __forceinline__ void lean_pass_a_ck(const uint4 *rq, int lo, int hi, int lane, float k, int CK,
                                               LeanAcc &Q, float *cks, float *ckc) {
    LeanAcc st;
    st.m2 = 0xff80ff80u; st.s = 0.f; st.c = 0.f;
    {   // one exponent reference for the whole warp: the maximum of its first vectors
        float m0 = neg_inf();
        if (lo + lane < hi) {
            const uint4 a = rq[lo + lane];
            m0 = bf2_hmax(bf2max(bf2max(a.x, a.y), bf2max(a.z, a.w)));
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) m0 = fmaxf(m0, __shfl_xor_sync(kFull, m0, o));
        if (m0 > neg_inf()) st.c = shift_of(m0, k);
    }
    float cref = st.c;              // the reference every lane is expected to hold
    float tot = 0.f, ctot = st.c;   // this thread's sum over all checkpoints, on the scale ctot
    int j = 0;
    // checkpoint: the warp's sum since the last one.  A lane that had to move its reference (sums
    // beyond 2^100, rare) is brought to the warp's largest reference first.
    auto checkpoint = [&]() {
        float contrib = st.s, cnow = cref;
        if (__any_sync(kFull, st.c != cref)) {
            float cm = st.c;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) cm = fmaxf(cm, __shfl_xor_sync(kFull, cm, o));
            contrib = st.s > 0.f ? st.s * ex2(st.c - cm) : 0.f;
            cnow = cm;
        }
        const float cs = warp_sum(contrib);
        if (lane == 0) { cks[j] = cs; ckc[j] = cnow; }
        ++j;
        if (st.c != ctot) { tot = tot > 0.f ? tot * ex2(ctot - st.c) : 0.f; ctot = st.c; }
        tot += st.s;
        st.s = 0.f;
    };
    const int iters = (hi - lo + 31) >> 5;   // lane-iterations of this warp
    const int nfull = (hi - lo) >> 5;        // those in which every lane has a vector
    const uint4 *p = rq + lo + lane;
    int it = 0, since = 0;
    // four vectors per lane in flight; the next four are requested before the current ones are
    // consumed, so that the checkpoint's shuffle chain overlaps the loads
    uint4 n0 = make_uint4(0, 0, 0, 0), n1 = n0, n2 = n0, n3 = n0;
    if (4 <= nfull) { n0 = p[0]; n1 = p[32]; n2 = p[64]; n3 = p[96]; }
    for (; it + 4 <= nfull; it += 4) {
        const uint4 a0 = n0, a1 = n1, a2 = n2, a3 = n3;
        if (it + 8 <= nfull) {
            n0 = p[32 * (it + 4)]; n1 = p[32 * (it + 5)]; n2 = p[32 * (it + 6)]; n3 = p[32 * (it + 7)];
        }
        lean_push(st, a0, k);
        lean_push(st, a1, k);
        lean_push(st, a2, k);
        lean_push(st, a3, k);
        since += 4;
        if (since >= CK) { checkpoint(); since = 0; }
    }
    for (; it < iters; ++it) {
        if (lo + lane + 32 * it < hi) lean_push(st, p[32 * it], k);
        if (++since >= CK) { checkpoint(); since = 0; }
    }
    if (since > 0) checkpoint();
    if (lane == 0)
        for (; j < kLeanCk; ++j) { cks[j] = 0.f; ckc[j] = 0.f; }
    Q.m2 = st.m2; Q.c = st.c; Q.s = tot;
}

// Inverse-CDF draw from softmax(row) without token `excl` (excl < 0: nothing left out) over the
// checkpoint sub-blocks.  C = the row's exponent shift.  Returns to every thread the token, -1 if
// nothing has mass.  Called by all threads of the CTA, after the checkpoints are visible.
__device__ int lean_ck_sample(const Geo &g, const __nv_bfloat16 *row, float k, float C, int CK, int excl,
                              float u, LeanCkShared &sh) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nslot = g.nwarps * kLeanCk;
    auto wf = [&](int vi, float(&w)[8]) {
        float v[8];
        load_vec<__nv_bfloat16, true>(row, vi, g.V, v);
#pragma unroll
        for (int i = 0; i < 8; ++i) w[i] = (vi * 8 + i == excl) ? 0.f : ex2(__fmaf_rn(v[i], k, -C));
    };
    for (int s = threadIdx.x; s < nslot; s += blockDim.x) {
        const float cs = sh.cks[s / kLeanCk][s % kLeanCk];
        sh.ckm[s] = cs > 0.f ? cs * ex2(sh.ckc[s / kLeanCk][s % kLeanCk] - C) : 0.f;
    }
    __syncthreads();
    if (excl >= 0) {
        // the sub-block that holds the excluded token is summed again without it: subtracting the
        // token's own term would cancel when that token carries most of the sub-block's mass
        const int ev = excl >> 3;
        const int w = g.warp_of_vec(ev), j = (ev - g.seg_lo(w)) / (32 * CK);
        const int b0 = g.seg_lo(w) + 32 * CK * j, b1 = min(g.seg_hi(w), b0 + 32 * CK);
        float s = 0.f;
        for (int vi = b0 + threadIdx.x; vi < b1; vi += blockDim.x) {
            float wt[8];
            wf(vi, wt);
            s += ((wt[0] + wt[1]) + (wt[2] + wt[3])) + ((wt[4] + wt[5]) + (wt[6] + wt[7]));
        }
        s = warp_sum(s);
        if (lane == 0) sh.mass[warp] = s;
        __syncthreads();
        if (threadIdx.x == 0) {
            float t = 0.f;
            for (int x = 0; x < g.nwarps; ++x) t += sh.mass[x];
            sh.ckm[w * kLeanCk + j] = t;
        }
        __syncthreads();
    }
    if (threadIdx.x < 32) {   // warp 0: prefix sums over the sub-blocks, in id order
        const int per = (nslot + 31) >> 5;
        float ls = 0.f;
        for (int i = 0; i < per; ++i) {
            const int s = lane * per + i;
            if (s < nslot) ls += sh.ckm[s];
        }
        float incl = ls;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const float up = __shfl_up_sync(kFull, incl, o);
            if (lane >= o) incl += up;
        }
        const float total = __shfl_sync(kFull, incl, 31);
        const float t = u * total;
        const unsigned pos = __ballot_sync(kFull, ls > 0.f);
        const unsigned hit = __ballot_sync(kFull, ls > 0.f && incl > t);
        if (!pos || !(total > 0.f)) {
            if (lane == 0) sh.blk = -1;
        } else {
            const int L = hit ? (__ffs(hit) - 1) : (31 - __clz(pos));
            if (lane == L) {
                float acc = incl - ls, lastacc = 0.f;
                int sel = -1, last = -1;
                for (int i = 0; i < per; ++i) {
                    const int s = lane * per + i;
                    const float m = s < nslot ? sh.ckm[s] : 0.f;
                    if (m > 0.f) {
                        last = s;
                        lastacc = acc;
                        if (sel < 0 && acc + m > t) { sel = s; sh.tt2 = t - acc; }
                    }
                    acc += m;
                }
                if (sel < 0) { sel = last; sh.tt2 = t - lastacc; }
                sh.blk = sel;
            }
        }
    }
    __syncthreads();
    const int slot = sh.blk;
    const float tt = sh.tt2;
    __syncthreads();   // range_sample3 reuses blk / tt2
    if (slot < 0) return -1;
    const int w = slot / kLeanCk, j = slot % kLeanCk;
    const int b0 = g.seg_lo(w) + 32 * CK * j, b1 = min(g.seg_hi(w), b0 + 32 * CK);
    return range_sample3(b0, b1, wf, sh, tt);
}

// Leaf rows (Figure 2: after the last accepted draft the bonus token is a draw from p) of a call
// whose rows are not split over clusters get a kernel of their own, shaped like the draft step:
// pass A over p with checkpoints, then the sub-block sampler.  CTAs of verifying rows leave at
// once; the verification kernels skip the leaf rows.  Up to three output sets receive the result
// (the three-method call: the methods share u_res, hence the bonus token).
struct NodeOutPtrs {
    int32_t *accept_idx, *token, *hub;
    float *beta, *rate;
    uint32_t *status;
};
struct LeafArgs {
    RowArgs r;
    NodeOutPtrs out[3];
    int n_out;
};

template <int THREADS>
__global__ void __launch_bounds__(THREADS, 1024 / THREADS) lean_leaf_kernel(LeafArgs A) {
    __shared__ LeanCkShared sh;
    const RowArgs &a = A.r;
    const long long r = blockIdx.x;
    const int b = static_cast<int>(r / a.nodes), n = static_cast<int>(r % a.nodes);
    if (!(a.node_kind && a.node_kind[n] == SPECHUB_NODE_LEAF)) return;
    const __nv_bfloat16 *rowp = static_cast<const __nv_bfloat16 *>(a.target) + b * a.stride_seq + n * a.stride_node;
    const uint4 *vp = reinterpret_cast<const uint4 *>(rowp);
    const Geo g = make_geo(a.vocab, 8);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int lo = g.seg_lo(warp), hi = g.seg_hi(warp);
    const float k = kLog2e / temperature_of(a, b);
    const float ures = a.uniforms[r * 5 + 4];
    const int CK = lean_ck_interval(g);
    LeanAcc tp, unused;
    unused.m2 = 0xff80ff80u; unused.s = 0.f; unused.c = 0.f;
    lean_pass_a_ck(vp, lo, hi, lane, k, CK, tp, sh.cks[warp], sh.ckc[warp]);
    ArgMaxSum Ps, unusedq;
    lean_reduce2<false>(tp, unused, vp, vp, lo, hi, k, sh, Ps, unusedq);
    const float Zp = Ps.sx + Ps.own(k);
    uint32_t status = 0;
    int tok = -1;
    if (!(Ps.ml > neg_inf()) || !(Ps.ml < -neg_inf()) || !finite_pos(Zp)) status = SPECHUB_ST_NONFINITE;
    else tok = lean_ck_sample(g, rowp, k, Ps.c, CK, -1, ures, sh);
    if (threadIdx.x == 0) {
        for (int m = 0; m < A.n_out; ++m) {
            const NodeOutPtrs &o = A.out[m];
            o.accept_idx[r] = -1;
            o.token[r] = tok;
            if (o.hub) o.hub[r] = -1;
            if (o.beta) { o.beta[2 * r] = 0.f; o.beta[2 * r + 1] = 0.f; }
            if (o.rate) { o.rate[3 * r] = 0.f; o.rate[3 * r + 1] = 0.f; o.rate[3 * r + 2] = status ? 0.f : 1.f; }
            if (o.status) o.status[r] = status;
        }
    }
}

// Passes B and C work on the exponentials themselves, in units of 1 / Z_p: with rho = Z_p / Z_q,
//   d = e_p - rho e_q = Z_p (p - q),   t = max(d, 0) - s rho e_q = Z_p (max(p - q, 0) - s q),
// two FMAs per vocabulary pair instead of two multiplications by 1/Z, a subtraction and an FMA.
// Identical target and draft rows give rho = 1 and e_p = e_q bit for bit, so d = 0 exactly.
__device__ __forceinline__ float lean_exp(float logit, float k, float c) { return ex2(__fmaf_rn(logit, k, -c)); }
__device__ __forceinline__ void lean_terms(float ep, float eq, float rho, float srho, float &d, float &t) {
    d = __fmaf_rn(-rho, eq, ep);
    t = __fmaf_rn(-srho, eq, fmaxf(d, 0.f));
}

// Sum of a row's exponentials outside id x, from the row's (maximum, argmax, sum without the argmax): RRSw's
// renormaliser 1 - q(x1) times Z_q without a pass over the row.  The argmax is left out of st.sx already; any
// other id holds at most half of the mass, so subtracting its own term costs at most one bit.
__device__ __forceinline__ float sum_without(const RowStat &st, const __nv_bfloat16 *row, int x, float k) {
    if (x == st.idx) return st.sx;
    return __fsub_rn(__fadd_rn(st.sx, st.own), lean_exp(load_one<__nv_bfloat16>(row, x), k, st.C));
}

// ------------------------------------------------------------------------------------------------
// Verification (SpecHub: Algorithm 3; RRS / RRSw: Algorithm 1) and leaf draws.
// ------------------------------------------------------------------------------------------------
// RING (RRS and RRSw, one CTA per row): the passes over both rows take their vectors from per-warp rings of
// bulk copies (spechub_ring.cuh; THREADS / 32 * kRingWarpBytes of dynamic shared memory) instead of loading
// them from global memory into registers.  Measured on V = 128256, 7936 rows: RRS 1.89 -> 1.72 ms, RRSw
// 1.99 -> 1.86 ms; SpecHub's two passes gain nothing from it (1.38 -> 1.38 .. 1.44 ms: the bookkeeping of
// the ring costs the issue slots that its pass B is short of), so SpecHub keeps the register-fed loops.
// STATS (one CTA per row): the maximum, argmax and sum of the draft row come from the record the draft
// step left (RowArgs::draft_stats_in), so pass A reads the target row only; a record that does not belong
// to the row (tag, argmax out of range, or another logit there than the recorded maximum) flags the row
// SPECHUB_ST_STATS.  The passes are register-fed, with L2 eviction hints on the loads (keep the target row
// after pass A, let the rows go at their last use): with a single row to keep in L2 between passes that
// beats the rings (RRS 1.53 -> 1.46 ms, RRSw 1.62 -> 1.60 ms on V = 128256, 7936 rows).
template <int METHOD, int THREADS, int CS, bool RING = false, bool STATS = false>
__global__ void __launch_bounds__(THREADS, 1024 / THREADS) lean_verify_kernel(RowArgs a) {
    static_assert(!RING || (CS == 1 && METHOD != kSpecHub), "the ring-fed form: whole rows, RRS and RRSw");
    static_assert(!STATS || (CS == 1 && !RING), "draft statistics: whole rows, register-fed passes");
    __shared__ LeanShared sh;
    extern __shared__ __align__(128) unsigned char ring_mem[];
    __shared__ __align__(8) uint64_t ring_bars[RING ? THREADS / 32 : 1][kRingStages];
    const int me = RowGroup<CS>::rank();
    const long long r = blockIdx.x / CS;
    const int b = static_cast<int>(r / a.nodes), n = static_cast<int>(r % a.nodes);
    const __nv_bfloat16 *rowp = static_cast<const __nv_bfloat16 *>(a.target) + b * a.stride_seq + n * a.stride_node;
    const __nv_bfloat16 *rowq = static_cast<const __nv_bfloat16 *>(a.draft) + b * a.stride_seq + n * a.stride_node;
    const uint4 *vp = reinterpret_cast<const uint4 *>(rowp), *vq = reinterpret_cast<const uint4 *>(rowq);
    const Geo g = make_geo(a.vocab, 8, CS, me);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int lo = g.seg_lo(warp), hi = g.seg_hi(warp);
    // Pass B walks this lane's vectors backwards: what pass A read last is read again first, so
    // the tail of the row is still in L2 even when the rows in flight exceed its capacity.
    const int last_vi = (lo + lane < hi) ? lo + lane + ((hi - 1 - lo - lane) / 32) * 32 : lo - 1;
    const float k = kLog2e / temperature_of(a, b);
    const float r1 = a.uniforms[r * 5 + 2], r2 = a.uniforms[r * 5 + 3], ures = a.uniforms[r * 5 + 4];
    const float pinf = -neg_inf();
    // leaf rows of an unsplit call belong to lean_leaf_kernel
    if (CS == 1 && a.node_kind && a.node_kind[n] == SPECHUB_NODE_LEAF) return;
    const bool leaf = CS > 1 && a.node_kind && a.node_kind[n] == SPECHUB_NODE_LEAF;
    const bool writer = (me == 0 && threadIdx.x == 0);

    NodeResult o;
    o.accept_idx = -1; o.token = -1; o.hub = -1; o.status = 0;
    o.beta[0] = o.beta[1] = 0.f; o.rate[0] = o.rate[1] = o.rate[2] = 0.f;
    // The token is written by the CTA that knows it: the row's first CTA for an accepted draft or
    // a flagged row, the CTA that draws for a residual / leaf token.
    bool token_elsewhere = false;

    if (STATS && threadIdx.x == THREADS - 1) {
        // The draft row's record, fetched and checked by one thread before it starts on pass A: its two
        // dependent look-ups (the record, then the draft logit at the recorded argmax) are off the path
        // between pass A and pass B.  (Nothing else writes these fields; they are read after barriers.)
        const DraftStat ds = static_cast<const DraftStat *>(a.draft_stats_in)[r];
        bool ok = ds.tag == (kDraftStatTag ^ __float_as_uint(k));
        // (a record of a row without a finite maximum or sum needs no look-up: the row is flagged
        // SPECHUB_ST_NONFINITE below, as it is without the record)
        if (ok && ds.ml > neg_inf() && ds.ml < pinf && finite_pos(ds.sx + 1.f))
            ok = ds.idx >= 0 && ds.idx < a.vocab && load_one<__nv_bfloat16>(rowq, ds.idx) == ds.ml;
        sh.stat_ok = ok;
        sh.x_ml[1] = ds.ml; sh.x_sx[1] = ds.sx; sh.x_idx[1] = ok ? ds.idx : 0;
    }
    // the row's stream: pass A forwards, pass B backwards, (RRS, RRSw) pass C forwards
    WarpRing R;
    if (RING) ring_begin(R, ring_mem + warp * kRingWarpBytes, ring_bars[warp], vp, vq, lo, hi, 3, 2u, lane);
    LeanAcc tp, tq;
    if (RING) lean_pass_a_ring(R, lane, k, tp, tq);
    else if (STATS) lean_pass_a_deep(vp, lo, hi, lane, k, tp);
    else if (leaf) lean_pass_a<false>(vp, vq, lo, hi, lane, k, tp, tq);
    else lean_pass_a<true, METHOD == kRRS>(vp, vq, lo, hi, lane, k, tp, tq);
    {
        ArgMaxSum Ps, Qs;
        if (leaf || STATS) lean_reduce2<false>(tp, tq, vp, vq, lo, hi, k, sh, Ps, Qs);
        else lean_reduce2<true>(tp, tq, vp, vq, lo, hi, k, sh, Ps, Qs);
        if (threadIdx.x == 0) {
            sh.x_ml[0] = Ps.ml; sh.x_sx[0] = Ps.sx; sh.x_idx[0] = Ps.idx;
            if (!STATS) { sh.x_ml[1] = Qs.ml; sh.x_sx[1] = Qs.sx; sh.x_idx[1] = Qs.idx; }
        }
    }
    RowGroup<CS>::sync();  // [1] slices published
    RowStat P, Q;
    merge_slices<CS>(sh, 0, k, P);
    merge_slices<CS>(sh, 1, k, Q);
    // (Z_p, its shift and rho change only in verification from draft statistics, when the two rows turn
    // out to be the same row: see below)
    float Zp = P.sx + P.own;
    const float Zq = Q.sx + Q.own;
    float cP = P.C, invZp = 1.f / Zp;
    const float cQ = Q.C, invZq = 1.f / Zq;
    float rho = __fdiv_rn(Zp, Zq);
    // With draft statistics Z_q was summed by another kernel, in another order than Z_p here.  That is
    // rounding, except when the target row is the draft row bit for bit: then Z_p = Z_q, every p - q is 0 and
    // the sums S1, R, A1 are exactly 0, which a rho of 1 +- 1e-7 would turn into noise that the tests then
    // divide by.  Pass B sees both rows and notices; the row is then redone with p's normaliser set to q's.
    unsigned diff = 0;
    auto rows_identical = [&]() {
        if (__syncthreads_or(diff != 0)) return false;
        Zp = Zq; invZp = invZq; cP = cQ; rho = 1.f;
        return true;
    };
    const int x1 = a.draft_tokens_in[2 * r], x2 = a.draft_tokens_in[2 * r + 1];
    auto prob_p = [&](int y) { return prob_of(load_one<__nv_bfloat16>(rowp, y), k, cP, invZp); };
    auto prob_q = [&](int y) { return prob_of(load_one<__nv_bfloat16>(rowq, y), k, cQ, invZq); };
    auto draw_from_p = [&]() {  // every CTA of the row calls it
        const int tok = lean_sample_row<CS>(g, rowp, k, P, me, -1, ures, 0, sh);
        if (tok != -2 && threadIdx.x == 0) a.token[r] = tok;
        token_elsewhere = true;
    };

    do {
        if (STATS && !sh.stat_ok) { o.status = SPECHUB_ST_STATS; break; }
        if (!(P.ml > neg_inf()) || !(P.ml < pinf) || !finite_pos(Zp)) { o.status = SPECHUB_ST_NONFINITE; break; }
        if (leaf) {
            // bonus token after the last accepted draft (Figure 2): a draw from p
            draw_from_p();
            o.rate[2] = 1.f;
            break;
        }
        if (!(Q.ml > neg_inf()) || !(Q.ml < pinf) || !finite_pos(Zq)) { o.status = SPECHUB_ST_NONFINITE; break; }
        if (METHOD == kSpecHub) {
            const int hubtok = Q.idx;
            o.hub = hubtok;
            const bool pair_xa = (x2 == hubtok && x1 != hubtok), pair_ax = (x1 == hubtok && x2 != hubtok);
            const int x = pair_xa ? x1 : x2;
            if (!(pair_xa || pair_ax) || x < 0 || x >= a.vocab) { o.status = SPECHUB_ST_TOKEN_RANGE; break; }
            const bool degenerate = !(Q.sx > 0.f);
            const float c = degenerate ? 0.f : Q.own / Q.sx;
            float crho = c * rho;
            const float qa = Q.own * invZq, rest = Q.sx * invZq;
            const int hubvec = hubtok >> 3, hubel = hubtok & 7;
            float px = prob_p(x);
            const float qx = prob_q(x);
            if (!a.beta && !a.rate) {
                // No probability is asked for: the first test needs scalars only, and if it accepts
                // the transport sums decide nothing.
                const bool acc1 = pair_xa ? accept_test(r1, px, qx, o.beta[0], true, o.status)
                                          : accept_test(r1, fmaxf(__fsub_rn(px, qx), 0.f), c * qx, o.beta[0], true, o.status);
                if (acc1) {
                    o.accept_idx = pair_xa ? 0 : 1;
                    o.token = x;
                    if (degenerate) o.status |= SPECHUB_ST_DEGENERATE_Q;
                    break;
                }
                o.status = 0;  // the full path below sets the flags again
            }
            // pass B: S1, S2, R over ids != a (Section 4, Appendix B.1)
            // (packed: the low lane takes the even ids of a vector, the high lane the odd ones)
            F2 s1, s2, rr;
            auto pass_b = [&]() {
            s1 = s2 = rr = f2_make(0.f, 0.f);
            const F2 k2 = f2_make(k, k), ncp2 = f2_make(-cP, -cP), ncq2 = f2_make(-cQ, -cQ);
            const F2 nrho2 = f2_make(-rho, -rho), ncrho2 = f2_make(-crho, -crho);
            auto vec_b = [&](int vi, const uint4 &cp, const uint4 &cq) {
                if (STATS) diff |= (cp.x ^ cq.x) | (cp.y ^ cq.y) | (cp.z ^ cq.z) | (cp.w ^ cq.w);
                unsigned wps[4] = {cp.x, cp.y, cp.z, cp.w}, wqs[4] = {cq.x, cq.y, cq.z, cq.w};
                if (vi == hubvec) {   // the hub's own pair is no part of the sums over y != a: -inf, mass 0
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        if (i == (hubel >> 1)) {
                            const unsigned keep = (hubel & 1) ? 0x0000ffffu : 0xffff0000u;
                            const unsigned ninf = (hubel & 1) ? 0xff800000u : 0x0000ff80u;
                            wps[i] = (wps[i] & keep) | ninf;
                            wqs[i] = (wqs[i] & keep) | ninf;
                        }
                    }
                }
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const F2 ep = f2_exp_word(wps[i], k2, ncp2), eq = f2_exp_word(wqs[i], k2, ncq2);
                    const F2 d = f2_fma(nrho2, eq, ep);       // Z_p (p - q)
                    const F2 m = f2_max0(d);
                    const F2 t = f2_fma(ncrho2, eq, m);       // Z_p (max(p - q, 0) - c q)
                    const F2 w = f2_max0(t);
                    s1 = f2_add(s1, f2_sub(m, d));            // max(-d, 0) = max(d, 0) - d, exactly
                    s2 = f2_add(s2, f2_sub(w, t));
                    rr = f2_add(rr, w);
                }
            };
            {
                // software pipeline: the next vector pair is in registers before this one is consumed.
                // This is the last use of both rows: the loads tell L2 to let these lines go first (one
                // CTA per row: 1.38 -> 1.30 ms on V = 128256; from draft statistics, where pass A also told
                // L2 to keep the target row's lines, 1.07 -> 1.02 ms.  Keep-hints on pass A of the kernel
                // that reads both rows twice cost it 7-13 %).
                uint64_t polf = 0;
                constexpr bool kHintB = STATS || CS == 1;
                if (kHintB) asm("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(polf));
                auto ldb = [&](const uint4 *ptr) { return kHintB ? ld_l2_hint(ptr, polf) : *ptr; };
                uint4 np = make_uint4(0, 0, 0, 0), nq = np;
                if (last_vi >= lo) { np = ldb(vp + last_vi); nq = ldb(vq + last_vi); }
#pragma unroll 1
                for (int vi = last_vi; vi >= lo; vi -= 32) {
                    const uint4 cp = np, cq = nq;
                    if (vi - 32 >= lo) { np = ldb(vp + vi - 32); nq = ldb(vq + vi - 32); }
                    vec_b(vi, cp, cq);
                }
            }
            };
            pass_b();
            if (STATS && rows_identical()) {
                crho = c;
                px = qx;
                pass_b();
            }
            float s1a, s1b, s2a, s2b, ra, rb;
            f2_get(s1, s1a, s1b);
            f2_get(s2, s2a, s2b);
            f2_get(rr, ra, rb);
            float acc[3] = {s1a + s1b, s2a + s2b, ra + rb};
            float part[3][CS];
            lean_row_sums<CS, 3, 0>(acc, part, sh);  // [2]
            // the sums are in units of 1 / Z_p; Rraw stays in them for the residual draw
            const float Rraw = acc[2];
            const float S1 = acc[0] * invZp, S2 = degenerate ? qa : acc[1] * invZp, R = Rraw * invZp;
            const float pa = prob_p(hubtok);
            const float hub_left = fmaxf(pa - S2, 0.f);
            o.rate[0] = fmaxf(rest - S1, 0.f) + fminf(pa, S2);
            o.rate[1] = (degenerate ? 0.f : fmaxf(qa - S2, 0.f)) + fminf(hub_left, S1);
            o.rate[2] = R;
            if (degenerate) o.status |= SPECHUB_ST_DEGENERATE_Q;
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
                o.accept_idx = -1;
                float base = 0.f;
                const int sel = (Rraw > 0.f) ? pick_part(part[2], CS, ures * Rraw, base) : -1;
                if (sel < 0) {
                    o.status |= SPECHUB_ST_ZERO_RESIDUAL;
                    draw_from_p();
                } else {
                    token_elsewhere = true;
                    if (sel == me) {
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
                        const int tok = block_sample3(g, wf, sh, ures * Rraw - base);
                        if (threadIdx.x == 0) a.token[r] = tok;
                    }
                }
            }
        } else {
            if (x1 < 0 || x1 >= a.vocab || x2 < 0 || x2 >= a.vocab) { o.status = SPECHUB_ST_TOKEN_RANGE; break; }
            if (!a.beta && !a.rate) {
                // no probability asked for: an accepted first draft needs no sum at all
                if (accept_test(r1, prob_p(x1), prob_q(x1), o.beta[0], true, o.status)) {
                    o.accept_idx = 0;
                    o.token = x1;
                    break;
                }
                o.status = 0;
            }
            // pass B: A1 = sum max(p - q, 0); RRSw also sums q outside x1 directly
            const int x1vec = x1 >> 3, x1el = x1 & 7;
            float dna = 0.f, dnb = 0.f;
            F2 a1;   // (packed: low lane = even ids of a vector, high lane = odd ids)
            const F2 k2 = f2_make(k, k), ncq2 = f2_make(-cQ, -cQ);
            F2 ncp2, nrho2;
            // RRSw: the next vector pair is loaded before the current one is consumed (measured:
            // 2.21 -> 2.03 ms on V = 128256; for RRS the plain loop unrolled twice is the faster one)
            constexpr bool PIPE = (METHOD == kRRSw);
            auto vec_b = [&](int vi, const uint4 &cp, const uint4 &cq) {
                if (STATS) diff |= (cp.x ^ cq.x) | (cp.y ^ cq.y) | (cp.z ^ cq.z) | (cp.w ^ cq.w);
                const unsigned wps[4] = {cp.x, cp.y, cp.z, cp.w}, wqs[4] = {cq.x, cq.y, cq.z, cq.w};
                F2 eq[4];   // e_q of the vector, by words
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    eq[i] = f2_exp_word(wqs[i], k2, ncq2);
                    a1 = f2_add(a1, f2_max0(f2_fma(nrho2, eq[i], f2_exp_word(wps[i], k2, ncp2))));
                }
                if (METHOD == kRRSw && !STATS) {   // (from draft statistics: sum_without, below)
                    float qq[8];
#pragma unroll
                    for (int i = 0; i < 4; ++i) f2_get(eq[i], qq[2 * i], qq[2 * i + 1]);
                    if (vi == x1vec) {
#pragma unroll
                        for (int i = 0; i < 8; ++i)
                            if (i == x1el) qq[i] = 0.f;
                    }
                    dna += (qq[0] + qq[1]) + (qq[2] + qq[3]);
                    dnb += (qq[4] + qq[5]) + (qq[6] + qq[7]);
                }
            };
            uint4 np = make_uint4(0, 0, 0, 0), nq = np;
            auto pass_b = [&](bool from_ring) {
            a1 = f2_make(0.f, 0.f); dna = 0.f; dnb = 0.f;
            ncp2 = f2_make(-cP, -cP); nrho2 = f2_make(-rho, -rho);
            if (RING && from_ring) {
#pragma unroll 1
                for (int c = R.nc - 1; c >= 0; --c) {
                    ring_wait(R);
                    const int v0 = lo + lane + c * kRingChunkVecs;
#pragma unroll
                    for (int j = kRingCh - 1; j >= 0; --j) {
                        uint4 x, y;
                        ring_load(R, j, lane, x, y);
                        if (j == 0) ring_release(R, lane);
                        if (v0 + j * 32 < hi) vec_b(v0 + j * 32, x, y);
                    }
                }
            } else {
                if (PIPE && last_vi >= lo) { np = vp[last_vi]; nq = vq[last_vi]; }
#pragma unroll(PIPE ? 1 : 2)
                for (int vi = last_vi; vi >= lo; vi -= 32) {
                    uint4 cp, cq;
                    if (PIPE) {
                        cp = np; cq = nq;
                        if (vi - 32 >= lo) { np = vp[vi - 32]; nq = vq[vi - 32]; }
                    } else {
                        cp = vp[vi]; cq = vq[vi];
                    }
                    vec_b(vi, cp, cq);
                }
            }
            };
            pass_b(true);
            if (STATS && rows_identical()) pass_b(false);
            float a1a, a1b;
            f2_get(a1, a1a, a1b);
            float acc[2] = {a1a + a1b, dna + dnb};
            float part2[2][CS];
            lean_row_sums<CS, 2, 0>(acc, part2, sh);  // [2]
            if (STATS && METHOD == kRRSw) acc[1] = sum_without(Q, rowq, x1, k);
            const float A1 = acc[0] * invZp, den = acc[1] * invZq;   // the sums are of exponentials
            const bool q1_zero = (METHOD == kRRSw) && !(den > 0.f);
            const float gq = (METHOD == kRRSw) ? (q1_zero ? 0.f : 1.f / den) : 1.f;
            const float A1g = A1 * gq;
            const float A1grho = A1g * rho;
            // pass C: mass of the residual after two rejections
            F2 w2 = f2_make(0.f, 0.f);
            const F2 nsc2 = f2_make(-A1grho, -A1grho);
            auto vec_c = [&](int vi, const uint4 &cp, const uint4 &cq) {
                const unsigned wps[4] = {cp.x, cp.y, cp.z, cp.w}, wqs[4] = {cq.x, cq.y, cq.z, cq.w};
                if (METHOD == kRRSw && vi == x1vec) {   // (one vector of the row) q1(x1) = 0: that lane's scale is 0
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        F2 nsc = nsc2;
                        if (i == (x1el >> 1)) nsc = (x1el & 1) ? f2_make(-A1grho, 0.f) : f2_make(0.f, -A1grho);
                        const F2 eq = f2_exp_word(wqs[i], k2, ncq2);
                        const F2 m = f2_max0(f2_fma(nrho2, eq, f2_exp_word(wps[i], k2, ncp2)));
                        w2 = f2_add(w2, f2_max0(f2_fma(nsc, eq, m)));
                    }
                    return;
                }
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const F2 eq = f2_exp_word(wqs[i], k2, ncq2);
                    const F2 m = f2_max0(f2_fma(nrho2, eq, f2_exp_word(wps[i], k2, ncp2)));
                    w2 = f2_add(w2, f2_max0(f2_fma(nsc2, eq, m)));
                }
            };
            if (RING) {
#pragma unroll 1
                for (int c = 0; c < R.nc; ++c) {
                    ring_wait(R);
                    const int v0 = lo + lane + c * kRingChunkVecs;
#pragma unroll
                    for (int j = 0; j < kRingCh; ++j) {
                        uint4 x, y;
                        ring_load(R, j, lane, x, y);
                        if (j == kRingCh - 1) ring_release(R, lane);
                        if (v0 + j * 32 < hi) vec_c(v0 + j * 32, x, y);
                    }
                }
            } else {
                uint64_t polc = 0;   // one CTA per row: the rows' last use, L2 may let these lines go first
                if (CS == 1) asm("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(polc));
                auto ldc = [&](const uint4 *ptr) { return CS == 1 ? ld_l2_hint(ptr, polc) : *ptr; };
                if (PIPE && lo + lane < hi) { np = ldc(vp + lo + lane); nq = ldc(vq + lo + lane); }
#pragma unroll(PIPE ? 1 : 2)
                for (int vi = lo + lane; vi < hi; vi += 32) {
                    uint4 cp, cq;
                    if (PIPE) {
                        cp = np; cq = nq;
                        if (vi + 32 < hi) { np = ldc(vp + vi + 32); nq = ldc(vq + vi + 32); }
                    } else {
                        cp = ldc(vp + vi); cq = ldc(vq + vi);
                    }
                    vec_c(vi, cp, cq);
                }
            }
            float w2a, w2b;
            f2_get(w2, w2a, w2b);
            float w2s[1] = {w2a + w2b};
            float part1[1][CS];
            lean_row_sums<CS, 1, 2>(w2s, part1, sh);  // [3]
            const float W2raw = w2s[0], W2 = W2raw * invZp;
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
                o.accept_idx = -1;
                float base = 0.f;
                const int sel = (A1 > 0.f && W2raw > 0.f) ? pick_part(part1[0], CS, ures * W2raw, base) : -1;
                if (sel < 0) {
                    o.status |= SPECHUB_ST_ZERO_RESIDUAL;
                    draw_from_p();
                } else {
                    token_elsewhere = true;
                    if (sel == me) {
                        if (threadIdx.x < g.nwarps) sh.mass[threadIdx.x] = sh.acc[0][threadIdx.x];
                        __syncthreads();
                        auto wf = [&](int vi, float(&w)[8]) {
                            float fp[8], fq[8];
                            unpack_bf16x8(vp[vi], fp);
                            unpack_bf16x8(vq[vi], fq);
#pragma unroll
                            for (int i = 0; i < 8; ++i) {
                                float d, t;
                                const float s = (METHOD == kRRSw && vi * 8 + i == x1) ? 0.f : A1grho;
                                lean_terms(lean_exp(fp[i], k, cP), lean_exp(fq[i], k, cQ), rho, s, d, t);
                                w[i] = fmaxf(t, 0.f);
                            }
                        };
                        const int tok = block_sample3(g, wf, sh, ures * W2raw - base);
                        if (threadIdx.x == 0) a.token[r] = tok;
                    }
                }
            }
        }
    } while (false);
    if (RING) {
        // no copy may be on its way into this CTA's shared memory when it ends; a stage that never arrived
        // (every wait is bounded) is reported with the row
        ring_drain(R);
        if (__syncthreads_or(R.timed_out)) o.status |= SPECHUB_ST_INTERNAL;
    }
    if (writer) {
        a.accept_idx[r] = o.accept_idx;
        if (!token_elsewhere) a.token[r] = o.token;
        if (a.hub) a.hub[r] = o.hub;
        if (a.beta) { a.beta[2 * r] = o.beta[0]; a.beta[2 * r + 1] = o.beta[1]; }
        if (a.rate) { a.rate[3 * r] = o.rate[0]; a.rate[3 * r + 1] = o.rate[1]; a.rate[3 * r + 2] = o.rate[2]; }
        if (a.status) a.status[r] = o.status;
    }
    if (CS > 1) RowGroup<CS>::sync();  // no CTA leaves while another may still read its shared memory
}

// ------------------------------------------------------------------------------------------------
// Draft step (Section 4 / Algorithm 3 for SpecHub; Algorithm 1 for RRS, RRSw).
// ------------------------------------------------------------------------------------------------
template <int THREADS, int CS>
__global__ void __launch_bounds__(THREADS, 1024 / THREADS) lean_draft_kernel(RowArgs a, int method) {
    __shared__ LeanShared sh;
    const int me = RowGroup<CS>::rank();
    const long long r = blockIdx.x / CS;
    const int b = static_cast<int>(r / a.nodes), n = static_cast<int>(r % a.nodes);
    const __nv_bfloat16 *rowq = static_cast<const __nv_bfloat16 *>(a.draft) + b * a.stride_seq + n * a.stride_node;
    const uint4 *vq = reinterpret_cast<const uint4 *>(rowq);
    const Geo g = make_geo(a.vocab, 8, CS, me);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int lo = g.seg_lo(warp), hi = g.seg_hi(warp);
    const float k = kLog2e / temperature_of(a, b);
    const float u1 = a.uniforms[r * 5 + 0], u2 = a.uniforms[r * 5 + 1];
    const bool writer = (me == 0 && threadIdx.x == 0);

    LeanAcc tq, unused;
    lean_pass_a<false>(vq, vq, lo, hi, lane, k, tq, unused);
    {
        ArgMaxSum q, unusedq;
        lean_reduce2<false>(tq, unused, vq, vq, lo, hi, k, sh, q, unusedq);
        if (threadIdx.x == 0) { sh.x_ml[0] = q.ml; sh.x_sx[0] = q.sx; sh.x_idx[0] = q.idx; sh.x_tok = -3; }
    }
    RowGroup<CS>::sync();  // [1]
    RowStat Q;
    merge_slices<CS>(sh, 0, k, Q);
    const float Zq = Q.sx + Q.own;
    uint32_t st = 0;
    const bool bad = !(Q.ml > neg_inf()) || !finite_pos(Zq) || !(Q.ml < -neg_inf());
    const int hubtok = bad ? -1 : Q.idx;
    if (writer) void_draft_stat(a, r);
    if (bad) {
        if (writer) {
            a.draft_tokens_out[2 * r] = -1; a.draft_tokens_out[2 * r + 1] = -1;
            if (a.hub) a.hub[r] = -1;
            if (a.draft_prob) { a.draft_prob[2 * r] = 0.f; a.draft_prob[2 * r + 1] = 0.f; }
            if (a.status) a.status[r] = SPECHUB_ST_NONFINITE;
        }
    } else {
        // x1 ~ q.  The CTA whose slice holds the target draws it and tells the others.
        const int t1 = lean_sample_row<CS>(g, rowq, k, Q, me, -1, u1, 0, sh);
        int x1 = t1;
        if (CS > 1) {
            if (t1 != -2 && threadIdx.x == 0) sh.x_tok = t1;
            RowGroup<CS>::sync();  // [2]
            x1 = -1;
#pragma unroll
            for (int c = 0; c < CS; ++c) {
                const int v = RowGroup<CS>::peer(&sh, c)->x_tok;
                if (v != -3) x1 = v;
            }
        }
        float prob0 = 0.f, prob1 = 0.f;
        bool x2_elsewhere = false;  // x2 (and its probability) written by the CTA that draws it
        int x2 = -1;
        if (method == kSpecHub) {
            prob0 = Q.own / Zq;
            if (x1 != hubtok) {
                x2 = hubtok;
                prob1 = ex2(fmaf(load_one<__nv_bfloat16>(rowq, x1), k, -Q.C)) / Zq;
            } else if (!(Q.sx > 0.f)) {
                x2 = (hubtok == 0) ? 1 : 0;
                st |= SPECHUB_ST_DEGENERATE_Q;
            } else {
                const int t2 = lean_sample_row<CS>(g, rowq, k, Q, me, hubtok, u2, 0, sh);
                x2_elsewhere = true;
                if (t2 != -2 && threadIdx.x == 0) {
                    a.draft_tokens_out[2 * r + 1] = t2;
                    if (a.draft_prob)
                        a.draft_prob[2 * r + 1] = prob0 * ex2(fmaf(load_one<__nv_bfloat16>(rowq, t2), k, -Q.C)) / Q.sx;
                }
            }
        } else if (method == kRRS) {
            const int t2 = lean_sample_row<CS>(g, rowq, k, Q, me, -1, u2, 0, sh);
            x2_elsewhere = true;
            if (t2 != -2 && threadIdx.x == 0) a.draft_tokens_out[2 * r + 1] = t2;
        } else {
            // q with q(x1) set to 0.  The mass of the slice that holds x1 is its sum minus x1's term:
            // unless x1 is that slice's argmax (which the published sum already leaves out), the
            // argmax's own term stays in, so at most half of the sum cancels.
            const int per = (g.nvec + CS - 1) / CS;
            const int ox = min((x1 >> 3) / per, CS - 1);
            const float lx1 = load_one<__nv_bfloat16>(rowq, x1);
            float m[CS];
            float total = 0.f;
#pragma unroll
            for (int c = 0; c < CS; ++c) {
                m[c] = slice_mass<CS>(sh, 0, Q, c, x1, k);
                if (c == ox && RowGroup<CS>::peer(&sh, c)->x_idx[0] != x1)
                    m[c] = fmaxf(m[c] - ex2(__fmaf_rn(lx1, k, -Q.C)), 0.f);
                total += m[c];
            }
            x2_elsewhere = true;
            float base = 0.f;
            const int sel = (total > 0.f) ? pick_part(m, CS, u2 * total, base) : -1;
            if (sel < 0) {
                st |= SPECHUB_ST_DEGENERATE_Q;
                if (writer) a.draft_tokens_out[2 * r + 1] = (x1 == 0) ? 1 : 0;
            } else if (sel == me) {
                const int t2 = lean_sample_slice(g, rowq, k, Q, x1, u2 * total - base, 0, sh);
                if (threadIdx.x == 0) a.draft_tokens_out[2 * r + 1] = t2;
            }
        }
        if (writer) {
            a.draft_tokens_out[2 * r] = x1;
            if (!x2_elsewhere) a.draft_tokens_out[2 * r + 1] = x2;
            if (a.hub) a.hub[r] = (method == kSpecHub) ? hubtok : -1;
            if (a.draft_prob) {
                a.draft_prob[2 * r] = prob0;
                if (!x2_elsewhere) a.draft_prob[2 * r + 1] = prob1;
            }
            if (a.status) a.status[r] = st;
        }
    }
    if (CS > 1) RowGroup<CS>::sync();
}

// ------------------------------------------------------------------------------------------------
// Draft step, one CTA per row (checkpointed pass A and sub-block sampler above).
// ------------------------------------------------------------------------------------------------
template <int THREADS>
__global__ void __launch_bounds__(THREADS, 1024 / THREADS) lean_draft_ck_kernel(RowArgs a, int method) {
    __shared__ LeanCkShared sh;
    const long long r = blockIdx.x;
    const int b = static_cast<int>(r / a.nodes), n = static_cast<int>(r % a.nodes);
    const __nv_bfloat16 *rowq = static_cast<const __nv_bfloat16 *>(a.draft) + b * a.stride_seq + n * a.stride_node;
    const uint4 *vq = reinterpret_cast<const uint4 *>(rowq);
    const Geo g = make_geo(a.vocab, 8);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int lo = g.seg_lo(warp), hi = g.seg_hi(warp);
    const float k = kLog2e / temperature_of(a, b);
    const float u1 = a.uniforms[r * 5 + 0], u2 = a.uniforms[r * 5 + 1];
    const int CK = lean_ck_interval(g);

    LeanAcc tq, unused;
    unused.m2 = 0xff80ff80u; unused.s = 0.f; unused.c = 0.f;
    lean_pass_a_ck(vq, lo, hi, lane, k, CK, tq, sh.cks[warp], sh.ckc[warp]);
    {
        ArgMaxSum q, unusedq;
        lean_reduce2<false>(tq, unused, vq, vq, lo, hi, k, sh, q, unusedq);
        if (threadIdx.x == 0) { sh.x_ml[0] = q.ml; sh.x_sx[0] = q.sx; sh.x_idx[0] = q.idx; }
    }
    __syncthreads();
    RowStat Q;
    merge_slices<1>(sh, 0, k, Q);
    const float Zq = Q.sx + Q.own;
    uint32_t st = 0;
    int x1 = -1, x2 = -1, hubtok = -1;
    float prob0 = 0.f, prob1 = 0.f;
    if (!(Q.ml > neg_inf()) || !finite_pos(Zq) || !(Q.ml < -neg_inf())) {
        st = SPECHUB_ST_NONFINITE;
    } else {
        hubtok = Q.idx;
        x1 = lean_ck_sample(g, rowq, k, Q.C, CK, -1, u1, sh);
        if (method == kSpecHub) {
            prob0 = Q.own / Zq;
            if (x1 != hubtok) {
                x2 = hubtok;
                prob1 = ex2(fmaf(load_one<__nv_bfloat16>(rowq, x1), k, -Q.C)) / Zq;
            } else if (!(Q.sx > 0.f)) {
                x2 = (hubtok == 0) ? 1 : 0;
                st |= SPECHUB_ST_DEGENERATE_Q;
            } else {
                x2 = lean_ck_sample(g, rowq, k, Q.C, CK, hubtok, u2, sh);
                prob1 = prob0 * ex2(fmaf(load_one<__nv_bfloat16>(rowq, x2), k, -Q.C)) / Q.sx;
            }
        } else if (method == kRRS) {
            x2 = lean_ck_sample(g, rowq, k, Q.C, CK, -1, u2, sh);
        } else {
            x2 = lean_ck_sample(g, rowq, k, Q.C, CK, x1, u2, sh);
            if (x2 < 0) {   // nothing left once x1 is removed
                x2 = (x1 == 0) ? 1 : 0;
                st |= SPECHUB_ST_DEGENERATE_Q;
            }
        }
    }
    if (threadIdx.x == 0) {
        if (a.draft_stats_out) {
            DraftStat ds;
            ds.ml = Q.ml; ds.sx = Q.sx; ds.idx = Q.idx; ds.tag = kDraftStatTag ^ __float_as_uint(k);
            static_cast<DraftStat *>(a.draft_stats_out)[r] = ds;
        }
        a.draft_tokens_out[2 * r] = x1;
        a.draft_tokens_out[2 * r + 1] = x2;
        if (a.hub) a.hub[r] = (method == kSpecHub) ? hubtok : -1;
        if (a.draft_prob) { a.draft_prob[2 * r] = prob0; a.draft_prob[2 * r + 1] = prob1; }
        if (a.status) a.status[r] = st;
    }
}

}  // namespace spechub
