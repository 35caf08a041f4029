// Device-side building blocks shared by the SpecHub / RRS kernels (sm_100a).
//
// Conventions used throughout:
//   * p = target, q = draft (Section 2 of arXiv 2411.05289); a = argmax q = hub.
//   * A row of V logits is cut into 16-byte vectors (8 bf16 or 4 fp32).  Warp w
//     of a CTA owns a contiguous run of `seg` vectors; its lanes take
//     consecutive vectors, so every warp-level load is one contiguous 512-byte
//     request and every partial sum belongs to a contiguous range of token
//     ids.  Inverse-CDF sampling needs exactly that: the per-warp partial sums
//     are the coarse CDF, and only the selected warp rescans its range.
//   * Exponentials are taken in base 2: with k = log2(e)/T and c = k * max
//     logit, e(y) = 2^(k*l(y) - c) from one FMA and one ex2.approx.
//   * All reductions have a fixed order (lane -> warp butterfly -> warps in
//     ascending order), so results are run-to-run deterministic.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace spechub {

constexpr int kMaxWarps = 32;
constexpr float kLog2e = 1.4426950408889634f;
constexpr unsigned kFull = 0xffffffffu;

__device__ __forceinline__ float neg_inf() { return __int_as_float(0xff800000); }

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

template <typename LT> struct VecOf;
template <> struct VecOf<float> { static constexpr int W = 4; };
template <> struct VecOf<__nv_bfloat16> { static constexpr int W = 8; };

// Vector `vi` of a row as floats; ids >= V read as -inf (probability 0).
template <typename LT, bool ALIGNED>
__device__ __forceinline__ void load_vec(const LT *__restrict__ row, int vi, int V,
                                         float (&out)[VecOf<LT>::W]);

template <>
__device__ __forceinline__ void load_vec<float, true>(const float *__restrict__ row, int vi, int V,
                                                      float (&out)[4]) {
    const int base = vi * 4;
    if (base + 4 <= V) {
        const float4 v = *reinterpret_cast<const float4 *>(row + base);
        out[0] = v.x; out[1] = v.y; out[2] = v.z; out[3] = v.w;
    } else {
#pragma unroll
        for (int i = 0; i < 4; ++i) out[i] = (base + i < V) ? row[base + i] : neg_inf();
    }
}
template <>
__device__ __forceinline__ void load_vec<float, false>(const float *__restrict__ row, int vi, int V,
                                                       float (&out)[4]) {
    const int base = vi * 4;
#pragma unroll
    for (int i = 0; i < 4; ++i) out[i] = (base + i < V) ? row[base + i] : neg_inf();
}

__device__ __forceinline__ float bf16_bits_to_float(unsigned short h) {
    return __uint_as_float(static_cast<unsigned>(h) << 16);
}

template <>
__device__ __forceinline__ void load_vec<__nv_bfloat16, true>(const __nv_bfloat16 *__restrict__ row,
                                                              int vi, int V, float (&out)[8]) {
    const int base = vi * 8;
    if (base + 8 <= V) {
        const uint4 v = *reinterpret_cast<const uint4 *>(row + base);
        out[0] = __uint_as_float(v.x << 16); out[1] = __uint_as_float(v.x & 0xffff0000u);
        out[2] = __uint_as_float(v.y << 16); out[3] = __uint_as_float(v.y & 0xffff0000u);
        out[4] = __uint_as_float(v.z << 16); out[5] = __uint_as_float(v.z & 0xffff0000u);
        out[6] = __uint_as_float(v.w << 16); out[7] = __uint_as_float(v.w & 0xffff0000u);
    } else {
        const unsigned short *r = reinterpret_cast<const unsigned short *>(row);
#pragma unroll
        for (int i = 0; i < 8; ++i) out[i] = (base + i < V) ? bf16_bits_to_float(r[base + i]) : neg_inf();
    }
}
template <>
__device__ __forceinline__ void load_vec<__nv_bfloat16, false>(const __nv_bfloat16 *__restrict__ row,
                                                               int vi, int V, float (&out)[8]) {
    const int base = vi * 8;
    const unsigned short *r = reinterpret_cast<const unsigned short *>(row);
#pragma unroll
    for (int i = 0; i < 8; ++i) out[i] = (base + i < V) ? bf16_bits_to_float(r[base + i]) : neg_inf();
}

template <typename LT>
__device__ __forceinline__ float load_one(const LT *row, int y);
template <> __device__ __forceinline__ float load_one<float>(const float *row, int y) { return row[y]; }
template <>
__device__ __forceinline__ float load_one<__nv_bfloat16>(const __nv_bfloat16 *row, int y) {
    return bf16_bits_to_float(reinterpret_cast<const unsigned short *>(row)[y]);
}

// How a row is cut over the warps of a CTA.
// v0 / nloc describe the part of the row this CTA works on (the whole row unless the row is split
// over the CTAs of a cluster); vector indices are always absolute.
struct Geo {
    int V, nvec, seg, nwarps, v0, nloc;
    __device__ __forceinline__ int seg_lo(int w) const { return v0 + min(w * seg, nloc); }
    __device__ __forceinline__ int seg_hi(int w) const { return v0 + min((w + 1) * seg, nloc); }
    __device__ __forceinline__ bool holds_vec(int vi) const { return vi >= v0 && vi < v0 + nloc; }
    __device__ __forceinline__ int warp_of_vec(int vi) const { return (vi - v0) / seg; }
};
__device__ __forceinline__ Geo make_geo(int V, int VW, int parts = 1, int part = 0) {
    Geo g;
    g.V = V;
    g.nvec = (V + VW - 1) / VW;
    g.nwarps = blockDim.x >> 5;
    const int per = (g.nvec + parts - 1) / parts;
    g.v0 = min(part * per, g.nvec);
    g.nloc = min(per, g.nvec - g.v0);
    g.seg = max(1, (g.nloc + g.nwarps - 1) / g.nwarps);
    return g;
}

// ---- running (max, sum of exponentials) -------------------------------------------------------
// s = sum 2^(k*l - c), c = k*ml (c = 0 while nothing finite was seen).
struct MaxSum {
    float ml, c, s;
    __device__ __forceinline__ void init() { ml = neg_inf(); c = 0.f; s = 0.f; }
};
// (the product is rounded on its own: were it contracted into a later subtraction, two copies of the
// same code could disagree in the last bit)
__device__ __forceinline__ float shift_of(float ml, float k) { return ml > neg_inf() ? __fmul_rn(ml, k) : 0.f; }
// 2^(c_from - c_to) for a partial whose maximum is ml_from; an empty partial (no finite
// logit yet) carries no mass, whatever the target shift is.
__device__ __forceinline__ float rescale(float ml_from, float c_from, float c_to) {
    return ml_from > neg_inf() ? ex2(c_from - c_to) : 0.f;
}

template <int W>
__device__ __forceinline__ void maxsum_push(MaxSum &st, const float (&v)[W], float k) {
    float vmax = v[0];
#pragma unroll
    for (int i = 1; i < W; ++i) vmax = fmaxf(vmax, v[i]);
    if (vmax > st.ml) {
        const float cn = __fmul_rn(vmax, k);
        st.s *= rescale(st.ml, st.c, cn);
        st.c = cn;
        st.ml = vmax;
    }
    float acc = 0.f;
#pragma unroll
    for (int i = 0; i < W; ++i) acc += ex2(fmaf(v[i], k, -st.c));
    st.s += acc;
}
__device__ __forceinline__ MaxSum maxsum_merge(const MaxSum &a, const MaxSum &b, float k) {
    MaxSum r;
    r.ml = fmaxf(a.ml, b.ml);
    r.c = shift_of(r.ml, k);
    r.s = a.s * rescale(a.ml, a.c, r.c) + b.s * rescale(b.ml, b.c, r.c);
    return r;
}
__device__ __forceinline__ MaxSum maxsum_warp(MaxSum st, float k) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        MaxSum ot;
        ot.ml = __shfl_xor_sync(kFull, st.ml, o);
        ot.c = __shfl_xor_sync(kFull, st.c, o);
        ot.s = __shfl_xor_sync(kFull, st.s, o);
        st = maxsum_merge(st, ot, k);
    }
    return st;
}

// ---- running (max, argmax, sum of exponentials EXCLUDING the argmax element) ------------------
// The hub's complement mass 1 - q(a) has to be summed directly: subtracting the
// hub's own term from the full sum cancels when q is peaked.  sx holds every
// element except the first occurrence of the maximum, relative to c = k*ml.
struct ArgMaxSum {
    float ml, c, sx;
    int idx;
    __device__ __forceinline__ void init() { ml = neg_inf(); c = 0.f; sx = 0.f; idx = 0x7fffffff; }
    // The argmax's own term on this scale, 2^(k ml - c).  c is k*ml rounded to fp32, so this is
    // 2^(rounding residual): 1 to within 1e-6 while |c| < 16, but 1 + 2e-5 at |c| = 500 (a large
    // maximum logit or a small temperature); taking it as 1 would put that error into Z.
    __device__ __forceinline__ float own(float k) const { return ml > neg_inf() ? ex2(fmaf(ml, k, -c)) : 0.f; }
};
template <int W>
__device__ __forceinline__ void argmaxsum_push(ArgMaxSum &st, const float (&v)[W], int base, float k) {
    float vmax = v[0];
#pragma unroll
    for (int i = 1; i < W; ++i) vmax = fmaxf(vmax, v[i]);
    float acc = 0.f;
    if (vmax > st.ml) {  // a new maximum: the old one becomes an ordinary element
        int pos = 0;
#pragma unroll
        for (int i = W - 1; i >= 0; --i) pos = (v[i] == vmax) ? i : pos;
        const float cn = __fmul_rn(vmax, k);
        st.sx = __fmul_rn(__fadd_rn(st.sx, st.own(k)), rescale(st.ml, st.c, cn));
        st.c = cn;
        st.ml = vmax;
        st.idx = base + pos;
#pragma unroll
        for (int i = 0; i < W; ++i) acc += (i == pos) ? 0.f : ex2(fmaf(v[i], k, -st.c));
    } else {
#pragma unroll
        for (int i = 0; i < W; ++i) acc += ex2(fmaf(v[i], k, -st.c));
    }
    st.sx += acc;
}
// own term of a maximum logit ml on its own scale shift_of(ml, k)
__device__ __forceinline__ float own_term(float ml, float k) {
    return ml > neg_inf() ? ex2(fmaf(ml, k, -shift_of(ml, k))) : 0.f;
}
__device__ __forceinline__ ArgMaxSum argmaxsum_merge(const ArgMaxSum &a, const ArgMaxSum &b, float k) {
    const bool b_wins = (b.ml > a.ml) || (b.ml == a.ml && b.idx < a.idx);
    const ArgMaxSum &w = b_wins ? b : a;
    const ArgMaxSum &l = b_wins ? a : b;
    ArgMaxSum r = w;
    // roundings pinned (no contraction into an FMA): the target and the draft row go through separately
    // inlined copies of this code and must give the same bits when the rows are equal
    r.sx = __fadd_rn(w.sx, __fmul_rn(__fadd_rn(l.sx, l.own(k)), rescale(l.ml, l.c, w.c)));
    return r;
}
__device__ __forceinline__ ArgMaxSum argmaxsum_warp(ArgMaxSum st, float k) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        ArgMaxSum ot;
        ot.ml = __shfl_xor_sync(kFull, st.ml, o);
        ot.c = __shfl_xor_sync(kFull, st.c, o);
        ot.sx = __shfl_xor_sync(kFull, st.sx, o);
        ot.idx = __shfl_xor_sync(kFull, st.idx, o);
        st = argmaxsum_merge(st, ot, k);
    }
    return st;
}

__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(kFull, x, o);
    return x;
}

// ---- inverse-CDF draw over a row, CTA-wide ----------------------------------------------------
// mass[w] (shared memory) = total weight of warp w's range.  weights(vi, w[]) must
// return the VW weights of vector vi (0 for ids that carry no mass or lie past V)
// and must be the same arithmetic that produced mass[].  Returns to every thread
// the lowest id whose inclusive prefix exceeds u * total; when rounding leaves
// none inside the selected range, the last id with positive weight there; -1 when
// the total is 0.  Must be called by all threads of the CTA.
// block_sample_at takes the target prefix t itself (a draw whose total spans more than this CTA's
// range); block_sample draws with u * (this range's total).
template <int VW, class WF>
__device__ int block_sample_at(const Geo &g, WF weights, const float *mass, float t, int *sh_tok) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    int wsel = -1, lastw = -1;
    float base = 0.f, lastbase = 0.f, run = 0.f;
    for (int w = 0; w < g.nwarps; ++w) {
        const float m = mass[w];
        if (m > 0.f) {
            lastw = w;
            lastbase = run;
            if (wsel < 0 && run + m > t) { wsel = w; base = run; }
        }
        run += m;
    }
    if (lastw < 0) return -1;
    if (wsel < 0) { wsel = lastw; base = lastbase; }
    if (warp == wsel) {
        const float tt = t - base;
        float prefix = 0.f;
        int found = -1, lastpos = -1;
        for (int v0 = g.seg_lo(warp); v0 < g.seg_hi(warp); v0 += 32) {
            const int vi = v0 + lane;
            float w[VW];
            if (vi < g.seg_hi(warp)) {
                weights(vi, w);
            } else {
#pragma unroll
                for (int i = 0; i < VW; ++i) w[i] = 0.f;
            }
            float lsum = 0.f;
            int lp = -1;
#pragma unroll
            for (int i = 0; i < VW; ++i) {
                lsum += w[i];
                if (w[i] > 0.f) lp = vi * VW + i;
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
                    for (int i = 0; i < VW; ++i) {
                        acc += w[i];
                        if (w[i] > 0.f) {
                            lastin = vi * VW + i;
                            if (cand < 0 && acc > tt) cand = lastin;
                        }
                    }
                    if (cand < 0) cand = lastin;
                }
                found = __shfl_sync(kFull, cand, L);
                break;
            }
            // remember the last id with mass in case rounding pushes tt past the range
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) lp = max(lp, __shfl_xor_sync(kFull, lp, o));
            lastpos = max(lastpos, lp);
            prefix += tot;
        }
        if (found < 0) found = lastpos;
        if (lane == 0) *sh_tok = found;
    }
    __syncthreads();
    const int tok = *sh_tok;
    __syncthreads();
    return tok;
}

template <int VW, class WF>
__device__ int block_sample(const Geo &g, WF weights, const float *mass, float u, int *sh_tok) {
    float total = 0.f;
    for (int w = 0; w < g.nwarps; ++w) total += mass[w];
    if (!(total > 0.f)) return -1;
    return block_sample_at<VW>(g, weights, mass, u * total, sh_tok);
}

}  // namespace spechub
