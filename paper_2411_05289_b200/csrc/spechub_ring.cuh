// Per-warp rings of bulk copies (cp.async.bulk, global -> shared, completion on an mbarrier) that feed
// the passes of the streaming verification kernels.
//
// A warp owns a contiguous range [lo, hi) of 16-byte vectors of the target row and of the draft row and
// goes over it once per pass, forwards or backwards.  The passes of a row form one stream of chunks
// (kRingCh vectors per lane of each row): lane 0 keeps kRingStages chunks of that stream in flight, also
// across the boundary between two passes, so that the loads of a pass are under way while the warp still
// reduces the previous one.  The warp that consumes a stage is the one that refills it: no barrier other
// than the stage's own mbarrier and a __syncwarp() is involved, and no other warp is ever waited for.
//
// Vector v of a chunk goes to lane v % 32, as in the kernels that load from global memory directly, so a
// thread sees the same vectors in the same order and every sum keeps its association.
//
// Every wait is bounded: a stage that does not arrive within kRingSpinLimit polls marks the ring as timed
// out, the kernel finishes the row and reports SPECHUB_ST_INTERNAL for it.
#pragma once

#include <cstdint>

namespace spechub {

constexpr int kRingCh = 3;       // vectors per lane, row and stage (measured: 1 / 2 / 3 / 4 -> 1.60 / 1.31 / 1.23 / 1.23 ms)
constexpr int kRingStages = 2;   // (2 / 3 stages at 2 vectors: 1.31 / 1.34 ms)
constexpr int kRingChunkVecs = kRingCh * 32;
constexpr int kRingStageBytes = 2 * kRingChunkVecs * 16;          // target half, draft half
constexpr int kRingWarpBytes = kRingStages * kRingStageBytes;     // 6 KB
constexpr unsigned kRingSpinLimit = 1u << 22;

__device__ __forceinline__ uint32_t ring_saddr(const void *p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

struct WarpRing {
    uint32_t data;   // shared-window address of this warp's stages
    uint32_t bars;   // shared-window address of its kRingStages mbarriers
    const uint4 *vp, *vq;
    int lo, hi;
    int nc;          // chunks per pass
    int ng;          // chunks of the whole stream
    int g;           // next chunk of the stream to consume
    int issued;      // chunks requested so far (the same in every lane; lane 0 issues)
    int ipass, ileft, iv0, istep;   // lane 0: the next chunk to request (its pass, chunks left in it, first vector, stride)
    unsigned back;   // bit i: pass i runs from the top of the range down
    bool timed_out;
};

// lane 0: request chunk `R.issued` of the stream
__device__ __forceinline__ void ring_issue(WarpRing &R) {
    const uint32_t bytes = static_cast<uint32_t>(min(kRingChunkVecs, R.hi - R.iv0)) * 16u;
    const uint32_t st = static_cast<uint32_t>(R.issued) & (kRingStages - 1);
    const uint32_t bar = R.bars + 8u * st, dst = R.data + st * kRingStageBytes;
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(2u * bytes) : "memory");
    asm volatile("cp.async.bulk.shared::cta.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(R.vp + R.iv0), "r"(bytes), "r"(bar) : "memory");
    asm volatile("cp.async.bulk.shared::cta.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst + kRingChunkVecs * 16), "l"(R.vq + R.iv0), "r"(bytes), "r"(bar) : "memory");
    // the chunk after this one: the next of this pass, or the first of the next pass
    if (--R.ileft > 0) R.iv0 += R.istep;
    else {
        ++R.ipass;
        R.ileft = R.nc;
        const bool down = (R.back >> R.ipass) & 1u;
        R.istep = down ? -kRingChunkVecs : kRingChunkVecs;
        R.iv0 = down ? R.lo + (R.nc - 1) * kRingChunkVecs : R.lo;
    }
}

// All lanes of the warp.  `data` / `bars`: this warp's kRingWarpBytes (16-byte aligned) and its kRingStages
// mbarriers in shared memory.  `passes` passes over [lo, hi); bit i of `back` makes pass i run backwards.
__device__ __forceinline__ void ring_begin(WarpRing &R, void *data, uint64_t *bars, const uint4 *vp, const uint4 *vq,
                                           int lo, int hi, int passes, unsigned back, int lane) {
    R.data = ring_saddr(data); R.bars = ring_saddr(bars);
    R.vp = vp; R.vq = vq; R.lo = lo; R.hi = hi;
    R.nc = hi > lo ? (hi - lo + kRingChunkVecs - 1) / kRingChunkVecs : 0;
    R.ng = passes * R.nc;
    R.g = 0; R.issued = 0; R.back = back; R.timed_out = false;
    R.ipass = 0; R.ileft = R.nc;
    R.istep = (back & 1u) ? -kRingChunkVecs : kRingChunkVecs;
    R.iv0 = (back & 1u) ? lo + (R.nc - 1) * kRingChunkVecs : lo;
    if (lane == 0) {
#pragma unroll
        for (int s = 0; s < kRingStages; ++s)
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(R.bars + 8u * s) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncwarp();
#pragma unroll
    for (int s = 0; s < kRingStages; ++s) {
        if (R.issued < R.ng) {
            if (lane == 0) ring_issue(R);
            ++R.issued;
        }
    }
}

// wait (bounded) until chunk R.g has arrived
__device__ __forceinline__ void ring_wait(WarpRing &R) {
    static_assert((kRingStages & (kRingStages - 1)) == 0, "stage index by mask");
    const uint32_t bar = R.bars + 8u * (static_cast<uint32_t>(R.g) & (kRingStages - 1));
    const uint32_t parity = (static_cast<uint32_t>(R.g) / kRingStages) & 1u;
    unsigned polls = 0;
    for (;;) {
        uint32_t ok;
        asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
                     : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
        if (ok) break;
        if (++polls > kRingSpinLimit) { R.timed_out = true; break; }
    }
}

// vector j (0 .. kRingCh - 1) of this lane in chunk R.g: target and draft
__device__ __forceinline__ void ring_load(const WarpRing &R, int j, int lane, uint4 &x, uint4 &y) {
    const uint32_t a = R.data + (static_cast<uint32_t>(R.g) & (kRingStages - 1)) * kRingStageBytes +
                       static_cast<uint32_t>(j * 32 + lane) * 16u;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(x.x), "=r"(x.y), "=r"(x.z), "=r"(x.w) : "r"(a));
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(y.x), "=r"(y.y), "=r"(y.z), "=r"(y.w) : "r"(a + kRingChunkVecs * 16));
}

// every lane has read chunk R.g: its stage takes the next chunk of the stream
__device__ __forceinline__ void ring_release(WarpRing &R, int lane) {
    __syncwarp();
    if (R.issued < R.ng) {
        if (lane == 0) {
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            ring_issue(R);
        }
        ++R.issued;
    }
    ++R.g;
}

// before the CTA ends or gives the stream up: no copy may still be on its way into shared memory
__device__ __forceinline__ void ring_drain(WarpRing &R) {
    while (R.g < R.issued) { ring_wait(R); ++R.g; }
    R.ng = R.issued;
}

}  // namespace spechub
