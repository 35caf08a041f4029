// C ABI of the library (see include/spechub.h): host-side argument checks and
// kernel launches.  Nothing here allocates or synchronises.
#include <cuda_runtime.h>
#include <math.h>
#include <stdlib.h>

#include <mutex>

#include "spechub.h"
#include "spechub_common.cuh"
#include "spechub_stream.cuh"
#include "spechub_lean.cuh"
#include "spechub_kary.cuh"
#include "spechub_fused.cuh"
#include "spechub_resident.cuh"
#include "spechub_resident_kary.cuh"
#include "spechub_shard.cuh"
#include "spechub_shard_rrs.cuh"

extern "C" size_t spechub_draft_stats_bytes(const spechub_desc *desc);

namespace {

using namespace spechub;

int check_desc(const spechub_desc *d) {
    if (!d) return SPECHUB_ERR_NULL;
    if (d->struct_size != sizeof(spechub_desc) || d->version != SPECHUB_ABI_VERSION)
        return SPECHUB_ERR_VERSION;
    if (d->batch < 0 || d->nodes < 1 || d->vocab < 2 || d->k < 2 || d->k > SPECHUB_MAX_K || d->levels < 1)
        return SPECHUB_ERR_SHAPE;
    if (d->dtype != SPECHUB_F32 && d->dtype != SPECHUB_BF16) return SPECHUB_ERR_DTYPE;
    if (d->stride_node < d->vocab) return SPECHUB_ERR_STRIDE;
    if (d->nodes > 1 && d->stride_seq < d->stride_node * (int64_t)(d->nodes - 1) + d->vocab)
        return SPECHUB_ERR_STRIDE;
    if (d->nodes == 1 && d->batch > 1 && d->stride_seq < d->vocab) return SPECHUB_ERR_STRIDE;
    if (!d->temperature_per_seq && !(d->temperature > 0.f && isfinite(d->temperature)))
        return SPECHUB_ERR_TEMPERATURE;
    const uint32_t split = d->flags & 7u;
    if ((d->flags & ~15u) != 0 || (split & (split - 1)) != 0) return SPECHUB_ERR_SHAPE;
    if ((d->flags & SPECHUB_FLAG_RESIDENT) && split) return SPECHUB_ERR_SHAPE;
    if ((int64_t)d->batch * d->nodes > 0x7fffffffLL) return SPECHUB_ERR_SHAPE;
    return SPECHUB_OK;
}

// rows whose every start is 16-byte aligned take the 128-bit load path
bool rows_aligned(const spechub_desc *d, const void *base) {
    const int esz = d->dtype == SPECHUB_BF16 ? 2 : 4;
    const int per16 = 16 / esz;
    return (reinterpret_cast<uintptr_t>(base) % 16 == 0) && (d->stride_node % per16 == 0) &&
           (d->stride_seq % per16 == 0);
}

int threads_for(const spechub_desc *d) {
    const int vw = d->dtype == SPECHUB_BF16 ? 8 : 4;
    const int nvec = (d->vocab + vw - 1) / vw;
    if (nvec >= 8192) return 512;
    if (nvec >= 2048) return 256;
    if (nvec >= 128) return 128;
    if (nvec >= 64) return 64;
    return 32;
}

RowArgs base_args(const spechub_desc *d) {
    RowArgs a = {};
    a.temperature_per_seq = d->temperature_per_seq;
    a.node_kind = d->node_kind;
    a.temperature = d->temperature;
    a.nodes = d->nodes;
    a.vocab = d->vocab;
    a.stride_seq = d->stride_seq;
    a.stride_node = d->stride_node;
    return a;
}

// The lean kernels take bf16 rows whose starts are 16-byte aligned and whose length is a
// multiple of 8 and large enough to keep 512 threads busy.
constexpr int kLeanDraftThreads = 128;
constexpr int kLeanThreads = 256;  // 4 CTAs per SM measured best (256/512/1024: 1.54/1.65/1.87 ms)
// Verification from draft statistics on shorter rows: 8 CTAs of 128 threads per SM overlap the fixed work of
// a row (reductions, tests, draws) better (V = 32000, 3840 rows: SpecHub 0.180 -> 0.158 ms, RRS 0.230 ->
// 0.205 ms; 64 threads: 0.171 ms; on V = 128256 the 256-thread CTA stays ahead, 1.02 against 1.06 ms).
constexpr int kLeanSmallThreads = 128;
constexpr int kLeanSmallVocab = 65536;

// CTAs per row.  With 4 CTAs per SM and 148 SMs, 592/CS rows are between their first and second
// read at any time; at CS = 4 on V = 128256 that fits L2 (DRAM reads drop from 2.0x to 1.0x the
// algorithmic bytes) but the per-CTA fixed work grows 4x, and the two cancel (1.6 vs 1.8 ms).
// 0 = no flag: one CTA per row (measured on B200: the per-CTA fixed work of a split row still outweighs
// the L2 hits), and the verification of RRS / RRSw takes its vectors from per-warp rings of bulk copies.
int lean_split(const spechub_desc *d) {
    if (d->flags & SPECHUB_FLAG_SPLIT_1) return 1;
    if (d->flags & SPECHUB_FLAG_SPLIT_2) return 2;
    if (d->flags & SPECHUB_FLAG_SPLIT_4) return 4;
    return 0;
}

constexpr int kMaxDevices = 64;
std::mutex g_attr_mutex;

template <class K, class... Args>
int launch_group(K kern, int cs, unsigned rows, cudaStream_t s, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = cs; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    cfg.attrs = at; cfg.numAttrs = cs > 1 ? 1 : 0;
    cfg.gridDim = dim3(rows * cs); cfg.blockDim = dim3(kLeanThreads); cfg.dynamicSmemBytes = 0; cfg.stream = s;
    return cudaLaunchKernelEx(&cfg, kern, args...) == cudaSuccess ? SPECHUB_OK : SPECHUB_ERR_LAUNCH;
}

template <int CS>
int launch_lean_verify_cs(int method, const RowArgs &a, unsigned rows, cudaStream_t s) {
    if (method == kSpecHub) return launch_group(lean_verify_kernel<kSpecHub, kLeanThreads, CS>, CS, rows, s, a);
    if (method == kRRS) return launch_group(lean_verify_kernel<kRRS, kLeanThreads, CS>, CS, rows, s, a);
    return launch_group(lean_verify_kernel<kRRSw, kLeanThreads, CS>, CS, rows, s, a);
}
// The leaf rows of an unsplit call (same CTA shape as the draft step).
int launch_lean_leaf(const RowArgs &a, const NodeOutPtrs *outs, int n_out, unsigned rows, cudaStream_t s) {
    LeafArgs la = {};
    la.r = a;
    la.n_out = n_out;
    for (int m = 0; m < n_out; ++m) la.out[m] = outs[m];
    lean_leaf_kernel<kLeanDraftThreads><<<rows, kLeanDraftThreads, 0, s>>>(la);
    return cudaGetLastError() == cudaSuccess ? SPECHUB_OK : SPECHUB_ERR_LAUNCH;
}

// One CTA per row, the passes fed by per-warp rings of bulk copies (spechub_ring.cuh).
template <int METHOD>
int launch_lean_verify_ring(const RowArgs &a, unsigned rows, cudaStream_t s) {
    auto kern = lean_verify_kernel<METHOD, kLeanThreads, 1, true>;
    constexpr int smem = kLeanThreads / 32 * kRingWarpBytes;
    static bool configured[kMaxDevices] = {};
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return SPECHUB_ERR_LAUNCH;
    {
        std::lock_guard<std::mutex> lock(g_attr_mutex);
        if (!configured[dev]) {
            if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) {
                cudaGetLastError();
                return SPECHUB_ERR_LAUNCH;
            }
            configured[dev] = true;
        }
    }
    kern<<<rows, kLeanThreads, smem, s>>>(a);
    return cudaGetLastError() == cudaSuccess ? SPECHUB_OK : SPECHUB_ERR_LAUNCH;
}

int launch_lean_verify(int method, int cs, const RowArgs &a, unsigned rows, cudaStream_t s) {
    if (cs == 4) return launch_lean_verify_cs<4>(method, a, rows, s);
    if (cs == 2) return launch_lean_verify_cs<2>(method, a, rows, s);
    if (a.node_kind) {
        const NodeOutPtrs o = {a.accept_idx, a.token, a.hub, a.beta, a.rate, a.status};
        const int lrc = launch_lean_leaf(a, &o, 1, rows, s);
        if (lrc != SPECHUB_OK) return lrc;
    }
    if (cs == 0 && a.draft_stats_in) {   // the draft row's statistics come from the draft step
        if (a.vocab <= kLeanSmallVocab) {
            if (method == kSpecHub) lean_verify_kernel<kSpecHub, kLeanSmallThreads, 1, false, true><<<rows, kLeanSmallThreads, 0, s>>>(a);
            else if (method == kRRS) lean_verify_kernel<kRRS, kLeanSmallThreads, 1, false, true><<<rows, kLeanSmallThreads, 0, s>>>(a);
            else lean_verify_kernel<kRRSw, kLeanSmallThreads, 1, false, true><<<rows, kLeanSmallThreads, 0, s>>>(a);
        } else
        if (method == kSpecHub) lean_verify_kernel<kSpecHub, kLeanThreads, 1, false, true><<<rows, kLeanThreads, 0, s>>>(a);
        else if (method == kRRS) lean_verify_kernel<kRRS, kLeanThreads, 1, false, true><<<rows, kLeanThreads, 0, s>>>(a);
        else lean_verify_kernel<kRRSw, kLeanThreads, 1, false, true><<<rows, kLeanThreads, 0, s>>>(a);
        return cudaGetLastError() == cudaSuccess ? SPECHUB_OK : SPECHUB_ERR_LAUNCH;
    }
    if (cs == 1 || method == kSpecHub) return launch_lean_verify_cs<1>(method, a, rows, s);
    if (method == kRRS) return launch_lean_verify_ring<kRRS>(a, rows, s);
    return launch_lean_verify_ring<kRRSw>(a, rows, s);
}
int launch_lean_draft(int method, int cs, const RowArgs &a, unsigned rows, cudaStream_t s) {
    if (cs == 4) return launch_group(lean_draft_kernel<kLeanThreads, 4>, 4, rows, s, a, method);
    if (cs == 2) return launch_group(lean_draft_kernel<kLeanThreads, 2>, 2, rows, s, a, method);
    // one CTA per row (cs 0 or 1): 128 threads, 8 CTAs per SM measured best for the single-pass draft step
    // (64 / 128 / 256 / 512 threads: 0.41 / 0.36 / 0.38 / 0.52 ms on V = 128256; 0.078 / 0.081 / 0.102 /
    // 0.165 ms on V = 32000)
    lean_draft_ck_kernel<kLeanDraftThreads><<<rows, kLeanDraftThreads, 0, s>>>(a, method);
    return cudaGetLastError() == cudaSuccess ? SPECHUB_OK : SPECHUB_ERR_LAUNCH;
}

bool lean_ok(const spechub_desc *d, bool aligned) {
    return d->dtype == SPECHUB_BF16 && aligned && d->vocab % 8 == 0 && d->vocab >= 8192;
}

// ---- verification with the exponentials resident on chip ------------------------------------------
// A row is spread over `cs` CTAs of 8 warps; every lane keeps `nb` batches of four 16-byte vectors
// of the row pair as fp32 exponentials (tensor memory, shared memory, registers).  The smallest
// cluster that holds the row with at most four batches per lane is taken.
struct ResShape { int cs, nb; };

bool resident_fits(const spechub_desc *d, bool aligned, ResShape *out);

// two drafts per node: on request (SPECHUB_FLAG_RESIDENT)
bool resident_shape(const spechub_desc *d, bool aligned, ResShape *out) {
    return (d->flags & SPECHUB_FLAG_RESIDENT) && resident_fits(d, aligned, out);
}

bool resident_fits(const spechub_desc *d, bool aligned, ResShape *out) {
    if (!lean_ok(d, aligned)) return false;
    const int nvec = d->vocab / 8;
    for (int cs = 1; cs <= 8; cs *= 2) {
        const int parts = cs * kResWarps;
        const int seg = (((nvec + parts - 1) / parts) + 7) & ~7;   // vectors per warp, as the kernel cuts them
        const int nb = (seg + 127) / 128;
        if (nb <= kResMaxBatches) { out->cs = cs; out->nb = nb; return true; }
    }
    return false;
}

template <int MASK, int CS>
int launch_resident_one(int nb, const FusedArgs &f, unsigned rows, cudaStream_t s) {
    auto kern = resident_verify_kernel<MASK, CS>;
    // tensor-memory columns of a CTA: two warps share each lane quarter, 32 columns per batch each
    const uint32_t cols = nb == 1 ? 64u : nb == 2 ? 128u : 256u;
    // Shared memory: e_q of all batches but the last.  A CTA that takes 256 columns asks for at least a
    // third of an SM's shared memory, so that no more than two such CTAs share the SM's 512 columns.
    int smem = (nb - 1) * 4 * 2 * kResThreads * 16;
    if (cols == 256u && smem < 76 * 1024) smem = 76 * 1024;
    constexpr int smem_max = (kResMaxBatches - 1) * 4 * 2 * kResThreads * 16;
    static bool configured[kMaxDevices] = {};
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return SPECHUB_ERR_LAUNCH;
    {
        std::lock_guard<std::mutex> lock(g_attr_mutex);
        if (!configured[dev]) {
            if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_max) != cudaSuccess) {
                cudaGetLastError();
                return SPECHUB_ERR_LAUNCH;
            }
            configured[dev] = true;
        }
    }
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = CS; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    cfg.attrs = at; cfg.numAttrs = CS > 1 ? 1 : 0;
    cfg.gridDim = dim3(rows * CS); cfg.blockDim = dim3(kResThreads); cfg.dynamicSmemBytes = smem; cfg.stream = s;
    return cudaLaunchKernelEx(&cfg, kern, f, nb, cols) == cudaSuccess ? SPECHUB_OK : SPECHUB_ERR_LAUNCH;
}

template <int MASK>
int launch_resident_mask(ResShape sh, const FusedArgs &f, unsigned rows, cudaStream_t s) {
    if (sh.cs == 1) return launch_resident_one<MASK, 1>(sh.nb, f, rows, s);
    if (sh.cs == 2) return launch_resident_one<MASK, 2>(sh.nb, f, rows, s);
    if (sh.cs == 4) return launch_resident_one<MASK, 4>(sh.nb, f, rows, s);
    return launch_resident_one<MASK, 8>(sh.nb, f, rows, s);
}

// Algorithm 1 with k > 2 drafts: the stages run over the exponentials kept on chip
template <int CS>
int launch_resident_kary_one(int nb, const KaryArgs &ka, unsigned rows, cudaStream_t s) {
    auto kern = resident_kary_kernel<CS>;
    const uint32_t cols = nb == 1 ? 64u : nb == 2 ? 128u : 256u;
    int smem = (nb - 1) * 4 * 2 * kResThreads * 16;
    if (cols == 256u && smem < 76 * 1024) smem = 76 * 1024;   // at most two CTAs of 256 columns per SM
    constexpr int smem_max = (kResMaxBatches - 1) * 4 * 2 * kResThreads * 16;
    static bool configured[kMaxDevices] = {};
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return SPECHUB_ERR_LAUNCH;
    {
        std::lock_guard<std::mutex> lock(g_attr_mutex);
        if (!configured[dev]) {
            if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_max) != cudaSuccess) {
                cudaGetLastError();
                return SPECHUB_ERR_LAUNCH;
            }
            configured[dev] = true;
        }
    }
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = CS; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    cfg.attrs = at; cfg.numAttrs = CS > 1 ? 1 : 0;
    cfg.gridDim = dim3(rows * CS); cfg.blockDim = dim3(kResThreads); cfg.dynamicSmemBytes = smem; cfg.stream = s;
    return cudaLaunchKernelEx(&cfg, kern, ka, nb, cols) == cudaSuccess ? SPECHUB_OK : SPECHUB_ERR_LAUNCH;
}

int launch_resident_kary(ResShape sh, const KaryArgs &ka, unsigned rows, cudaStream_t s) {
    if (sh.cs == 1) return launch_resident_kary_one<1>(sh.nb, ka, rows, s);
    if (sh.cs == 2) return launch_resident_kary_one<2>(sh.nb, ka, rows, s);
    if (sh.cs == 4) return launch_resident_kary_one<4>(sh.nb, ka, rows, s);
    return launch_resident_kary_one<8>(sh.nb, ka, rows, s);
}

// mask: bit m set = method m (0 SpecHub, 1 RRS, 2 RRSw) is verified; leaf rows go to lean_leaf_kernel
int launch_resident(int mask, ResShape sh, const FusedArgs &f, unsigned rows, cudaStream_t s) {
    if (f.r.node_kind) {
        NodeOutPtrs outs[3];
        int n_out = 0;
        for (int m = 0; m < 3; ++m)
            if (mask & (1 << m)) outs[n_out++] = f.out[m];
        const int lrc = launch_lean_leaf(f.r, outs, n_out, rows, s);
        if (lrc != SPECHUB_OK) return lrc;
    }
    if (mask == kMaskSpecHub) return launch_resident_mask<kMaskSpecHub>(sh, f, rows, s);
    if (mask == kMaskRRS) return launch_resident_mask<kMaskRRS>(sh, f, rows, s);
    if (mask == kMaskRRSw) return launch_resident_mask<kMaskRRSw>(sh, f, rows, s);
    return launch_resident_mask<7>(sh, f, rows, s);
}

int launch_status() { return cudaGetLastError() == cudaSuccess ? SPECHUB_OK : SPECHUB_ERR_LAUNCH; }

int draft_common(const spechub_desc *d, const void *draft_logits, const float *uniforms, int method,
                 int32_t *draft_tokens, int32_t *hub, float *draft_prob, uint32_t *status,
                 void *stream, void *draft_stats = nullptr) {
    const int rc = check_desc(d);
    if (rc != SPECHUB_OK) return rc;
    if (d->batch == 0) return SPECHUB_OK;  // nothing to do; pointers are not looked at
    if (!draft_logits || !uniforms || !draft_tokens) return SPECHUB_ERR_NULL;
    if (reinterpret_cast<uintptr_t>(draft_stats) % 16 != 0) return SPECHUB_ERR_STRIDE;
    RowArgs a = base_args(d);
    // Only the one-CTA-per-row kernel of the large-vocabulary bf16 shapes leaves statistics; every other
    // kernel leaves records that no verification accepts (all zero), and the verification paths that pair
    // with them do not look at the records.
    a.draft_stats_out = draft_stats;
    a.draft = draft_logits;
    a.uniforms = uniforms;
    a.draft_tokens_out = draft_tokens;
    a.hub = hub;
    a.draft_prob = draft_prob;
    a.status = status;
    const unsigned rows = (unsigned)(d->batch * (int64_t)d->nodes);
    const int th = threads_for(d);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const bool al = rows_aligned(d, draft_logits);
    if (d->k > 2) {
        if (method == kSpecHub) return SPECHUB_ERR_SHAPE;
        KaryArgs ka;
        ka.r = a; ka.k = d->k; ka.without_replacement = (method == kRRSw);
        if (d->dtype == SPECHUB_BF16) {
            if (al) kary_draft_kernel<__nv_bfloat16, true><<<rows, th, 0, s>>>(ka);
            else kary_draft_kernel<__nv_bfloat16, false><<<rows, th, 0, s>>>(ka);
        } else {
            if (al) kary_draft_kernel<float, true><<<rows, th, 0, s>>>(ka);
            else kary_draft_kernel<float, false><<<rows, th, 0, s>>>(ka);
        }
    } else if (lean_ok(d, al)) {
        const int lrc = launch_lean_draft(method, lean_split(d), a, rows, s);
        if (lrc != SPECHUB_OK) return lrc;
    } else if (d->dtype == SPECHUB_BF16) {
        if (al) draft_rows_kernel<__nv_bfloat16, true><<<rows, th, 0, s>>>(a, method);
        else draft_rows_kernel<__nv_bfloat16, false><<<rows, th, 0, s>>>(a, method);
    } else {
        if (al) draft_rows_kernel<float, true><<<rows, th, 0, s>>>(a, method);
        else draft_rows_kernel<float, false><<<rows, th, 0, s>>>(a, method);
    }
    return launch_status();
}

template <int METHOD>
void launch_verify(const spechub_desc *d, const RowArgs &a, bool al, unsigned rows, int th,
                   cudaStream_t s) {
    if (d->dtype == SPECHUB_BF16) {
        if (al) verify_rows_kernel<__nv_bfloat16, true, METHOD><<<rows, th, 0, s>>>(a);
        else verify_rows_kernel<__nv_bfloat16, false, METHOD><<<rows, th, 0, s>>>(a);
    } else {
        if (al) verify_rows_kernel<float, true, METHOD><<<rows, th, 0, s>>>(a);
        else verify_rows_kernel<float, false, METHOD><<<rows, th, 0, s>>>(a);
    }
}

int launch_walk(const spechub_desc *d, const spechub_node_out *no, const spechub_seq_out *so, cudaStream_t s) {
    if (!(so && (so->n_accepted || so->n_emitted || so->path_nodes || so->path_tokens))) return SPECHUB_OK;
    WalkArgs w;
    w.accept_idx = no->accept_idx;
    w.token = no->token;
    w.child = d->child;
    w.node_kind = d->node_kind;
    w.n_accepted = so->n_accepted;
    w.n_emitted = so->n_emitted;
    w.path_nodes = so->path_nodes;
    w.path_tokens = so->path_tokens;
    w.batch = d->batch;
    w.nodes = d->nodes;
    w.levels = d->levels;
    if (d->k > 2) {
        WalkKArgs wk;
        wk.w = w; wk.k = d->k;
        walk_k_kernel<<<(d->batch + 127) / 128, 128, 0, s>>>(wk);
    } else {
        walk_kernel<<<(d->batch + 127) / 128, 128, 0, s>>>(w);
    }
    return launch_status();
}

int verify_common(const spechub_desc *d, const void *target_logits, const void *draft_logits,
                  const int32_t *draft_tokens, const float *uniforms, int method,
                  const spechub_node_out *no, const spechub_seq_out *so, void *workspace,
                  size_t workspace_bytes, void *stream, const void *draft_stats = nullptr) {
    const int rc = check_desc(d);
    if (rc != SPECHUB_OK) return rc;
    if (d->batch == 0) return SPECHUB_OK;  // nothing to do; pointers are not looked at
    if (!target_logits || !draft_logits || !draft_tokens || !uniforms || !no || !no->accept_idx ||
        !no->token)
        return SPECHUB_ERR_NULL;
    if (workspace_bytes < spechub_workspace_bytes(d)) return SPECHUB_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(draft_stats) % 16 != 0) return SPECHUB_ERR_STRIDE;
    (void)workspace;
    RowArgs a = base_args(d);
    a.draft_stats_in = draft_stats;
    a.target = target_logits;
    a.draft = draft_logits;
    a.uniforms = uniforms;
    a.draft_tokens_in = draft_tokens;
    a.hub = no->hub;
    a.accept_idx = no->accept_idx;
    a.token = no->token;
    a.beta = no->beta;
    a.rate = no->rate;
    a.status = no->status;
    const unsigned rows = (unsigned)(d->batch * (int64_t)d->nodes);
    const int th = threads_for(d);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const bool al = rows_aligned(d, target_logits) && rows_aligned(d, draft_logits);
    if (d->k > 2) {
        if (method == kSpecHub) return SPECHUB_ERR_SHAPE;
        KaryArgs ka;
        ka.r = a; ka.k = d->k; ka.without_replacement = (method == kRRSw);
        ResShape rs;
        if (!(d->flags & 7u) && resident_fits(d, al, &rs)) {   // (a split flag asks for the streaming kernel)
            const int lrc = launch_resident_kary(rs, ka, rows, s);
            if (lrc != SPECHUB_OK) return lrc;
        } else if (d->dtype == SPECHUB_BF16) {
            if (al) kary_verify_kernel<__nv_bfloat16, true><<<rows, th, 0, s>>>(ka);
            else kary_verify_kernel<__nv_bfloat16, false><<<rows, th, 0, s>>>(ka);
        } else {
            if (al) kary_verify_kernel<float, true><<<rows, th, 0, s>>>(ka);
            else kary_verify_kernel<float, false><<<rows, th, 0, s>>>(ka);
        }
    } else if (ResShape rs; resident_shape(d, al, &rs)) {
        FusedArgs f = {};
        f.r = a;
        f.tok[method] = draft_tokens;
        f.out[method] = NodeOutPtrs{a.accept_idx, a.token, a.hub, a.beta, a.rate, a.status};
        const int lrc = launch_resident(1 << method, rs, f, rows, s);
        if (lrc != SPECHUB_OK) return lrc;
    } else if (lean_ok(d, al)) {
        const int lrc = launch_lean_verify(method, lean_split(d), a, rows, s);
        if (lrc != SPECHUB_OK) return lrc;
    } else if (method == kSpecHub) launch_verify<kSpecHub>(d, a, al, rows, th, s);
    else if (method == kRRS) launch_verify<kRRS>(d, a, al, rows, th, s);
    else launch_verify<kRRSw>(d, a, al, rows, th, s);
    const int lrc = launch_status();
    if (lrc != SPECHUB_OK) return lrc;
    return launch_walk(d, no, so, s);
}

// One kernel for the three methods where the lean kernels apply, the three separate paths otherwise.
int compare_draft(const spechub_desc *d, const void *draft_logits, const float *uniforms,
                  int32_t *const draft_tokens[3], int32_t *hub, float *draft_prob,
                  uint32_t *const status[3], void *stream, void *draft_stats = nullptr) {
    const int rc = check_desc(d);
    if (rc != SPECHUB_OK) return rc;
    if (d->k != 2) return SPECHUB_ERR_SHAPE;
    if (d->batch == 0) return SPECHUB_OK;
    if (!draft_logits || !uniforms || !draft_tokens || !draft_tokens[0] || !draft_tokens[1] || !draft_tokens[2])
        return SPECHUB_ERR_NULL;
    if (reinterpret_cast<uintptr_t>(draft_stats) % 16 != 0) return SPECHUB_ERR_STRIDE;
    if (!lean_ok(d, rows_aligned(d, draft_logits))) {
        for (int m = 0; m < 3; ++m) {
            const int mrc = draft_common(d, draft_logits, uniforms, m, draft_tokens[m], m == 0 ? hub : nullptr,
                                         m == 0 ? draft_prob : nullptr, status ? status[m] : nullptr, stream,
                                         m == 0 ? draft_stats : nullptr);   // (void records)
            if (mrc != SPECHUB_OK) return mrc;
        }
        return SPECHUB_OK;
    }
    FusedArgs f = {};
    f.r = base_args(d);
    f.r.draft = draft_logits;
    f.r.uniforms = uniforms;
    // records are kept where the per-method calls keep them: no split flag
    if (draft_stats && lean_split(d) != 0 &&
        cudaMemsetAsync(draft_stats, 0, spechub_draft_stats_bytes(d), static_cast<cudaStream_t>(stream)) != cudaSuccess)
        return SPECHUB_ERR_LAUNCH;
    f.r.draft_stats_out = lean_split(d) == 0 ? draft_stats : nullptr;
    for (int m = 0; m < 3; ++m) {
        f.tok_out[m] = draft_tokens[m];
        f.dstatus[m] = status ? status[m] : nullptr;
    }
    const unsigned rows = (unsigned)(d->batch * (int64_t)d->nodes);
    // same CTA shape as lean_draft_ck_kernel: the results are to be the same bit for bit
    fused_draft_kernel<kLeanDraftThreads><<<rows, kLeanDraftThreads, 0, static_cast<cudaStream_t>(stream)>>>(f, hub, draft_prob);
    return launch_status();
}

int compare_verify(const spechub_desc *d, const void *target_logits, const void *draft_logits,
                   const int32_t *const draft_tokens[3], const float *uniforms,
                   const spechub_node_out *no, const spechub_seq_out *so, void *workspace,
                   size_t workspace_bytes, void *stream, const void *draft_stats = nullptr) {
    const int rc = check_desc(d);
    if (rc != SPECHUB_OK) return rc;
    if (d->k != 2) return SPECHUB_ERR_SHAPE;
    if (d->batch == 0) return SPECHUB_OK;
    if (!target_logits || !draft_logits || !uniforms || !no || !draft_tokens) return SPECHUB_ERR_NULL;
    for (int m = 0; m < 3; ++m)
        if (!draft_tokens[m] || !no[m].accept_idx || !no[m].token) return SPECHUB_ERR_NULL;
    if (workspace_bytes < spechub_workspace_bytes(d)) return SPECHUB_ERR_WORKSPACE;
    const bool al = rows_aligned(d, target_logits) && rows_aligned(d, draft_logits);
    if (!lean_ok(d, al)) {
        for (int m = 0; m < 3; ++m) {
            const int mrc = verify_common(d, target_logits, draft_logits, draft_tokens[m], uniforms, m, &no[m],
                                          so ? &so[m] : nullptr, workspace, workspace_bytes, stream, draft_stats);
            if (mrc != SPECHUB_OK) return mrc;
        }
        return SPECHUB_OK;
    }
    FusedArgs f = {};
    f.r = base_args(d);
    f.r.target = target_logits;
    f.r.draft = draft_logits;
    f.r.uniforms = uniforms;
    for (int m = 0; m < 3; ++m) {
        f.tok[m] = draft_tokens[m];
        f.out[m].accept_idx = no[m].accept_idx; f.out[m].token = no[m].token; f.out[m].hub = no[m].hub;
        f.out[m].beta = no[m].beta; f.out[m].rate = no[m].rate; f.out[m].status = no[m].status;
    }
    const unsigned rows = (unsigned)(d->batch * (int64_t)d->nodes);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int lrc;
    if (ResShape rs; resident_shape(d, al, &rs)) {
        lrc = launch_resident(7, rs, f, rows, s);
    } else {
        if (d->node_kind) {
            const int llrc = launch_lean_leaf(f.r, f.out, 3, rows, s);
            if (llrc != SPECHUB_OK) return llrc;
        }
        if (draft_stats && lean_split(d) == 0) {
            f.r.draft_stats_in = draft_stats;
            // (the CTA shape of the per-method kernels, whose results these are bit for bit)
            if (d->vocab <= kLeanSmallVocab) fused_verify_kernel<kLeanSmallThreads, true><<<rows, kLeanSmallThreads, 0, s>>>(f);
            else fused_verify_kernel<kLeanThreads, true><<<rows, kLeanThreads, 0, s>>>(f);
        } else {
            fused_verify_kernel<kLeanThreads><<<rows, kLeanThreads, 0, s>>>(f);
        }
        lrc = launch_status();
    }
    for (int m = 0; m < 3 && lrc == SPECHUB_OK && so; ++m) lrc = launch_walk(d, &no[m], &so[m], s);
    return lrc;
}

// ---- vocabulary-sharded phases ------------------------------------------------------------------
int check_shard(const spechub_desc *d, const spechub_shard *sh) {
    const int rc = check_desc(d);
    if (rc != SPECHUB_OK) return rc;
    if (!sh) return SPECHUB_ERR_NULL;
    if (d->k != 2) return SPECHUB_ERR_SHAPE;
    if (sh->nranks < 1 || sh->nranks > 64 || sh->rank < 0 || sh->rank >= sh->nranks || sh->id_offset < 0 ||
        sh->vocab_total < 2 || (int64_t)sh->id_offset + d->vocab > sh->vocab_total)
        return SPECHUB_ERR_SHAPE;
    return SPECHUB_OK;
}

ShardArgs shard_args(const spechub_desc *d, const spechub_shard *sh) {
    ShardArgs a = {};
    a.r = base_args(d);
    a.rank = sh->rank; a.nranks = sh->nranks; a.id_offset = sh->id_offset; a.vocab_total = sh->vocab_total;
    a.rows = d->batch * (int64_t)d->nodes;
    return a;
}

enum ShardPhase { kPhaseStats, kPhaseSums, kPhaseDecide, kPhaseDraft, kPhaseRrsSums, kPhaseRrsDecide, kPhaseRrsDraft };

template <typename LT, bool AL>
void launch_shard_phase(int phase, const ShardArgs &a, unsigned rows, int th, cudaStream_t s) {
    if (phase == kPhaseStats) shard_stats_kernel<LT, AL><<<rows, th, 0, s>>>(a);
    else if (phase == kPhaseSums) shard_sums_kernel<LT, AL><<<rows, th, 0, s>>>(a);
    else if (phase == kPhaseDecide) shard_decide_kernel<LT, AL><<<rows, th, 0, s>>>(a);
    else if (phase == kPhaseDraft) shard_draft_kernel<LT, AL><<<rows, th, 0, s>>>(a);
    else if (phase == kPhaseRrsSums) rrs_shard_sums_kernel<LT, AL><<<rows, th, 0, s>>>(a);
    else if (phase == kPhaseRrsDecide) rrs_shard_decide_kernel<LT, AL><<<rows, th, 0, s>>>(a);
    else rrs_shard_draft_kernel<LT, AL><<<rows, th, 0, s>>>(a);
}

int run_shard_phase(int phase, const spechub_desc *d, const ShardArgs &a, void *stream) {
    const unsigned rows = (unsigned)a.rows;
    const int th = threads_for(d);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const bool al = (!a.r.target || rows_aligned(d, a.r.target)) && (!a.r.draft || rows_aligned(d, a.r.draft));
    if (d->dtype == SPECHUB_BF16) {
        if (al) launch_shard_phase<__nv_bfloat16, true>(phase, a, rows, th, s);
        else launch_shard_phase<__nv_bfloat16, false>(phase, a, rows, th, s);
    } else {
        if (al) launch_shard_phase<float, true>(phase, a, rows, th, s);
        else launch_shard_phase<float, false>(phase, a, rows, th, s);
    }
    return launch_status();
}

}  // namespace

extern "C" {

int spechub_draft_sample(const spechub_desc *desc, const void *draft_logits, const float *uniforms,
                         int32_t *draft_tokens, int32_t *hub, float *draft_prob, uint32_t *status,
                         void *stream) {
    return draft_common(desc, draft_logits, uniforms, kSpecHub, draft_tokens, hub, draft_prob, status,
                        stream);
}

int rrs_draft_sample(const spechub_desc *desc, const void *draft_logits, const float *uniforms,
                     int without_replacement, int32_t *draft_tokens, uint32_t *status, void *stream) {
    if (without_replacement != 0 && without_replacement != 1) return SPECHUB_ERR_METHOD;
    return draft_common(desc, draft_logits, uniforms, without_replacement ? kRRSw : kRRS,
                        draft_tokens, nullptr, nullptr, status, stream);
}

int spechub_draft_sample_stats(const spechub_desc *desc, const void *draft_logits, const float *uniforms,
                               int32_t *draft_tokens, int32_t *hub, float *draft_prob, uint32_t *status,
                               void *draft_stats, void *stream) {
    if (!draft_stats && desc && desc->batch != 0) return SPECHUB_ERR_NULL;
    return draft_common(desc, draft_logits, uniforms, kSpecHub, draft_tokens, hub, draft_prob, status,
                        stream, draft_stats);
}

int rrs_draft_sample_stats(const spechub_desc *desc, const void *draft_logits, const float *uniforms,
                           int without_replacement, int32_t *draft_tokens, uint32_t *status,
                           void *draft_stats, void *stream) {
    if (without_replacement != 0 && without_replacement != 1) return SPECHUB_ERR_METHOD;
    if (!draft_stats && desc && desc->batch != 0) return SPECHUB_ERR_NULL;
    return draft_common(desc, draft_logits, uniforms, without_replacement ? kRRSw : kRRS,
                        draft_tokens, nullptr, nullptr, status, stream, draft_stats);
}

int spechub_verify_tree_stats(const spechub_desc *desc, const void *target_logits, const void *draft_logits,
                              const void *draft_stats, const int32_t *draft_tokens, const float *uniforms,
                              const spechub_node_out *node_out, const spechub_seq_out *seq_out,
                              void *workspace, size_t workspace_bytes, void *stream) {
    if (!draft_stats && desc && desc->batch != 0) return SPECHUB_ERR_NULL;
    return verify_common(desc, target_logits, draft_logits, draft_tokens, uniforms, kSpecHub,
                         node_out, seq_out, workspace, workspace_bytes, stream, draft_stats);
}

int rrs_verify_tree_stats(const spechub_desc *desc, const void *target_logits, const void *draft_logits,
                          const void *draft_stats, const int32_t *draft_tokens, const float *uniforms,
                          int without_replacement, const spechub_node_out *node_out,
                          const spechub_seq_out *seq_out, void *workspace, size_t workspace_bytes,
                          void *stream) {
    if (without_replacement != 0 && without_replacement != 1) return SPECHUB_ERR_METHOD;
    if (!draft_stats && desc && desc->batch != 0) return SPECHUB_ERR_NULL;
    return verify_common(desc, target_logits, draft_logits, draft_tokens, uniforms,
                         without_replacement ? kRRSw : kRRS, node_out, seq_out, workspace,
                         workspace_bytes, stream, draft_stats);
}

int spechub_verify_tree(const spechub_desc *desc, const void *target_logits,
                        const void *draft_logits, const int32_t *draft_tokens,
                        const float *uniforms, const spechub_node_out *node_out,
                        const spechub_seq_out *seq_out, void *workspace, size_t workspace_bytes,
                        void *stream) {
    return verify_common(desc, target_logits, draft_logits, draft_tokens, uniforms, kSpecHub,
                         node_out, seq_out, workspace, workspace_bytes, stream);
}

int rrs_verify_tree(const spechub_desc *desc, const void *target_logits, const void *draft_logits,
                    const int32_t *draft_tokens, const float *uniforms, int without_replacement,
                    const spechub_node_out *node_out, const spechub_seq_out *seq_out,
                    void *workspace, size_t workspace_bytes, void *stream) {
    if (without_replacement != 0 && without_replacement != 1) return SPECHUB_ERR_METHOD;
    return verify_common(desc, target_logits, draft_logits, draft_tokens, uniforms,
                         without_replacement ? kRRSw : kRRS, node_out, seq_out, workspace,
                         workspace_bytes, stream);
}

int mdsd_compare_draft_sample(const spechub_desc *desc, const void *draft_logits, const float *uniforms,
                              int32_t *const draft_tokens[3], int32_t *hub, float *draft_prob,
                              uint32_t *const status[3], void *stream) {
    return compare_draft(desc, draft_logits, uniforms, draft_tokens, hub, draft_prob, status, stream);
}

int mdsd_compare_draft_sample_stats(const spechub_desc *desc, const void *draft_logits, const float *uniforms,
                                    int32_t *const draft_tokens[3], int32_t *hub, float *draft_prob,
                                    uint32_t *const status[3], void *draft_stats, void *stream) {
    if (!draft_stats && desc && desc->batch != 0) return SPECHUB_ERR_NULL;
    return compare_draft(desc, draft_logits, uniforms, draft_tokens, hub, draft_prob, status, stream, draft_stats);
}

int mdsd_compare_verify_tree_stats(const spechub_desc *desc, const void *target_logits, const void *draft_logits,
                                   const void *draft_stats, const int32_t *const draft_tokens[3],
                                   const float *uniforms, const spechub_node_out node_out[3],
                                   const spechub_seq_out *seq_out, void *workspace, size_t workspace_bytes,
                                   void *stream) {
    if (!draft_stats && desc && desc->batch != 0) return SPECHUB_ERR_NULL;
    if (reinterpret_cast<uintptr_t>(draft_stats) % 16 != 0) return SPECHUB_ERR_STRIDE;
    return compare_verify(desc, target_logits, draft_logits, draft_tokens, uniforms, node_out, seq_out,
                          workspace, workspace_bytes, stream, draft_stats);
}

int mdsd_compare_verify_tree(const spechub_desc *desc, const void *target_logits, const void *draft_logits,
                             const int32_t *const draft_tokens[3], const float *uniforms,
                             const spechub_node_out node_out[3], const spechub_seq_out *seq_out,
                             void *workspace, size_t workspace_bytes, void *stream) {
    return compare_verify(desc, target_logits, draft_logits, draft_tokens, uniforms, node_out, seq_out,
                          workspace, workspace_bytes, stream);
}

int spechub_walk_tree(const spechub_desc *desc, const int32_t *accept_idx, const int32_t *token,
                      const spechub_seq_out *seq_out, void *stream) {
    const int rc = check_desc(desc);
    if (rc != SPECHUB_OK) return rc;
    if (desc->batch == 0) return SPECHUB_OK;
    if (!accept_idx || !token || !seq_out) return SPECHUB_ERR_NULL;
    spechub_node_out no = {};
    no.accept_idx = const_cast<int32_t *>(accept_idx);
    no.token = const_cast<int32_t *>(token);
    return launch_walk(desc, &no, seq_out, static_cast<cudaStream_t>(stream));
}

int spechub_shard_stats(const spechub_desc *desc, const spechub_shard *shard, const void *target_slice,
                        const void *draft_slice, float *stats, void *stream) {
    const int rc = check_shard(desc, shard);
    if (rc != SPECHUB_OK) return rc;
    if (desc->batch == 0) return SPECHUB_OK;
    if (!draft_slice || !stats) return SPECHUB_ERR_NULL;
    ShardArgs a = shard_args(desc, shard);
    a.r.target = target_slice; a.r.draft = draft_slice; a.out = stats;
    return run_shard_phase(kPhaseStats, desc, a, stream);
}

int spechub_shard_sums(const spechub_desc *desc, const spechub_shard *shard, const void *target_slice,
                       const void *draft_slice, const int32_t *draft_tokens, const float *gathered_stats,
                       float *sums, void *stream) {
    const int rc = check_shard(desc, shard);
    if (rc != SPECHUB_OK) return rc;
    if (desc->batch == 0) return SPECHUB_OK;
    if (!target_slice || !draft_slice || !draft_tokens || !gathered_stats || !sums) return SPECHUB_ERR_NULL;
    ShardArgs a = shard_args(desc, shard);
    a.r.target = target_slice; a.r.draft = draft_slice; a.r.draft_tokens_in = draft_tokens;
    a.gstats = gathered_stats; a.out = sums;
    return run_shard_phase(kPhaseSums, desc, a, stream);
}

int spechub_shard_decide(const spechub_desc *desc, const spechub_shard *shard, const void *target_slice,
                         const void *draft_slice, const int32_t *draft_tokens, const float *uniforms,
                         const float *gathered_stats, const float *gathered_sums,
                         const spechub_node_out *no, void *stream) {
    const int rc = check_shard(desc, shard);
    if (rc != SPECHUB_OK) return rc;
    if (desc->batch == 0) return SPECHUB_OK;
    if (!target_slice || !draft_slice || !draft_tokens || !uniforms || !gathered_stats || !gathered_sums ||
        !no || !no->accept_idx || !no->token)
        return SPECHUB_ERR_NULL;
    ShardArgs a = shard_args(desc, shard);
    a.r.target = target_slice; a.r.draft = draft_slice; a.r.draft_tokens_in = draft_tokens;
    a.r.uniforms = uniforms; a.gstats = gathered_stats; a.gsums = gathered_sums;
    a.r.hub = no->hub; a.r.accept_idx = no->accept_idx; a.r.token = no->token;
    a.r.beta = no->beta; a.r.rate = no->rate; a.r.status = no->status;
    return run_shard_phase(kPhaseDecide, desc, a, stream);
}

int spechub_shard_draft(const spechub_desc *desc, const spechub_shard *shard, const void *draft_slice,
                        const float *uniforms, const float *gathered_stats, int32_t *cand, void *stream) {
    const int rc = check_shard(desc, shard);
    if (rc != SPECHUB_OK) return rc;
    if (desc->batch == 0) return SPECHUB_OK;
    if (!draft_slice || !uniforms || !gathered_stats || !cand) return SPECHUB_ERR_NULL;
    ShardArgs a = shard_args(desc, shard);
    a.r.draft = draft_slice; a.r.uniforms = uniforms; a.gstats = gathered_stats; a.cand_out = cand;
    return run_shard_phase(kPhaseDraft, desc, a, stream);
}

int spechub_shard_draft_finish(const spechub_desc *desc, const spechub_shard *shard,
                               const float *gathered_stats, const int32_t *cand_max,
                               int32_t *draft_tokens, int32_t *hub, uint32_t *status, void *stream) {
    const int rc = check_shard(desc, shard);
    if (rc != SPECHUB_OK) return rc;
    if (desc->batch == 0) return SPECHUB_OK;
    if (!gathered_stats || !cand_max || !draft_tokens) return SPECHUB_ERR_NULL;
    ShardArgs a = shard_args(desc, shard);
    a.gstats = gathered_stats; a.cand = cand_max;
    a.r.draft_tokens_out = draft_tokens; a.r.hub = hub; a.r.status = status;
    shard_draft_finish_kernel<<<(unsigned)((a.rows + 127) / 128), 128, 0, static_cast<cudaStream_t>(stream)>>>(a);
    return launch_status();
}

int rrs_shard_sums(const spechub_desc *desc, const spechub_shard *shard, int without_replacement,
                   const void *target_slice, const void *draft_slice, const int32_t *draft_tokens,
                   const float *gathered_stats, const float *gathered_sums, float *out, void *stream) {
    if (without_replacement != 0 && without_replacement != 1) return SPECHUB_ERR_METHOD;
    const int rc = check_shard(desc, shard);
    if (rc != SPECHUB_OK) return rc;
    if (desc->batch == 0) return SPECHUB_OK;
    if (!target_slice || !draft_slice || !draft_tokens || !gathered_stats || !out) return SPECHUB_ERR_NULL;
    ShardArgs a = shard_args(desc, shard);
    a.without_replacement = without_replacement;
    a.r.target = target_slice; a.r.draft = draft_slice; a.r.draft_tokens_in = draft_tokens;
    a.gstats = gathered_stats; a.gsums = gathered_sums; a.out = out;
    return run_shard_phase(kPhaseRrsSums, desc, a, stream);
}

int rrs_shard_decide(const spechub_desc *desc, const spechub_shard *shard, int without_replacement,
                     const void *target_slice, const void *draft_slice, const int32_t *draft_tokens,
                     const float *uniforms, const float *gathered_stats, const float *gathered_sums,
                     const float *gathered_w2, const spechub_node_out *no, void *stream) {
    if (without_replacement != 0 && without_replacement != 1) return SPECHUB_ERR_METHOD;
    const int rc = check_shard(desc, shard);
    if (rc != SPECHUB_OK) return rc;
    if (desc->batch == 0) return SPECHUB_OK;
    if (!target_slice || !draft_slice || !draft_tokens || !uniforms || !gathered_stats || !gathered_sums ||
        !gathered_w2 || !no || !no->accept_idx || !no->token)
        return SPECHUB_ERR_NULL;
    ShardArgs a = shard_args(desc, shard);
    a.without_replacement = without_replacement;
    a.r.target = target_slice; a.r.draft = draft_slice; a.r.draft_tokens_in = draft_tokens;
    a.r.uniforms = uniforms; a.gstats = gathered_stats; a.gsums = gathered_sums; a.gw2 = gathered_w2;
    a.r.hub = no->hub; a.r.accept_idx = no->accept_idx; a.r.token = no->token;
    a.r.beta = no->beta; a.r.rate = no->rate; a.r.status = no->status;
    return run_shard_phase(kPhaseRrsDecide, desc, a, stream);
}

int rrs_shard_draft(const spechub_desc *desc, const spechub_shard *shard, int without_replacement,
                    const void *draft_slice, const float *uniforms, const float *gathered_stats,
                    const int32_t *cand_max, const float *ex1_max, int32_t *cand, float *ex1, void *stream) {
    if (without_replacement != 0 && without_replacement != 1) return SPECHUB_ERR_METHOD;
    const int rc = check_shard(desc, shard);
    if (rc != SPECHUB_OK) return rc;
    if (desc->batch == 0) return SPECHUB_OK;
    if (!draft_slice || !uniforms || !gathered_stats || !cand) return SPECHUB_ERR_NULL;
    if ((cand_max == nullptr) != (ex1_max == nullptr)) return SPECHUB_ERR_NULL;
    if (cand_max && !without_replacement) return SPECHUB_ERR_METHOD;   // only RRSw has a second round
    ShardArgs a = shard_args(desc, shard);
    a.without_replacement = without_replacement;
    a.r.draft = draft_slice; a.r.uniforms = uniforms; a.gstats = gathered_stats;
    a.x1_known = cand_max; a.ex1_known = ex1_max; a.cand_out = cand; a.ex1_out = ex1;
    return run_shard_phase(kPhaseRrsDraft, desc, a, stream);
}

int rrs_shard_draft_finish(const spechub_desc *desc, const spechub_shard *shard, int without_replacement,
                           const float *gathered_stats, const int32_t *cand_max, int32_t *draft_tokens,
                           uint32_t *status, void *stream) {
    if (without_replacement != 0 && without_replacement != 1) return SPECHUB_ERR_METHOD;
    const int rc = check_shard(desc, shard);
    if (rc != SPECHUB_OK) return rc;
    if (desc->batch == 0) return SPECHUB_OK;
    if (!gathered_stats || !cand_max || !draft_tokens) return SPECHUB_ERR_NULL;
    ShardArgs a = shard_args(desc, shard);
    a.without_replacement = without_replacement;
    a.gstats = gathered_stats; a.cand = cand_max;
    a.r.draft_tokens_out = draft_tokens; a.r.status = status;
    rrs_shard_draft_finish_kernel<<<(unsigned)((a.rows + 127) / 128), 128, 0, static_cast<cudaStream_t>(stream)>>>(a);
    return launch_status();
}

size_t spechub_workspace_bytes(const spechub_desc *desc) {
    (void)desc;
    return 0;
}

size_t spechub_draft_stats_bytes(const spechub_desc *desc) {
    if (!desc || desc->batch < 0 || desc->nodes < 1) return 0;
    return sizeof(DraftStat) * static_cast<size_t>(desc->batch) * static_cast<size_t>(desc->nodes);
}

const char *spechub_status_string(int code) {
    switch (code) {
        case SPECHUB_OK: return "ok";
        case SPECHUB_ERR_NULL: return "a required pointer is NULL";
        case SPECHUB_ERR_VERSION: return "descriptor struct_size/version mismatch";
        case SPECHUB_ERR_SHAPE: return "bad shape: need batch >= 0, nodes >= 1, vocab >= 2, 2 <= k <= 8 (k == 2 for SpecHub), levels >= 1, valid flags";
        case SPECHUB_ERR_DTYPE: return "dtype must be SPECHUB_F32 or SPECHUB_BF16";
        case SPECHUB_ERR_STRIDE: return "strides too small for the given shape";
        case SPECHUB_ERR_TEMPERATURE: return "temperature must be finite and > 0";
        case SPECHUB_ERR_WORKSPACE: return "workspace smaller than spechub_workspace_bytes()";
        case SPECHUB_ERR_LAUNCH: return "kernel launch failed";
        case SPECHUB_ERR_METHOD: return "without_replacement must be 0 or 1";
        case SPECHUB_ERR_TOO_LARGE: return "batch * nodes exceeds SPECHUB_STATIC_MAX_ROWS of spechub_verify_tree_static";
        default: return "unknown status";
    }
}

int spechub_abi_version(void) { return SPECHUB_ABI_VERSION; }

}  // extern "C"

// ---- verification without any allocation ---------------------------------------------------------
// Scratch of spechub_verify_tree_static: per row the "stats" record and the "sums" record of the
// phase kernels (8 floats each).  Lives in every GPU that loads the library until the process ends.
static __device__ __align__(256) float g_static_scratch[(size_t)SPECHUB_STATIC_MAX_ROWS * 2 * spechub::kShardRecord];

namespace {

std::mutex g_static_mutex;
float *g_static_ptr[kMaxDevices] = {};

// Device address of g_static_scratch on the current device.  In host code the array's name is only
// a handle for the runtime, never an address a kernel may be given, so the address is looked up
// once per device (with that device current) and kept.
int static_scratch(float **out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return SPECHUB_ERR_LAUNCH;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_ptr[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) {
            cudaGetLastError();
            return SPECHUB_ERR_LAUNCH;
        }
        g_static_ptr[dev] = static_cast<float *>(p);
    }
    *out = g_static_ptr[dev];
    return SPECHUB_OK;
}

}  // namespace

extern "C" int spechub_verify_tree_static(const spechub_desc *desc, const void *target_logits,
                                          const void *draft_logits, const int32_t *draft_tokens,
                                          const float *uniforms, const spechub_node_out *no,
                                          const spechub_seq_out *so, void *stream) {
    const int rc = check_desc(desc);
    if (rc != SPECHUB_OK) return rc;
    if (desc->k != 2) return SPECHUB_ERR_SHAPE;
    if (desc->batch == 0) return SPECHUB_OK;
    if (!target_logits || !draft_logits || !draft_tokens || !uniforms || !no || !no->accept_idx || !no->token)
        return SPECHUB_ERR_NULL;
    const int64_t rows = desc->batch * (int64_t)desc->nodes;
    if (rows > SPECHUB_STATIC_MAX_ROWS) return SPECHUB_ERR_TOO_LARGE;
    float *scratch = nullptr;
    const int src = static_scratch(&scratch);
    if (src != SPECHUB_OK) return src;
    float *stats = scratch, *sums = scratch + rows * kShardRecord;

    // one rank that holds the whole vocabulary: the phase kernels, back to back on the stream
    spechub_shard whole = {0, 1, 0, desc->vocab};
    ShardArgs a = shard_args(desc, &whole);
    a.r.target = target_logits; a.r.draft = draft_logits; a.r.draft_tokens_in = draft_tokens;
    a.r.uniforms = uniforms;
    a.out = stats;                     // every record is written in full: nothing has to start at zero
    int prc = run_shard_phase(kPhaseStats, desc, a, stream);
    if (prc != SPECHUB_OK) return prc;
    a.gstats = stats; a.out = sums;
    prc = run_shard_phase(kPhaseSums, desc, a, stream);
    if (prc != SPECHUB_OK) return prc;
    a.gsums = sums; a.out = nullptr;
    a.r.hub = no->hub; a.r.accept_idx = no->accept_idx; a.r.token = no->token;
    a.r.beta = no->beta; a.r.rate = no->rate; a.r.status = no->status;
    prc = run_shard_phase(kPhaseDecide, desc, a, stream);
    if (prc != SPECHUB_OK) return prc;
    return launch_walk(desc, no, so, static_cast<cudaStream_t>(stream));
}
