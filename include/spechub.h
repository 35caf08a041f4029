/*
 * spechub.h -- C ABI of the sampling-verification step of multi-draft
 * speculative decoding: SpecHub (k = 2) with Recursive Rejection Sampling
 * with and without replacement (RRS, RRSw) as the comparison path
 * (arXiv 2411.05289).
 *
 * Notation is the paper's (Section 2): p = target distribution, q = draft
 * distribution over a vocabulary of size V; a = argmax q is the hub token
 * (Section 4); each tree node carries k = 2 draft tokens (x1, x2), one per
 * child.  Both distributions are given as logits and a temperature T:
 * p = softmax(target_logits / T), q = softmax(draft_logits / T).
 *
 * General rules for every entry point
 *   - All data pointers are DEVICE pointers owned by the caller, valid until
 *     the work enqueued on `stream` has finished.  The descriptor itself is
 *     read on the host during the call.  The library allocates nothing and
 *     keeps no state between calls (spechub_verify_tree_static alone holds a
 *     static scratch array; see there).
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *     Calls enqueue work and return without synchronising.
 *   - Return value: SPECHUB_OK (0) when the work was enqueued; a negative
 *     SPECHUB_ERR_* when an argument was rejected on the host (nothing was
 *     launched) or a launch failed.  Nothing is printed, nothing throws.
 *     batch = 0 is a valid empty call: it returns SPECHUB_OK without looking
 *     at any data pointer.
 *   - Per-row problems found on the device are reported as bits in the row's
 *     `status` word and give the documented fallback output; kernels never
 *     trap and wait only on hardware barriers, on the completion of bulk
 *     copies they issued themselves (a bounded wait: SPECHUB_ST_INTERNAL if
 *     it runs out) and, where stated, on the hardware's tensor-memory
 *     allocator.
 *   - Layout: logits are [batch][nodes][vocab] with element strides
 *     `stride_seq`, `stride_node` (rows are contiguous in the vocabulary).
 *     Rows that start on a 16-byte boundary are read with 128-bit loads; other
 *     rows are still read correctly, element by element.
 *     uniforms are float [batch][nodes][5] = (u_d1, u_d2, r1, r2, u_res), each
 *     in [0, 1): u_d1, u_d2 drive the two draft draws; r1, r2 the first and
 *     second acceptance test performed at the node; u_res the residual (or
 *     leaf) draw.  draft_tokens are int32 [batch][nodes][2]; per-node outputs
 *     are [batch][nodes] (row-major), with 2 or 3 trailing entries where
 *     stated.  With k drafts per node (RRS / RRSw only) the same layouts
 *     hold with k in place of 2: uniforms [..][2k+1] = (u_d1..u_dk, r_1..r_k,
 *     u_res), draft_tokens [..][k], beta [..][k], rate [..][k+1], child
 *     [nodes][k] (NULL = complete k-ary tree, child i of n is k*n + 1 + i),
 *     accept_idx in {-1, 0..k-1}.
 *   - Sampling from a non-negative weight vector w with a uniform u always
 *     means: the lowest token id j whose inclusive prefix sum over ascending
 *     ids exceeds u * sum(w); zero-weight ids are never returned.
 *   - An acceptance test with probability min(N/D, 1) is the strict test
 *     r * D < N; D = 0 rejects.
 */
#ifndef SPECHUB_H_
#define SPECHUB_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SPECHUB_ABI_VERSION 1
#define SPECHUB_MAX_K 8 /* most drafts per node the RRS / RRSw entry points take */

/* return codes */
#define SPECHUB_OK 0
#define SPECHUB_ERR_NULL (-1)        /* a required pointer is NULL                        */
#define SPECHUB_ERR_VERSION (-2)     /* struct_size / version do not match this library   */
#define SPECHUB_ERR_SHAPE (-3)       /* batch < 0, nodes < 1, vocab < 2, k outside 2..8 (SpecHub: k != 2), levels < 1, bad flags */
#define SPECHUB_ERR_DTYPE (-4)       /* dtype is not SPECHUB_F32 / SPECHUB_BF16            */
#define SPECHUB_ERR_STRIDE (-5)      /* stride_node < vocab or stride_seq too small; draft_stats not 16-byte aligned */
#define SPECHUB_ERR_TEMPERATURE (-6) /* temperature not a finite number > 0               */
#define SPECHUB_ERR_WORKSPACE (-7)   /* workspace smaller than spechub_workspace_bytes()   */
#define SPECHUB_ERR_LAUNCH (-8)      /* the CUDA runtime refused a launch                  */
#define SPECHUB_ERR_METHOD (-9)      /* without_replacement is not 0 or 1                  */
#define SPECHUB_ERR_TOO_LARGE (-10)  /* more rows than spechub_verify_tree_static can hold */

/* logits element type */
#define SPECHUB_F32 0
#define SPECHUB_BF16 1

/* per-row status bits */
#define SPECHUB_ST_NONFINITE 1u       /* NaN or +inf logit, or no finite logit: row output is -1 */
#define SPECHUB_ST_TOKEN_RANGE 2u     /* draft token out of range / pair lacks the hub: output -1  */
#define SPECHUB_ST_DEGENERATE_Q 4u    /* draft mass outside the excluded token is 0 (one-hot q)    */
#define SPECHUB_ST_ZERO_MASS_DRAFT 8u /* a performed acceptance test had denominator 0: rejected   */
#define SPECHUB_ST_ZERO_RESIDUAL 16u  /* residual mass 0 on rejection: the token was drawn from p  */
#define SPECHUB_ST_STATS 64u          /* *_stats verification: the row's draft statistics are not those of its draft logits and temperature: output -1 */
#define SPECHUB_ST_INTERNAL 32u       /* a bulk copy into shared memory did not arrive within the kernel's bounded wait */

/* descriptor flags: how many CTAs of a thread-block cluster share one row in the large-vocabulary
 * bf16 kernels (a tuning hint; results do not depend on it beyond fp32 summation order).  At most
 * one of the three may be set; none = the library chooses: one CTA per row, and for RRS / RRSw the
 * verification passes read the rows through per-warp rings of bulk copies into shared memory
 * (cp.async.bulk) -- same results, bit for bit, as SPECHUB_FLAG_SPLIT_1, whose loads go to registers. */
#define SPECHUB_FLAG_SPLIT_1 1u
#define SPECHUB_FLAG_SPLIT_2 2u
#define SPECHUB_FLAG_SPLIT_4 4u
/* Verification with the exponentials resident on chip (tensor memory + shared memory): one read of the
 * row pair from HBM instead of two.  Not combined with a split flag.  Applies to the same shapes as the
 * large-vocabulary bf16 kernels, up to 262144 ids; other shapes ignore it.  These kernels allocate
 * tensor memory (tcgen05.alloc) for the lifetime of a CTA and release it before the CTA ends; among
 * themselves they never ask an SM for more than it has.  Another kernel that holds tensor memory on
 * the same SMs at the same time (a tensor-core GEMM on another stream) makes their CTAs wait until its
 * CTAs have finished -- a delay, not a deadlock. */
#define SPECHUB_FLAG_RESIDENT 8u

/* node kinds */
#define SPECHUB_NODE_VERIFY 0 /* run the accept/reject tests on the node's two drafts         */
#define SPECHUB_NODE_LEAF 1   /* no drafts below: draw the bonus token from p with u_res       */

typedef struct spechub_desc {
    uint32_t struct_size; /* sizeof(spechub_desc)                                            */
    uint32_t version;     /* SPECHUB_ABI_VERSION                                             */
    int32_t batch;        /* sequences B                                                     */
    int32_t nodes;        /* tree nodes per sequence N, level order, node 0 = root           */
    int32_t vocab;        /* V >= 2                                                          */
    int32_t k;            /* drafts per node: 2 for SpecHub (Section 4); 2..SPECHUB_MAX_K for
                             RRS / RRSw (Algorithm 1 is stated for k candidates)             */
    int32_t dtype;        /* SPECHUB_F32 or SPECHUB_BF16 logits                              */
    int32_t levels;       /* longest root-to-leaf path in nodes; bounds the walk, row length
                             of the path outputs                                             */
    int64_t stride_seq;   /* elements between consecutive sequences of a logits tensor       */
    int64_t stride_node;  /* elements between consecutive nodes                              */
    float temperature;    /* T > 0, used when temperature_per_seq is NULL                    */
    const float *temperature_per_seq; /* device [batch] or NULL                               */
    const int32_t *child;   /* device [nodes][2]: node reached by accepting draft i, < 0 = none;
                               NULL = complete binary tree in heap order, child i of n is 2n+1+i */
    const uint8_t *node_kind; /* device [nodes]: SPECHUB_NODE_*; NULL = every node verifies    */
    uint32_t flags;       /* SPECHUB_FLAG_* bits; 0 = library defaults                        */
} spechub_desc;

/* Per-node outputs, each a device array [batch][nodes] (x trailing count).
 * accept_idx and token are required; the others may be NULL.  When beta and rate are both NULL
 * no probability is reported, and a row whose first test accepts is finished after the first
 * pass over its logits (the transport sums could not change its outcome). */
typedef struct spechub_node_out {
    int32_t *accept_idx; /* 0 / 1: child whose draft was accepted; -1: rejected, leaf or flagged */
    int32_t *token;      /* token emitted at this node: accepted draft, residual or leaf draw;
                            -1 on SPECHUB_ST_NONFINITE / SPECHUB_ST_TOKEN_RANGE                */
    int32_t *hub;        /* a (SpecHub), -1 for RRS / RRSw and leaves                          */
    float *beta;         /* [..][2] acceptance probability of test 1 / test 2 for this pair     */
    float *rate;         /* [..][3] row masses: accept child 0, accept child 1, reject          */
    uint32_t *status;    /* SPECHUB_ST_* bits                                                   */
} spechub_node_out;

/* Per-sequence outputs of the tree walk (Figure 2); any pointer may be NULL,
 * and a NULL seq_out skips the walk. */
typedef struct spechub_seq_out {
    int32_t *n_accepted;  /* [batch] accepted draft tokens on the path                         */
    int32_t *n_emitted;   /* [batch] tokens emitted this step (accepted + residual/bonus)       */
    int32_t *path_nodes;  /* [batch][levels] visited nodes, padded with -1                      */
    int32_t *path_tokens; /* [batch][levels] emitted tokens, padded with -1                     */
} spechub_seq_out;

/*
 * Draft step of SpecHub (Section 4; Algorithm 3, "Sample draft tokens
 * x1, x2 ~ Q").  For every node: a = argmax of the draft logits (lowest id on
 * ties); (x1, x2) is drawn from the sparse joint distribution
 *   Q(x, a) = q(x),   Q(a, x) = q(a) q(x) / (1 - q(a))   (x != a), 0 elsewhere:
 * x1 is drawn from q with u_d1; if x1 != a then x2 = a, otherwise x2 is drawn
 * with u_d2 from q restricted to ids != a.
 *   draft_logits  [B][N][V] of desc->dtype        (in)
 *   uniforms      [B][N][5]                       (in; entries 0 and 1 are used)
 *   draft_tokens  [B][N][2]                       (out)
 *   hub           [B][N]                          (out, may be NULL)
 *   draft_prob    [B][N][2] = (q(a), Q(x1, x2))   (out, may be NULL)
 *   status        [B][N]                          (out, may be NULL)
 * A one-hot q (1 - q(a) = 0) yields (a, lowest id != a) with
 * SPECHUB_ST_DEGENERATE_Q; a flagged NONFINITE row yields (-1, -1).
 */
int spechub_draft_sample(const spechub_desc *desc, const void *draft_logits, const float *uniforms,
                         int32_t *draft_tokens, int32_t *hub, float *draft_prob, uint32_t *status,
                         void *stream);

/*
 * Draft step of RRS / RRSw (Algorithm 1, "Generate k samples ... independently
 * or without replacement from q").  x1 is drawn from q with u_d1; x2 from q
 * with u_d2 (without_replacement = 0) or from q with q(x1) set to 0
 * (without_replacement = 1).  Arguments as above.  For desc->k > 2 draw i uses
 * u_di and, without replacement, q with q(x1..x_{i-1}) set to 0; if nothing is
 * left to draw from, the lowest id not drawn yet is returned with
 * SPECHUB_ST_DEGENERATE_Q.
 */
int rrs_draft_sample(const spechub_desc *desc, const void *draft_logits, const float *uniforms,
                     int without_replacement, int32_t *draft_tokens, uint32_t *status, void *stream);

/*
 * Verification with SpecHub (Algorithm 3 with Algorithm 2, Appendix B.1; the
 * closed-form transport of Section 4) of every node, then the tree walk
 * (Figure 2).  With c = q(a) / (1 - q(a)) and, over ids y != a,
 *   S1 = sum max(q - p, 0),  S2 = sum max(c q - max(p - q, 0), 0),
 *   R  = sum max(max(p - q, 0) - c q, 0):
 *   pair (x, a): accept x (child 0) iff r1 q(x) < p(x); else accept a (child 1)
 *                iff r2 S1 < max(p(a) - S2, 0);
 *   pair (a, x): accept x (child 1) iff r1 c q(x) < max(p(x) - q(x), 0); else
 *                accept a (child 0) iff r2 S2 < p(a);
 *   otherwise the token is drawn with u_res from the residual
 *   max(max(p - q, 0) - c q, 0), which has no mass on a.
 * rate = (sum min(p,q) + min(p(a), S2),
 *         sum min(max(p-q,0), c q) + min(max(p(a) - S2, 0), S1),  R).
 * A pair that does not contain the hub exactly once is flagged TOKEN_RANGE.
 * Leaf nodes (desc->node_kind) read only target_logits.
 *   target_logits, draft_logits [B][N][V]   (in)
 *   draft_tokens [B][N][2], uniforms [B][N][5] (in; entries 2, 3, 4 are used)
 *   node_out (required), seq_out (may be NULL)
 *   workspace: device scratch of at least spechub_workspace_bytes(desc) bytes;
 *   may be NULL when that is 0.
 */
int spechub_verify_tree(const spechub_desc *desc, const void *target_logits,
                        const void *draft_logits, const int32_t *draft_tokens,
                        const float *uniforms, const spechub_node_out *node_out,
                        const spechub_seq_out *seq_out, void *workspace, size_t workspace_bytes,
                        void *stream);

/*
 * Draft statistics handed from the draft step to verification.
 *
 * Both steps of a decoding iteration read the same draft logits: the draft step
 * to sample x1, x2 ~ Q (Algorithm 3; Algorithm 1 for RRS / RRSw), verification
 * for a = argmax q, q(a) and the normaliser of q (Section 4).  The draft step
 * knows all three once it has read the row.  spechub_draft_sample_stats /
 * rrs_draft_sample_stats are spechub_draft_sample / rrs_draft_sample that also
 * leave, per (sequence, node), a 16-byte record (maximum draft logit, argmax,
 * sum of the other exponentials, a tag) in draft_stats: device memory of
 * spechub_draft_stats_bytes(desc) bytes, 16-byte aligned, owned by the caller.
 * spechub_verify_tree_stats / rrs_verify_tree_stats are spechub_verify_tree /
 * rrs_verify_tree that take those records instead of making their first pass
 * over the draft row: that pass then reads the target row only (half its
 * bytes, half its exponentials).  Everything else -- arguments, outputs,
 * status bits, the tree walk -- is as in the plain calls, and the results agree
 * with theirs up to the fp32 summation order of the draft row's normaliser
 * (accept / reject decisions can differ only where the plain call's decision
 * is itself within rounding of its threshold).
 *
 * The records are opaque and tied to the library build, the descriptor (shape,
 * strides, dtype, temperature, flags) and the draft logits they were made
 * from; they may be used by any number of verification calls until those
 * change.  A record that cannot be this row's -- wrong tag (other temperature
 * or library), argmax out of range, or a draft logit at the argmax other than
 * the recorded maximum -- flags the row SPECHUB_ST_STATS with outputs -1; other
 * inconsistencies are the caller's responsibility.  Only the default path of
 * the large-vocabulary bf16 shapes (no SPECHUB_FLAG_*, k = 2, rows 16-byte
 * aligned, vocab % 8 == 0, vocab >= 8192) writes and reads records; on every
 * other path the draft call clears draft_stats and the verification call
 * ignores it, so the four calls may be used unconditionally.
 */
size_t spechub_draft_stats_bytes(const spechub_desc *desc);
int spechub_draft_sample_stats(const spechub_desc *desc, const void *draft_logits, const float *uniforms,
                               int32_t *draft_tokens, int32_t *hub, float *draft_prob, uint32_t *status,
                               void *draft_stats, void *stream);
int rrs_draft_sample_stats(const spechub_desc *desc, const void *draft_logits, const float *uniforms,
                           int without_replacement, int32_t *draft_tokens, uint32_t *status,
                           void *draft_stats, void *stream);
int spechub_verify_tree_stats(const spechub_desc *desc, const void *target_logits, const void *draft_logits,
                              const void *draft_stats, const int32_t *draft_tokens, const float *uniforms,
                              const spechub_node_out *node_out, const spechub_seq_out *seq_out,
                              void *workspace, size_t workspace_bytes, void *stream);
int rrs_verify_tree_stats(const spechub_desc *desc, const void *target_logits, const void *draft_logits,
                          const void *draft_stats, const int32_t *draft_tokens, const float *uniforms,
                          int without_replacement, const spechub_node_out *node_out,
                          const spechub_seq_out *seq_out, void *workspace, size_t workspace_bytes,
                          void *stream);

/*
 * Verification with Recursive Rejection Sampling (Algorithm 1) of every node,
 * then the tree walk.  With A1 = sum max(p - q, 0) and q1 = q (RRS) or q with
 * q(x1) zeroed and renormalised (RRSw):
 *   accept x1 (child 0) iff r1 q(x1) < p(x1); else accept x2 (child 1) iff
 *   r2 A1 q1(x2) < max(p(x2) - q(x2), 0); otherwise draw with u_res from
 *   max(max(p - q, 0) - A1 q1, 0).
 * rate = (sum min(p,q), A1 - W2, W2), W2 the mass of that last residual (for
 * RRSw the last two are for the given x1).  hub is written as -1.
 * For desc->k > 2 the loop of Algorithm 1 runs over all k drafts: with P_0 = p,
 * m_0 = 1, draft x_j is accepted iff r_j m_{j-1} q_j(x_j) < P_{j-1}(x_j), where
 * q_j = q (RRS) or q with q(x_1..x_{j-1}) zeroed and renormalised (RRSw),
 * P_j = max(P_{j-1} - m_{j-1} q_j, 0) and m_j = sum P_j; the residual token is
 * drawn from P_k; rate[j] = m_j - m_{j+1} (j < k), rate[k] = m_k.
 * For desc->k > 2 on bf16 rows that are 16-byte aligned with 8192 <= vocab <=
 * 262144, vocab % 8 == 0 and no split flag, the stages run over exponentials
 * kept in the SMs' tensor memory and shared memory (see SPECHUB_FLAG_RESIDENT
 * for what that means for other work on the GPU).
 */
int rrs_verify_tree(const spechub_desc *desc, const void *target_logits, const void *draft_logits,
                    const int32_t *draft_tokens, const float *uniforms, int without_replacement,
                    const spechub_node_out *node_out, const spechub_seq_out *seq_out,
                    void *workspace, size_t workspace_bytes, void *stream);

/*
 * SpecHub, RRS and RRSw side by side on the same p, q and uniforms (the
 * comparison of Section 5: all methods verify the same draft tree shapes).
 * Results are those of spechub_draft_sample / rrs_draft_sample(0) /
 * rrs_draft_sample(1), bit for bit; index 0 = SpecHub, 1 = RRS, 2 = RRSw.
 * Where the rows are bf16, 16-byte aligned, vocab % 8 == 0 and vocab >= 8192,
 * one kernel reads q once for the three methods (x1 is the same draw for all,
 * since they share u_d1); otherwise the three calls are made one after another.
 * desc->k must be 2.  draft_tokens[m] is [B][N][2] (out, required);
 * status may be NULL or hold three pointers, each of which may be NULL;
 * hub and draft_prob are SpecHub's.
 */
int mdsd_compare_draft_sample(const spechub_desc *desc, const void *draft_logits, const float *uniforms,
                              int32_t *const draft_tokens[3], int32_t *hub, float *draft_prob,
                              uint32_t *const status[3], void *stream);

/*
 * Verification by the three methods from shared reads of p and q, then one tree
 * walk per method.  node_out[m] (three records, accept_idx and token required
 * in each) and seq_out (NULL, or three records) receive what
 * spechub_verify_tree / rrs_verify_tree(0) / rrs_verify_tree(1) would write,
 * bit for bit, given draft_tokens[m] ([B][N][2], in) and the same uniforms.
 * On the shapes named above one kernel makes three passes over a row pair
 * (common max / sum / hub; S1, S2, R, A1 and RRSw's renormaliser; the two
 * second-stage residual masses of Algorithm 1) instead of eight.
 */
int mdsd_compare_verify_tree(const spechub_desc *desc, const void *target_logits, const void *draft_logits,
                             const int32_t *const draft_tokens[3], const float *uniforms,
                             const spechub_node_out node_out[3], const spechub_seq_out *seq_out,
                             void *workspace, size_t workspace_bytes, void *stream);

/*
 * The three-method calls with the hand-over of draft statistics (see
 * spechub_draft_sample_stats): one record per row serves the three methods.
 * Results are those of the per-method *_stats calls, bit for bit.
 */
int mdsd_compare_draft_sample_stats(const spechub_desc *desc, const void *draft_logits, const float *uniforms,
                                    int32_t *const draft_tokens[3], int32_t *hub, float *draft_prob,
                                    uint32_t *const status[3], void *draft_stats, void *stream);
int mdsd_compare_verify_tree_stats(const spechub_desc *desc, const void *target_logits, const void *draft_logits,
                                   const void *draft_stats, const int32_t *const draft_tokens[3],
                                   const float *uniforms, const spechub_node_out node_out[3],
                                   const spechub_seq_out *seq_out, void *workspace, size_t workspace_bytes,
                                   void *stream);

/*
 * Tree walk alone (Figure 2) over per-node results already in device memory:
 * accept_idx, token [B][N] (in), seq_out as in spechub_verify_tree.  Used after
 * the vocabulary-sharded phases below, once the tokens have been exchanged.
 */
int spechub_walk_tree(const spechub_desc *desc, const int32_t *accept_idx, const int32_t *token,
                      const spechub_seq_out *seq_out, void *stream);

/*
 * SpecHub with the vocabulary axis sharded over ranks (each rank's LM head
 * produces the logits of a contiguous id range).  The paper has no counterpart:
 * it states the method on whole distributions (Section 4, Algorithm 3); these
 * calls compute the same quantities from slices.  desc->vocab is the width of
 * this rank's slice, the logits pointers are its slices ([B][N][vocab] with the
 * descriptor's strides); token ids everywhere are global.  desc->k must be 2.
 *
 * The caller runs, per rank and in lockstep:
 *   draft:  spechub_shard_stats(target = NULL) -> all-gather of stats in rank
 *           order -> spechub_shard_draft -> element-wise maximum of cand over
 *           ranks -> spechub_shard_draft_finish;
 *   verify: spechub_shard_stats -> all-gather -> spechub_shard_sums ->
 *           all-gather -> spechub_shard_decide -> element-wise maximum of
 *           node_out->token over ranks -> spechub_walk_tree.
 * stats, sums: [B][N][8] floats (out); gathered_*: [nranks][B][N][8] (in).
 * All ranks take identical decisions (the gathered partials are merged in rank
 * order everywhere); a residual or bonus token is drawn by the rank whose slice
 * holds the inverse-CDF target and is -2 on the others until the maximum is
 * taken.  Results agree with spechub_draft_sample / spechub_verify_tree on the
 * concatenated rows up to fp32 summation order.
 */
typedef struct {
    int32_t rank, nranks;     /* 0 <= rank < nranks <= 64 */
    int32_t id_offset;        /* global id of this slice's first token */
    int32_t vocab_total;      /* sum of the slices' widths */
} spechub_shard;

int spechub_shard_stats(const spechub_desc *desc, const spechub_shard *shard, const void *target_slice,
                        const void *draft_slice, float *stats, void *stream);
int spechub_shard_sums(const spechub_desc *desc, const spechub_shard *shard, const void *target_slice,
                       const void *draft_slice, const int32_t *draft_tokens, const float *gathered_stats,
                       float *sums, void *stream);
int spechub_shard_decide(const spechub_desc *desc, const spechub_shard *shard, const void *target_slice,
                         const void *draft_slice, const int32_t *draft_tokens, const float *uniforms,
                         const float *gathered_stats, const float *gathered_sums,
                         const spechub_node_out *node_out, void *stream);
/* cand [B][N][2] (out): x1 and the second draw of a pair (a, x); -2 where another rank draws. */
int spechub_shard_draft(const spechub_desc *desc, const spechub_shard *shard, const void *draft_slice,
                        const float *uniforms, const float *gathered_stats, int32_t *cand, void *stream);
/* cand_max: cand after the maximum over ranks; draft_tokens [B][N][2], hub, status as in spechub_draft_sample. */
int spechub_shard_draft_finish(const spechub_desc *desc, const spechub_shard *shard,
                               const float *gathered_stats, const int32_t *cand_max,
                               int32_t *draft_tokens, int32_t *hub, uint32_t *status, void *stream);

/*
 * RRS / RRSw (Algorithm 1, k = 2) on vocabulary-sharded logits: the phases above
 * for the comparison methods.  As with SpecHub the paper has no counterpart.
 *   verify: spechub_shard_stats -> all-gather -> rrs_shard_sums(gathered_sums =
 *           NULL): A1 and RRSw's renormaliser over the slice, p and q at x1, x2
 *           from their owners -> all-gather -> rrs_shard_sums(gathered_sums):
 *           the second-stage residual mass W2 over the slice -> all-gather ->
 *           rrs_shard_decide -> maximum of node_out->token -> spechub_walk_tree.
 *   draft:  spechub_shard_stats(target = NULL) -> all-gather ->
 *           rrs_shard_draft(cand_max = ex1_max = NULL): x1 ~ q and, for RRS, x2 ~ q
 *           (each -2 where another rank draws); ex1 [B][N] = the exponential of
 *           x1's logit on the row's scale from its owner, -1 elsewhere -> maximum
 *           of cand and of ex1 over ranks -> RRSw only: rrs_shard_draft(cand_max,
 *           ex1_max): x2 ~ q with q(x1) set to 0 -> maximum of cand ->
 *           rrs_shard_draft_finish.
 * out, gathered_*: as for SpecHub ([B][N][8] and [nranks][B][N][8] floats).
 */
int rrs_shard_sums(const spechub_desc *desc, const spechub_shard *shard, int without_replacement,
                   const void *target_slice, const void *draft_slice, const int32_t *draft_tokens,
                   const float *gathered_stats, const float *gathered_sums, float *out, void *stream);
int rrs_shard_decide(const spechub_desc *desc, const spechub_shard *shard, int without_replacement,
                     const void *target_slice, const void *draft_slice, const int32_t *draft_tokens,
                     const float *uniforms, const float *gathered_stats, const float *gathered_sums,
                     const float *gathered_w2, const spechub_node_out *node_out, void *stream);
int rrs_shard_draft(const spechub_desc *desc, const spechub_shard *shard, int without_replacement,
                    const void *draft_slice, const float *uniforms, const float *gathered_stats,
                    const int32_t *cand_max, const float *ex1_max, int32_t *cand, float *ex1, void *stream);
int rrs_shard_draft_finish(const spechub_desc *desc, const spechub_shard *shard, int without_replacement,
                           const float *gathered_stats, const int32_t *cand_max, int32_t *draft_tokens,
                           uint32_t *status, void *stream);

/*
 * SpecHub verification and tree walk for callers that cannot allocate device
 * memory.  (The paper has no counterpart: this is a property of the library,
 * not of the method.)  Inference servers that reserve the whole GPU for their
 * own pools at start-up, code running inside another framework's memory plan,
 * and real-time loops that may not enter the driver's allocator all fall in
 * this class: for them every cudaMalloc is either forbidden or a stall.  This
 * call runs the phase kernels of the vocabulary-sharded path as a single rank
 * that holds the whole vocabulary -- stats, sums, decide, walk, back to back
 * on `stream` -- and keeps the two per-row records those phases hand to one
 * another (64 bytes per row) in a static array inside the library instead of
 * buffers somebody would have to allocate.  It calls no cudaMalloc, cudaFree or
 * other allocating routine.  Inputs and outputs are the caller's, with the
 * meaning they have in spechub_verify_tree (desc->k must be 2; seq_out may be
 * NULL); results equal spechub_verify_tree's up to fp32 summation order.
 *
 * Limits and rules:
 *   - batch * nodes <= SPECHUB_STATIC_MAX_ROWS, else SPECHUB_ERR_TOO_LARGE and
 *     nothing is launched.  The array takes SPECHUB_STATIC_MAX_ROWS * 64 bytes
 *     (1 MiB) of every GPU that loads the library, until the process exits.
 *   - The first call on each device looks the array's device address up (with
 *     that device current) and keeps it; make that first call outside any
 *     stream capture.  A failed look-up returns SPECHUB_ERR_LAUNCH.
 *   - All calls on a device share the array.  Each call rewrites every record
 *     it reads, so nothing has to be cleared and a call never sees another
 *     call's leftovers; but two calls that overlap on the GPU (different
 *     streams, no dependency between them) race on it.  Order them.
 */
#define SPECHUB_STATIC_MAX_ROWS 16384
int spechub_verify_tree_static(const spechub_desc *desc, const void *target_logits,
                               const void *draft_logits, const int32_t *draft_tokens,
                               const float *uniforms, const spechub_node_out *node_out,
                               const spechub_seq_out *seq_out, void *stream);

/* Scratch bytes the two verify calls need for this descriptor (0 is possible). */
size_t spechub_workspace_bytes(const spechub_desc *desc);

/* Static, NUL-terminated description of a return code. */
const char *spechub_status_string(int code);

/* SPECHUB_ABI_VERSION the library was built with. */
int spechub_abi_version(void);

#ifdef __cplusplus
}
#endif
#endif /* SPECHUB_H_ */
