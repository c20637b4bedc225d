/*
 * branch_attn.h -- C ABI of the B200 (sm_100a) draft-branch-attention library.
 *
 * The operation (paper Section 3.2, "Branch Attention under Context
 * Parallelism"): over a packed batch of variable-length main sequences, every
 * main query attends causally inside its own sequence, and every branch query
 * attends to two key sets -- the causal prefix of its main sequence up to and
 * including its anchor, and the keys of its own branch under a branch-local
 * mask (EAGLE-3 chain, DFlash block, or a tree given by parent indices).
 * Partial results over disjoint key sets are combined with Eq. (lse-merge);
 * the backward pass accumulates gradients over key chunks.
 *
 * Conventions
 *   - Every pointer marked "device" is CUDA device memory owned by the caller;
 *     the library allocates no device memory.  `stream` is a cudaStream_t
 *     passed as void* (NULL = the legacy default stream).  Data calls only
 *     enqueue work on that stream and return; ba_plan_create synchronises the
 *     stream once to read back its validation result.
 *   - Tensors are contiguous, row-major, innermost dimension head_dim:
 *       q_main  [N, h_q, D]      q_branch [M, h_q, D]
 *       k, v    [N + M, h_kv, D] main rows first, then branch tokens
 *       O, dO   [N + M, h_q, D]  LSE [N + M, h_q] (fp32, natural log)
 *     Branch tokens are stored branch-major in anchor order.  Query head h uses
 *     KV head h / (h_q / h_kv).
 *   - Element type of q/k/v/O/dO is ba_problem_t.dtype.  Supported: BA_FP32 and
 *     BA_BF16 with head_dim 64 or 128; a branch holds at most 64 tokens.
 *   - Every function returns BA_OK (0) or a negative ba_status; nothing throws.
 */
#ifndef BRANCH_ATTN_H_
#define BRANCH_ATTN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum ba_status {
    BA_OK = 0,
    BA_EINVAL = -1,        /* bad argument (NULL pointer, negative size, bad range) */
    BA_EUNSUPPORTED = -2,  /* dtype / head_dim / branch length not supported */
    BA_EWORKSPACE = -3,    /* plan memory or workspace too small / misaligned */
    BA_EMETA = -4,         /* device-side validation of the metadata failed */
    BA_ECUDA = -5,         /* a CUDA runtime call failed; see ba_last_cuda_error */
    BA_ETIMEOUT = -6       /* a bounded device-side wait expired */
} ba_status;

enum { BA_BF16 = 0, BA_FP32 = 1 };
enum { BA_MASK_CHAIN = 0, BA_MASK_BLOCK = 1, BA_MASK_TREE = 2 };
enum { BA_PART_MAIN = 1, BA_PART_BRANCH = 2 };
enum { BA_OP_FWD = 0, BA_OP_BWD = 1, BA_OP_BWD_FUSED = 2, BA_OP_BWD_DEPTH = 3 };
enum { BA_STAGE_PREP = 1, BA_STAGE_DQ = 2, BA_STAGE_DKDV = 4, BA_STAGE_ALL = 7,
       BA_STAGE_FUSED = 8, BA_STAGE_ALL_FUSED = 9 };

/* Which kernels a plan uses: the tensor-core (tcgen05) path where the shape
 * allows it (bf16, head_dim 128), or the plain-FMA path (any supported shape;
 * the only path for fp32). */
enum { BA_IMPL_AUTO = 0, BA_IMPL_SIMT = 1, BA_IMPL_TC = 2 };

typedef struct ba_problem {
    int64_t n_main;                /* N: packed main tokens */
    int64_t n_branch;              /* M: branch tokens (sum of branch lengths) */
    int32_t num_seqs;              /* B */
    int32_t num_branches;          /* A */
    int32_t h_q, h_kv, head_dim;
    int32_t dtype;                 /* BA_BF16 / BA_FP32 */
    float softmax_scale;           /* 0 => 1/sqrt(head_dim) */
    int32_t mask_kind;             /* BA_MASK_* */
    int32_t uniform_len;           /* > 0: every branch has this many tokens and
                                      branch_offsets may be NULL */
    int32_t impl;                  /* BA_IMPL_* */
    const int32_t *cu_seqlens;     /* device [B+1], cu[0] = 0, cu[B] = N, non-decreasing */
    const int32_t *anchor_idx;     /* device [A], global packed index in [0, N), non-decreasing */
    const int32_t *branch_offsets; /* device [A+1] token offsets (0 .. M); may be NULL with
                                      uniform_len > 0 or with A = 0 (it is not read then) */
    const int32_t *parent;         /* device [M], BA_MASK_TREE only: branch-local parent index,
                                      -1 = root, parent[i] < i */
} ba_problem_t;

typedef struct ba_plan ba_plan_t;  /* opaque; host object owned by the library */

const char *ba_status_string(int status);
/* cudaError_t of the most recent failed CUDA call on this thread (0 if none). */
int ba_last_cuda_error(void);

/*
 * Metadata builder ("varlen packing and anchor / branch-mask metadata").
 * ba_plan_bytes: device bytes the plan needs for the given sizes (only the
 *   integer fields of *p are read).
 * ba_plan_create: validates *p, derives per-row key bounds, per-token branch
 *   start and 64-bit branch masks, per-key query ranges (for dK/dV) into
 *   `plan_mem` (device, 256-byte aligned, >= ba_plan_bytes), synchronises
 *   `stream`, and returns a host handle in *out.  The metadata arrays in *p
 *   must stay alive only until this call returns; plan_mem until
 *   ba_plan_destroy.  Bad metadata (unsorted anchors, anchor out of range,
 *   parent[i] >= i, branch longer than 64, offsets not ending at M) gives
 *   BA_EMETA and no plan; no data kernel ever sees unvalidated metadata.
 * ba_plan_destroy: frees the host handle (not plan_mem).
 */
size_t ba_plan_bytes(const ba_problem_t *p);
int ba_plan_create(const ba_problem_t *p, void *plan_mem, size_t plan_bytes, void *stream,
                   ba_plan_t **out);
int ba_plan_destroy(ba_plan_t *plan);

/* Scratch bytes (device, 256-byte aligned) that `op` needs; may be 0.
 * BA_OP_BWD_FUSED = BA_OP_BWD plus an fp32 dQ accumulator of (N + M) * h_q * head_dim
 * floats: what BA_STAGE_FUSED needs when the gradients are written in the input
 * dtype (accumulate = 0).  BA_OP_BWD_DEPTH = BA_OP_BWD plus an fp32 dQ accumulator of
 * num_branches * h_q * head_dim floats (branch_attn_bwd_depth). */
size_t ba_workspace_bytes(const ba_plan_t *plan, int op);

/* Exact number of (query row, visible key) pairs per query head of the whole
 * problem, as counted by the metadata builder (host value). */
int64_t ba_plan_pairs(const ba_plan_t *plan);

/* Which kernels the plan resolved to: BA_IMPL_SIMT or BA_IMPL_TC. */
int ba_plan_impl(const ba_plan_t *plan);

/* Synchronises `stream` and reports whether any kernel launched with this plan
 * gave up a bounded device-side wait since the last check: BA_OK or BA_ETIMEOUT
 * (the outputs of such a launch are undefined).  The flag is cleared. */
int ba_plan_check(ba_plan_t *plan, void *stream);

/*
 * Self-test of the bounded device-side waits (no counterpart in the paper: every
 * barrier wait inside the tensor-core kernels gives up after a cycle limit instead of
 * spinning forever, and this shows that path working).  Launches one warp that
 * waits, for at most `limit_cycles` SM cycles (1 .. 1e8, i.e. well under a tenth of
 * a second), on a barrier nobody signals; the kernel then returns normally and
 * leaves BA_ETIMEOUT in the plan's status word, which the next ba_plan_check
 * reports and clears.  Nothing else is touched; later calls work as usual.
 */
int ba_selftest_bounded_wait(ba_plan_t *plan, int64_t limit_cycles, void *stream);

/*
 * Forward, both key sets fused in one online-softmax pass (Section 3.2: the
 * causal main-sequence component and the branch-local component; Eq.
 * (lse-merge) applied tile by tile).
 *   q_main may be NULL: only branch queries are computed (rows [N, N+M) of the
 *   outputs are written).  O has the input dtype, LSE is fp32.
 */
int branch_attn_fwd(const ba_plan_t *plan, const void *q_main, const void *q_branch,
                    const void *k, const void *v, void *O, float *LSE,
                    void *workspace, size_t ws_bytes, void *stream);

/*
 * Partial forward over an explicit key set: one ring step of the packed
 * zigzag-ring layout of Section 3.2, emulated on one GPU.
 *   queries: main rows [qm_begin, qm_end) and the tokens of branches
 *            [br_begin, br_end); either range may be empty.
 *   keys:    main keys [kv_begin, kv_end) if parts & BA_PART_MAIN (still limited
 *            to each query's causal prefix), own-branch keys if parts &
 *            BA_PART_BRANCH.
 *   outputs: compact, fp32: O_part [(qm_end-qm_begin) + T, h_q, D] and
 *            LSE_part [.., h_q], main range first, then the T branch tokens.  A
 *            query that sees no key in the set gets LSE = -inf and O = 0.
 */
int branch_attn_fwd_partial(const ba_plan_t *plan, const void *q_main, const void *q_branch,
                            const void *k, const void *v,
                            int64_t qm_begin, int64_t qm_end, int64_t br_begin, int64_t br_end,
                            int64_t kv_begin, int64_t kv_end, int parts,
                            float *O_part, float *LSE_part,
                            void *workspace, size_t ws_bytes, void *stream);

/*
 * The same partial forward with Eq. (lse-merge) applied in the kernel's epilogue:
 * (O_acc, LSE_acc), compact fp32 as above and holding the result of the key sets
 * seen so far (first filled by branch_attn_fwd_partial), are replaced by their
 * merge with this call's partial result.  Saves the separate lse_merge pass of a
 * ring step.  Tensor-core plans only (BA_EUNSUPPORTED otherwise).
 */
int branch_attn_fwd_partial_merge(const ba_plan_t *plan, const void *q_main, const void *q_branch,
                                  const void *k, const void *v,
                                  int64_t qm_begin, int64_t qm_end, int64_t br_begin, int64_t br_end,
                                  int64_t kv_begin, int64_t kv_end, int parts,
                                  float *O_acc, float *LSE_acc,
                                  void *workspace, size_t ws_bytes, void *stream);

/*
 * Eq. (lse-merge):  l = log(e^la + e^lb),  O = e^(la-l) Oa + e^(lb-l) Ob,
 * evaluated in max-subtracted form; la = lb = -inf gives l = -inf, O = 0.
 *   rows_heads = number of (row, head) pairs; O_a/O_b fp32 [rows_heads, d],
 *   LSE_* fp32 [rows_heads].  O_out has out_dtype (BA_FP32 / BA_BF16) and may
 *   alias O_a when out_dtype is BA_FP32; LSE_out may alias LSE_a or be NULL.
 */
int lse_merge(int64_t rows_heads, int d, const float *O_a, const float *LSE_a,
              const float *O_b, const float *LSE_b, void *O_out, int out_dtype,
              float *LSE_out, void *stream);

/*
 * Backward (Section 3.2: "replays the same K/V ring and accumulates gradients
 * locally").  Loss = sum_r <dO_r, O_r>.  O and LSE are the COMPLETE forward
 * results (after all merges), global layout; the query / key ranges and
 * `parts` select which (query, key) terms this call adds, exactly as in
 * branch_attn_fwd_partial.  Full ranges with accumulate = 0 give the whole
 * gradient in one call.
 *   accumulate = 0: dQ_main [N,h_q,D], dQ_branch [M,h_q,D], dK, dV [N+M,h_kv,D]
 *     have the input dtype; rows of the selected query range (dQ) and of the
 *     selected key set (dK, dV) are overwritten, all other rows untouched.
 *   accumulate = 1: the four outputs are fp32 and the terms are added to them
 *     (the caller zeroes them first and converts with ba_finalize_grads).
 *   q_main NULL: branch queries only (dQ_main untouched, may be NULL).
 *   workspace: ba_workspace_bytes(plan, BA_OP_BWD).
 */
int branch_attn_bwd(const ba_plan_t *plan, const void *q_main, const void *q_branch,
                    const void *k, const void *v, const void *O, const float *LSE,
                    const void *dO,
                    int64_t qm_begin, int64_t qm_end, int64_t br_begin, int64_t br_end,
                    int64_t kv_begin, int64_t kv_end, int parts, int accumulate,
                    void *dQ_main, void *dQ_branch, void *dK, void *dV,
                    void *workspace, size_t ws_bytes, void *stream);

/*
 * The same backward, one stage at a time (same arguments, same workspace):
 *   BA_STAGE_PREP  delta = <dO, O> and -LSE log2(e) of the selected query rows
 *                  into the workspace (must precede the other two stages),
 *   BA_STAGE_DQ    dQ of the selected query rows,
 *   BA_STAGE_DKDV  dK, dV of the selected key set.
 * `stages` is a bit mask; BA_STAGE_ALL is branch_attn_bwd.  Lets a caller time
 * or overlap the three kernels separately.
 *   BA_STAGE_FUSED replaces BA_STAGE_DQ | BA_STAGE_DKDV (it cannot be combined
 *                  with them) by ONE key-stationary kernel that forms S and dP
 *                  once per tile pair (10 D flop per visible pair instead of 14 D)
 *                  and sums dQ into its fp32 accumulator with atomic adds.
 *                  Needs the tensor-core kernels, else BA_EUNSUPPORTED.  With
 *                  accumulate = 0 the workspace must hold
 *                  ba_workspace_bytes(plan, BA_OP_BWD_FUSED) (all stages of one
 *                  backward use the same workspace): dQ is summed there in fp32
 *                  and converted at the end.  dK and dV stay bit-reproducible;
 *                  the last bits of dQ depend on the order in which the key
 *                  tiles arrive.
 *   BA_STAGE_ALL_FUSED = BA_STAGE_PREP | BA_STAGE_FUSED.
 */
int branch_attn_bwd_stages(const ba_plan_t *plan, const void *q_main, const void *q_branch,
                           const void *k, const void *v, const void *O, const float *LSE,
                           const void *dO,
                           int64_t qm_begin, int64_t qm_end, int64_t br_begin, int64_t br_end,
                           int64_t kv_begin, int64_t kv_end, int parts, int accumulate,
                           void *dQ_main, void *dQ_branch, void *dK, void *dV,
                           void *workspace, size_t ws_bytes, void *stream, int stages);

/*
 * Backward without caller-provided scratch.  (No counterpart in the paper: this
 * is a packaging variant of branch_attn_bwd, same arithmetic, same results.)
 *
 * For callers that cannot allocate device memory when they call -- code running
 * inside a fixed, pre-planned memory arena, or under a framework hook where
 * allocator calls are forbidden -- and so have nothing to pass as `workspace`.
 * The per-row scalars of the backward (delta and -LSE log2 e) are kept in an
 * array of BA_STATIC_SCRATCH_BYTES that is part of the library image; every GPU
 * that loads the library holds that much memory until the process exits.
 *   - Arguments are those of branch_attn_bwd without workspace / ws_bytes; the
 *     caller still owns all inputs and outputs.
 *   - The size limit is checked first: a problem beyond it gets BA_EWORKSPACE
 *     even for a call whose ranges are empty (where branch_attn_bwd returns BA_OK).
 *   - Limit: ba_workspace_bytes(plan, BA_OP_BWD) must not exceed
 *     BA_STATIC_SCRATCH_BYTES (8 MiB: 2 * h_q * (N + M + 128, rounded up to 64)
 *     floats, e.g. 32 query heads and up to 32,640 rows); larger problems get
 *     BA_EWORKSPACE and nothing is launched.
 *   - The first call on each device looks up the array's device address (with
 *     that device current); make that first call outside any stream capture.
 *     No call allocates or frees device memory.
 *   - All calls on a device share the one array, which keeps whatever the last
 *     call left in it.  Nothing in it needs clearing (each call rewrites every
 *     entry it reads), but two calls whose kernels overlap in time on the GPU --
 *     different streams, or different host threads -- race on it: serialise them.
 */
#define BA_STATIC_SCRATCH_BYTES (8u << 20)
int branch_attn_bwd_static(const ba_plan_t *plan, const void *q_main, const void *q_branch,
                           const void *k, const void *v, const void *O, const float *LSE,
                           const void *dO,
                           int64_t qm_begin, int64_t qm_end, int64_t br_begin, int64_t br_end,
                           int64_t kv_begin, int64_t kv_end, int parts, int accumulate,
                           void *dQ_main, void *dQ_branch, void *dK, void *dV, void *stream);

/*
 * One ring step on a RECEIVED K/V shard (Section 3.2, "Communication cost and
 * overlap": K/V shards circulate between the context-parallel ranks while the
 * queries stay local; Eq. (cp-comm) counts the shard bytes).  The same partial
 * forward / backward as above for the causal-prefix keys only (BA_PART_MAIN), but
 * the keys come from a buffer that holds just the shard:
 *   k_shard, v_shard  [kv_end - kv_begin, h_kv, D]: main key rows [kv_begin,
 *                     kv_end) as received (e.g. in a local double buffer); both
 *                     ends must be multiples of 128 (kv_end may also be N),
 *                     else BA_EINVAL.  Nothing outside the shard is read.
 *   forward:  merge = 0 writes the compact fp32 partial (O_acc, LSE_acc) as
 *             branch_attn_fwd_partial does, merge = 1 merges it into them as
 *             branch_attn_fwd_partial_merge does.
 *   backward: always accumulates.  dQ_main / dQ_branch are the local fp32
 *             accumulators (global layout); dK_shard, dV_shard
 *             [kv_end - kv_begin, h_kv, D] fp32 are the shard's gradient
 *             accumulators, which travel around the ring with the shard and
 *             return to its owner.  `stages` as in branch_attn_bwd_stages.
 * The branch-local keys never move: the owner handles them in its local step
 * with the calls above.
 */
int branch_attn_fwd_shard(const ba_plan_t *plan, const void *q_main, const void *q_branch,
                          const void *k_shard, const void *v_shard,
                          int64_t qm_begin, int64_t qm_end, int64_t br_begin, int64_t br_end,
                          int64_t kv_begin, int64_t kv_end, int merge,
                          float *O_acc, float *LSE_acc, void *stream);
int branch_attn_bwd_shard(const ba_plan_t *plan, const void *q_main, const void *q_branch,
                          const void *k_shard, const void *v_shard, const void *O, const float *LSE,
                          const void *dO,
                          int64_t qm_begin, int64_t qm_end, int64_t br_begin, int64_t br_end,
                          int64_t kv_begin, int64_t kv_end,
                          float *dQ_main, float *dQ_branch, float *dK_shard, float *dV_shard,
                          void *workspace, size_t ws_bytes, void *stream, int stages);

/*
 * Step-major (per-depth) calls for training-time-test drafts (Section 3.2, draft
 * families: the EAGLE-3 style draft feeds its own previous prediction back over
 * several steps, so the tokens of depth d exist only after depth d - 1 has been
 * computed; a trainer therefore needs one attention call per depth).
 *
 * Plan: BA_MASK_CHAIN with uniform_len = number of depths n, tensor-core kernels
 * (bf16, head_dim 128); otherwise BA_EUNSUPPORTED.  `depth` is 1 .. n.
 * Layout (depth-major, unlike the all-depths calls above):
 *   q_depth, O_depth, dO_depth, dQ_depth  [A, h_q, D]   row b = the depth-`depth`
 *                                         token of branch b;  LSE_depth [A, h_q]
 *   k, v     [N + n * A, h_kv, D]  main rows, then the branch tokens of depth 1
 *            (A rows, branch order), of depth 2, ...  Only the rows of depths
 *            <= depth are read: later rows need not be written yet.
 *   dK, dV   fp32, same layout as k, v; the terms of this call are ADDED (zero
 *            them before the first call of a backward pass, convert with
 *            ba_finalize_grads after the last).
 * Query b sees the main keys of its causal prefix (up to and including its
 * anchor) and the tokens of depths 1 .. depth of its own branch.  Branches
 * [br_begin, br_end) are computed; other rows of the outputs are left alone.
 * Running depth = 1 .. n over all branches gives the rows of branch_attn_fwd;
 * the backward calls together (plus the main rows' own backward) give its
 * gradients.  dQ_depth is summed with fp32 atomic adds and converted (as in
 * BA_STAGE_FUSED).  workspace: ba_workspace_bytes(plan, BA_OP_BWD_DEPTH).
 */
int branch_attn_fwd_depth(const ba_plan_t *plan, int depth, const void *q_depth, const void *k,
                          const void *v, int64_t br_begin, int64_t br_end, void *O_depth,
                          float *LSE_depth, void *stream);
int branch_attn_bwd_depth(const ba_plan_t *plan, int depth, const void *q_depth, const void *k,
                          const void *v, const void *O_depth, const float *LSE_depth,
                          const void *dO_depth, int64_t br_begin, int64_t br_end, void *dQ_depth,
                          float *dK, float *dV, void *workspace, size_t ws_bytes, void *stream);

/* fp32 accumulators -> dst_dtype (round to nearest even), `count` elements. */
int ba_finalize_grads(const float *src, void *dst, int64_t count, int dst_dtype, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* BRANCH_ATTN_H_ */
