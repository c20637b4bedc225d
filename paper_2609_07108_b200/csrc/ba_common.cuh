// Shared declarations of the branch-attention CUDA library (internal).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "branch_attn.h"

// Device-side view of the metadata a plan holds (all pointers into plan_mem).
// Rows are numbered "main rows [0, N) then branch tokens [N, N + M)".
struct BaMeta {
    int64_t n_main, n_branch;
    const int32_t *row_lo;        // [N+M] first visible main key (start of the row's sequence)
    const int32_t *row_hi;        // [N+M] last visible main key (own index, or the anchor)
    const int32_t *br_start;      // [M] first token of the token's own branch
    const int32_t *br_end;        // [M] one past the last token of the token's own branch
    const uint64_t *br_mask;      // [M] bit u set: the token sees token br_start + u
    const int32_t *key_qend;      // [N] one past the last main query row that sees key x
    const int32_t *key_bq_begin;  // [N] first branch token whose anchor is >= x
    const int32_t *key_bq_end;    // [N] first branch token anchored beyond x's sequence
};

struct ba_plan {
    ba_problem_t prob;            // copy; the metadata pointers in it are NOT kept alive
    BaMeta meta;
    float scale;
    int impl;                     // BA_IMPL_SIMT or BA_IMPL_TC (resolved)
    int64_t pairs;
    int64_t row_pitch;            // rows per head of the head-major backward scratch (>= N + M + 128)
    int32_t *host_offsets;        // host copy of branch_offsets (NULL when uniform_len > 0)
    int32_t *dev_status;          // one int32 in plan_mem: device-side status word
};

// Query / key selection of one call (monolithic = everything).
struct BaRange {
    int64_t qm_begin, qm_end;     // main query rows
    int64_t tok_begin, tok_end;   // branch tokens (query side and branch-key side)
    int64_t kv_begin, kv_end;     // main keys
    int parts;
};

extern thread_local int g_ba_last_cuda_error;

#define BA_CUDA_CHECK(expr)                                  \
    do {                                                     \
        cudaError_t e__ = (expr);                            \
        if (e__ != cudaSuccess) {                            \
            g_ba_last_cuda_error = (int)e__;                 \
            return BA_ECUDA;                                 \
        }                                                    \
    } while (0)

static inline int ba_check_launch() {
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
        g_ba_last_cuda_error = (int)e;
        return BA_ECUDA;
    }
    return BA_OK;
}

// --- kernels implemented in the other translation units -------------------
// Plain-FMA path (ba_simt.cu)
int ba_simt_fwd(const ba_plan *pl, const BaRange &r, const void *q_main, const void *q_branch,
                const void *k, const void *v, void *o, float *lse, bool partial_out,
                cudaStream_t st);
int ba_simt_bwd(const ba_plan *pl, const BaRange &r, const void *q_main, const void *q_branch,
                const void *k, const void *v, const float *lse, const float *delta,
                const void *d_o, int accumulate, void *dq_main, void *dq_branch, void *dk,
                void *dv, cudaStream_t st, int stages);
// Tensor-core path (ba_tc_fwd.cu / ba_tc_bwd.cu)
// partial_out: 0 = final layout in the input dtype, 1 = compact fp32, 2 = compact fp32 merged in place
// depth > 0: step-major call (queries = the depth-`depth` tokens of branches [r.tok_begin, r.tok_end),
// q_branch / o / lse indexed by branch, branch keys stored depth-major after the main rows)
int ba_tc_fwd(const ba_plan *pl, const BaRange &r, const void *q_main, const void *q_branch,
              const void *k, const void *v, void *o, float *lse, int partial_out,
              cudaStream_t st, int depth = 0);
int ba_tc_bwd(const ba_plan *pl, const BaRange &r, const void *q_main, const void *q_branch,
              const void *k, const void *v, const float *lse, const float *delta,
              const void *d_o, int accumulate, void *dq_main, void *dq_branch, void *dk,
              void *dv, cudaStream_t st, int stages);
// One-kernel backward (ba_tc_bwd_fused.cu): dq_* are fp32 accumulators (atomic adds) in either mode
int ba_tc_bwd_fused(const ba_plan *pl, const BaRange &r, const void *q_main, const void *q_branch,
                    const void *k, const void *v, const float *delta, const void *d_o,
                    int accumulate, void *dq_main, void *dq_branch, void *dk, void *dv,
                    cudaStream_t st, int depth = 0);
bool ba_tc_supported(const ba_problem_t *p);
// Elementwise (ba_elementwise.cu)
// Backward preprocess into head-major scratch [h_q, row_pitch]:
//   delta_t[h, r] = <dO[r, h], O[r, h]>,  nlse2_t[h, r] = -LSE[r, h] * log2(e)
// for two row segments [row_a_begin, row_a_end) and [row_b_begin, row_b_end) (either may be empty)
int ba_delta(const void *o, const void *d_o, const float *lse, float *delta_t, float *nlse2_t,
             int64_t row_pitch, int64_t row_a_begin, int64_t row_a_end, int64_t row_b_begin,
             int64_t row_b_end, int h_q, int d, int dtype, cudaStream_t st);
static inline int64_t ba_row_pitch(int64_t rows) { return (rows + 128 + 63) / 64 * 64; }
