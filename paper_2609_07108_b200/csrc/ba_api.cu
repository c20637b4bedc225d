// C-ABI entry points: argument checks and dispatch to the plain-FMA or the
// tensor-core kernels.  No device memory is allocated here; every call only
// enqueues kernels on the caller's stream.
#include "ba_common.cuh"

namespace {

inline size_t align256(size_t x) { return (x + 255) / 256 * 256; }

// Branch index range -> branch token range.
int token_range(const ba_plan *pl, int64_t br_begin, int64_t br_end, int64_t *t0, int64_t *t1) {
    const int64_t a = pl->prob.num_branches;
    if (br_begin < 0 || br_end < br_begin || br_end > a) return BA_EINVAL;
    if (pl->prob.uniform_len > 0) {
        *t0 = br_begin * pl->prob.uniform_len;
        *t1 = br_end * pl->prob.uniform_len;
    } else if (a > 0) {
        *t0 = pl->host_offsets[br_begin];
        *t1 = pl->host_offsets[br_end];
    } else {
        *t0 = *t1 = 0;
    }
    return BA_OK;
}

int make_range(const ba_plan *pl, int64_t qm_begin, int64_t qm_end, int64_t br_begin, int64_t br_end,
               int64_t kv_begin, int64_t kv_end, int parts, BaRange *r) {
    const int64_t n = pl->prob.n_main;
    if (qm_begin < 0 || qm_end < qm_begin || qm_end > n) return BA_EINVAL;
    if (kv_begin < 0 || kv_end < kv_begin || kv_end > n) return BA_EINVAL;
    if (parts < 0 || parts > (BA_PART_MAIN | BA_PART_BRANCH)) return BA_EINVAL;
    r->qm_begin = qm_begin; r->qm_end = qm_end;
    r->kv_begin = kv_begin; r->kv_end = kv_end;
    r->parts = parts;
    return token_range(pl, br_begin, br_end, &r->tok_begin, &r->tok_end);
}

}  // namespace

extern "C" size_t ba_workspace_bytes(const ba_plan_t *plan, int op) {
    if (!plan) return 0;
    // delta and -LSE*log2(e), fp32, head-major [h_q, row_pitch] each
    const size_t scalars = align256((size_t)2 * plan->row_pitch * plan->prob.h_q * sizeof(float));
    if (op == BA_OP_BWD) return scalars;
    if (op == BA_OP_BWD_DEPTH)  // plus an fp32 dQ accumulator with one row per branch
        return scalars + align256((size_t)plan->prob.num_branches * plan->prob.h_q * plan->prob.head_dim *
                                  sizeof(float));
    if (op == BA_OP_BWD_FUSED)  // plus the fp32 dQ accumulator of the one-kernel backward
        return scalars + align256((size_t)(plan->prob.n_main + plan->prob.n_branch) * plan->prob.h_q *
                                  plan->prob.head_dim * sizeof(float));
    return 0;
}

static int fwd_common(const ba_plan_t *plan, const BaRange &r, const void *q_main, const void *q_branch,
                      const void *k, const void *v, void *o, float *lse, int partial, void *stream) {
    const bool has_main_q = q_main != nullptr && r.qm_end > r.qm_begin;
    const bool has_branch_q = r.tok_end > r.tok_begin;
    if (!has_main_q && !has_branch_q) return BA_OK;
    if (!k || !v || !o || !lse) return BA_EINVAL;
    if (has_branch_q && !q_branch) return BA_EINVAL;
    cudaStream_t st = (cudaStream_t)stream;
    if (plan->impl == BA_IMPL_TC) return ba_tc_fwd(plan, r, q_main, q_branch, k, v, o, lse, partial, st);
    if (partial == 2) return BA_EUNSUPPORTED;   // merge in the epilogue: tensor-core kernel only
    return ba_simt_fwd(plan, r, q_main, q_branch, k, v, o, lse, partial != 0, st);
}

extern "C" int branch_attn_fwd(const ba_plan_t *plan, const void *q_main, const void *q_branch,
                               const void *k, const void *v, void *O, float *LSE, void *workspace,
                               size_t ws_bytes, void *stream) {
    (void)workspace; (void)ws_bytes;
    if (!plan) return BA_EINVAL;
    BaRange r;
    int rc = make_range(plan, 0, plan->prob.n_main, 0, plan->prob.num_branches, 0, plan->prob.n_main,
                        BA_PART_MAIN | BA_PART_BRANCH, &r);
    if (rc != BA_OK) return rc;
    return fwd_common(plan, r, q_main, q_branch, k, v, O, LSE, 0, stream);
}

extern "C" int branch_attn_fwd_partial(const ba_plan_t *plan, const void *q_main, const void *q_branch,
                                       const void *k, const void *v, int64_t qm_begin, int64_t qm_end,
                                       int64_t br_begin, int64_t br_end, int64_t kv_begin,
                                       int64_t kv_end, int parts, float *O_part, float *LSE_part,
                                       void *workspace, size_t ws_bytes, void *stream) {
    (void)workspace; (void)ws_bytes;
    if (!plan) return BA_EINVAL;
    BaRange r;
    int rc = make_range(plan, qm_begin, qm_end, br_begin, br_end, kv_begin, kv_end, parts, &r);
    if (rc != BA_OK) return rc;
    if (!q_main && qm_end > qm_begin) return BA_EINVAL;
    return fwd_common(plan, r, q_main, q_branch, k, v, O_part, LSE_part, 1, stream);
}

extern "C" int branch_attn_fwd_partial_merge(const ba_plan_t *plan, const void *q_main, const void *q_branch,
                                             const void *k, const void *v, int64_t qm_begin, int64_t qm_end,
                                             int64_t br_begin, int64_t br_end, int64_t kv_begin,
                                             int64_t kv_end, int parts, float *O_acc, float *LSE_acc,
                                             void *workspace, size_t ws_bytes, void *stream) {
    (void)workspace; (void)ws_bytes;
    if (!plan) return BA_EINVAL;
    BaRange r;
    int rc = make_range(plan, qm_begin, qm_end, br_begin, br_end, kv_begin, kv_end, parts, &r);
    if (rc != BA_OK) return rc;
    if (!q_main && qm_end > qm_begin) return BA_EINVAL;
    return fwd_common(plan, r, q_main, q_branch, k, v, O_acc, LSE_acc, 2, stream);
}

extern "C" int branch_attn_bwd(const ba_plan_t *plan, const void *q_main, const void *q_branch,
                               const void *k, const void *v, const void *O, const float *LSE,
                               const void *dO, int64_t qm_begin, int64_t qm_end, int64_t br_begin,
                               int64_t br_end, int64_t kv_begin, int64_t kv_end, int parts,
                               int accumulate, void *dQ_main, void *dQ_branch, void *dK, void *dV,
                               void *workspace, size_t ws_bytes, void *stream) {
    return branch_attn_bwd_stages(plan, q_main, q_branch, k, v, O, LSE, dO, qm_begin, qm_end, br_begin, br_end,
                                  kv_begin, kv_end, parts, accumulate, dQ_main, dQ_branch, dK, dV, workspace,
                                  ws_bytes, stream, BA_STAGE_ALL);
}

extern "C" int branch_attn_bwd_stages(const ba_plan_t *plan, const void *q_main, const void *q_branch,
                                      const void *k, const void *v, const void *O, const float *LSE,
                                      const void *dO, int64_t qm_begin, int64_t qm_end, int64_t br_begin,
                                      int64_t br_end, int64_t kv_begin, int64_t kv_end, int parts,
                                      int accumulate, void *dQ_main, void *dQ_branch, void *dK, void *dV,
                                      void *workspace, size_t ws_bytes, void *stream, int stages) {
    if (!plan) return BA_EINVAL;
    if (stages <= 0 || stages > (BA_STAGE_ALL | BA_STAGE_FUSED)) return BA_EINVAL;
    if ((stages & BA_STAGE_FUSED) && (stages & (BA_STAGE_DQ | BA_STAGE_DKDV))) return BA_EINVAL;
    BaRange r;
    int rc = make_range(plan, qm_begin, qm_end, br_begin, br_end, kv_begin, kv_end, parts, &r);
    if (rc != BA_OK) return rc;
    if (!q_main) r.qm_end = r.qm_begin;  // branch queries only
    const bool has_main_q = r.qm_end > r.qm_begin;
    const bool has_branch_q = r.tok_end > r.tok_begin;
    if (!has_main_q && !has_branch_q) return BA_OK;
    if (!k || !v || !O || !LSE || !dO || !dK || !dV) return BA_EINVAL;
    if (has_main_q && !dQ_main) return BA_EINVAL;
    if (has_branch_q && (!q_branch || !dQ_branch)) return BA_EINVAL;
    if (accumulate != 0 && accumulate != 1) return BA_EINVAL;
    const bool fused_scratch = (stages & BA_STAGE_FUSED) && !accumulate;
    const size_t need = ba_workspace_bytes(plan, fused_scratch ? BA_OP_BWD_FUSED : BA_OP_BWD);
    if (!workspace || ws_bytes < need || ((uintptr_t)workspace & 255)) return BA_EWORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    float *delta = (float *)workspace;
    float *nlse2 = delta + (size_t)plan->row_pitch * plan->prob.h_q;
    const int64_t rp = plan->row_pitch;
    const int64_t n = plan->prob.n_main;
    const int hq = plan->prob.h_q, d = plan->prob.head_dim, dt = plan->prob.dtype;
    if (stages & BA_STAGE_PREP) {   // main rows and branch rows of the call in one launch
        const int64_t ma = has_main_q ? r.qm_begin : 0, mb = has_main_q ? r.qm_end : 0;
        const int64_t ba_ = has_branch_q ? n + r.tok_begin : 0, bb = has_branch_q ? n + r.tok_end : 0;
        if ((rc = ba_delta(O, dO, LSE, delta, nlse2, rp, ma, mb, ba_, bb, hq, d, dt, st)) != BA_OK) return rc;
    }
    if (!(stages & (BA_STAGE_DQ | BA_STAGE_DKDV | BA_STAGE_FUSED))) return BA_OK;
    const void *qm = has_main_q ? q_main : nullptr;
    if (stages & BA_STAGE_FUSED) {
        if (plan->impl != BA_IMPL_TC) return BA_EUNSUPPORTED;
        if (accumulate)
            return ba_tc_bwd_fused(plan, r, qm, q_branch, k, v, delta, dO, 1, dQ_main, dQ_branch, dK, dV, st);
        // gradients in the input dtype: dQ of the selected rows is summed in the workspace, then converted
        const size_t row_elems = (size_t)hq * d;
        float *acc_main = (float *)((char *)workspace + ba_workspace_bytes(plan, BA_OP_BWD));
        float *acc_branch = acc_main + (size_t)n * row_elems;
        if (has_main_q)
            BA_CUDA_CHECK(cudaMemsetAsync(acc_main + (size_t)r.qm_begin * row_elems, 0,
                                          (size_t)(r.qm_end - r.qm_begin) * row_elems * sizeof(float), st));
        if (has_branch_q)
            BA_CUDA_CHECK(cudaMemsetAsync(acc_branch + (size_t)r.tok_begin * row_elems, 0,
                                          (size_t)(r.tok_end - r.tok_begin) * row_elems * sizeof(float), st));
        rc = ba_tc_bwd_fused(plan, r, qm, q_branch, k, v, delta, dO, 0, acc_main, acc_branch, dK, dV, st);
        if (rc != BA_OK) return rc;
        if (has_main_q &&
            (rc = ba_finalize_grads(acc_main + (size_t)r.qm_begin * row_elems,
                                    (__nv_bfloat16 *)dQ_main + (size_t)r.qm_begin * row_elems,
                                    (int64_t)((r.qm_end - r.qm_begin) * row_elems), dt, stream)) != BA_OK)
            return rc;
        if (has_branch_q &&
            (rc = ba_finalize_grads(acc_branch + (size_t)r.tok_begin * row_elems,
                                    (__nv_bfloat16 *)dQ_branch + (size_t)r.tok_begin * row_elems,
                                    (int64_t)((r.tok_end - r.tok_begin) * row_elems), dt, stream)) != BA_OK)
            return rc;
        return BA_OK;
    }
    if (plan->impl == BA_IMPL_TC)
        return ba_tc_bwd(plan, r, qm, q_branch, k, v, LSE, delta, dO, accumulate, dQ_main, dQ_branch, dK,
                         dV, st, stages);
    return ba_simt_bwd(plan, r, qm, q_branch, k, v, LSE, delta, dO, accumulate, dQ_main, dQ_branch, dK, dV,
                       st, stages);
}

// ---------------------------------------------------------------- step-major (per-depth) calls

static int depth_range(const ba_plan_t *plan, int depth, int64_t br_begin, int64_t br_end, BaRange *r) {
    if (!plan) return BA_EINVAL;
    const ba_problem_t &pr = plan->prob;
    if (plan->impl != BA_IMPL_TC || pr.mask_kind != BA_MASK_CHAIN || pr.uniform_len <= 0) return BA_EUNSUPPORTED;
    if (depth < 1 || depth > pr.uniform_len) return BA_EINVAL;
    if (br_begin < 0 || br_end < br_begin || br_end > pr.num_branches) return BA_EINVAL;
    r->qm_begin = r->qm_end = 0;
    r->tok_begin = br_begin; r->tok_end = br_end;   // branch indices: one query row per branch
    r->kv_begin = 0; r->kv_end = pr.n_main;
    r->parts = BA_PART_MAIN | BA_PART_BRANCH;
    return BA_OK;
}

extern "C" int branch_attn_fwd_depth(const ba_plan_t *plan, int depth, const void *q_depth, const void *k,
                                     const void *v, int64_t br_begin, int64_t br_end, void *O_depth,
                                     float *LSE_depth, void *stream) {
    BaRange r;
    int rc = depth_range(plan, depth, br_begin, br_end, &r);
    if (rc != BA_OK) return rc;
    if (br_end == br_begin) return BA_OK;
    if (!q_depth || !k || !v || !O_depth || !LSE_depth) return BA_EINVAL;
    return ba_tc_fwd(plan, r, nullptr, q_depth, k, v, O_depth, LSE_depth, 0, (cudaStream_t)stream, depth);
}

extern "C" int branch_attn_bwd_depth(const ba_plan_t *plan, int depth, const void *q_depth, const void *k,
                                     const void *v, const void *O_depth, const float *LSE_depth,
                                     const void *dO_depth, int64_t br_begin, int64_t br_end, void *dQ_depth,
                                     float *dK, float *dV, void *workspace, size_t ws_bytes, void *stream) {
    BaRange r;
    int rc = depth_range(plan, depth, br_begin, br_end, &r);
    if (rc != BA_OK) return rc;
    if (br_end == br_begin) return BA_OK;
    if (!q_depth || !k || !v || !O_depth || !LSE_depth || !dO_depth || !dQ_depth || !dK || !dV) return BA_EINVAL;
    if (!workspace || ws_bytes < ba_workspace_bytes(plan, BA_OP_BWD_DEPTH) || ((uintptr_t)workspace & 255))
        return BA_EWORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    const ba_problem_t &pr = plan->prob;
    float *delta = (float *)workspace;
    float *nlse2 = delta + (size_t)plan->row_pitch * pr.h_q;
    float *acc = (float *)((char *)workspace + ba_workspace_bytes(plan, BA_OP_BWD));
    const size_t row_elems = (size_t)pr.h_q * pr.head_dim;
    // per-row scalars of the selected branches' depth-`depth` rows (rows are indexed by branch here)
    if ((rc = ba_delta(O_depth, dO_depth, LSE_depth, delta, nlse2, plan->row_pitch, 0, 0, br_begin, br_end,
                       pr.h_q, pr.head_dim, pr.dtype, st)) != BA_OK)
        return rc;
    BA_CUDA_CHECK(cudaMemsetAsync(acc + (size_t)br_begin * row_elems, 0,
                                  (size_t)(br_end - br_begin) * row_elems * sizeof(float), st));
    rc = ba_tc_bwd_fused(plan, r, nullptr, q_depth, k, v, delta, dO_depth, 1, nullptr, acc, dK, dV, st, depth);
    if (rc != BA_OK) return rc;
    return ba_finalize_grads(acc + (size_t)br_begin * row_elems,
                             (__nv_bfloat16 *)dQ_depth + (size_t)br_begin * row_elems,
                             (int64_t)((br_end - br_begin) * row_elems), pr.dtype, stream);
}

// ---------------------------------------------------------------- ring steps on a received K/V shard

// The kernels address keys by their global row; a shard holds only rows [kv_begin, kv_end).
// Tiles of 128 keys start at multiples of 128, so with both ends on such a multiple every row a
// kernel touches lies inside the shard, and the shard can be addressed as if it were the full
// tensor by moving its base back by kv_begin rows (no byte before the shard is ever read).
static int shard_ok(const ba_plan_t *plan, int64_t kv_begin, int64_t kv_end) {
    if (!plan) return BA_EINVAL;
    if (kv_begin < 0 || kv_end < kv_begin || kv_end > plan->prob.n_main) return BA_EINVAL;
    if ((kv_begin % 128) != 0 || ((kv_end % 128) != 0 && kv_end != plan->prob.n_main)) return BA_EINVAL;
    return BA_OK;
}

static inline const void *rebase(const void *shard, int64_t rows_back, size_t row_bytes) {
    return shard ? (const void *)((const char *)shard - (size_t)rows_back * row_bytes) : nullptr;
}

extern "C" int branch_attn_fwd_shard(const ba_plan_t *plan, const void *q_main, const void *q_branch,
                                     const void *k_shard, const void *v_shard, int64_t qm_begin, int64_t qm_end,
                                     int64_t br_begin, int64_t br_end, int64_t kv_begin, int64_t kv_end,
                                     int merge, float *O_acc, float *LSE_acc, void *stream) {
    int rc = shard_ok(plan, kv_begin, kv_end);
    if (rc != BA_OK) return rc;
    if (merge != 0 && merge != 1) return BA_EINVAL;
    if (kv_end > kv_begin && (!k_shard || !v_shard)) return BA_EINVAL;
    const size_t esz = plan->prob.dtype == BA_FP32 ? 4 : 2;
    const size_t row_bytes = (size_t)plan->prob.h_kv * plan->prob.head_dim * esz;
    const void *k = rebase(k_shard, kv_begin, row_bytes), *v = rebase(v_shard, kv_begin, row_bytes);
    if (merge)
        return branch_attn_fwd_partial_merge(plan, q_main, q_branch, k, v, qm_begin, qm_end, br_begin, br_end,
                                             kv_begin, kv_end, BA_PART_MAIN, O_acc, LSE_acc, nullptr, 0, stream);
    return branch_attn_fwd_partial(plan, q_main, q_branch, k, v, qm_begin, qm_end, br_begin, br_end, kv_begin,
                                   kv_end, BA_PART_MAIN, O_acc, LSE_acc, nullptr, 0, stream);
}

extern "C" int branch_attn_bwd_shard(const ba_plan_t *plan, const void *q_main, const void *q_branch,
                                     const void *k_shard, const void *v_shard, const void *O, const float *LSE,
                                     const void *dO, int64_t qm_begin, int64_t qm_end, int64_t br_begin,
                                     int64_t br_end, int64_t kv_begin, int64_t kv_end, float *dQ_main,
                                     float *dQ_branch, float *dK_shard, float *dV_shard, void *workspace,
                                     size_t ws_bytes, void *stream, int stages) {
    int rc = shard_ok(plan, kv_begin, kv_end);
    if (rc != BA_OK) return rc;
    if (kv_end > kv_begin && (!k_shard || !v_shard || !dK_shard || !dV_shard)) return BA_EINVAL;
    const size_t esz = plan->prob.dtype == BA_FP32 ? 4 : 2;
    const size_t row_elems = (size_t)plan->prob.h_kv * plan->prob.head_dim;
    const void *k = rebase(k_shard, kv_begin, row_elems * esz), *v = rebase(v_shard, kv_begin, row_elems * esz);
    void *dk = (void *)rebase(dK_shard, kv_begin, row_elems * sizeof(float));
    void *dv = (void *)rebase(dV_shard, kv_begin, row_elems * sizeof(float));
    return branch_attn_bwd_stages(plan, q_main, q_branch, k, v, O, LSE, dO, qm_begin, qm_end, br_begin, br_end,
                                  kv_begin, kv_end, BA_PART_MAIN, 1, dQ_main, dQ_branch, dk, dv, workspace,
                                  ws_bytes, stream, stages);
}
