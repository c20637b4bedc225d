// Metadata builder: varlen packing, anchors and branch masks -> per-row key
// bounds, per-token branch start / 64-bit visibility mask, per-key query ranges.
// (Paper Section 3.2: each branch query has two key sets -- the causal prefix of
// its packed main sequence up to its anchor, and its branch-local keys.)
//
// Every kernel here is safe on arbitrary (even invalid) metadata: searches are
// bounded, indices are clamped, the tree walk is capped at 64 steps.  Invalid
// metadata raises a flag that ba_plan_create reads before any data kernel can
// be launched with the plan.
#include <math.h>
#include <stdlib.h>
#include <string.h>

#include "ba_common.cuh"

thread_local int g_ba_last_cuda_error = 0;

namespace {

constexpr size_t kAlign = 256;
inline size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

struct PlanLayout {
    size_t row_lo, row_hi, br_start, br_end, br_mask, key_qend, key_bq_begin, key_bq_end, status,
        pairs, total;
};

PlanLayout plan_layout(int64_t n, int64_t m) {
    PlanLayout l;
    size_t off = 0;
    auto take = [&](size_t bytes) {
        size_t o = off;
        off += align_up(bytes ? bytes : 1);
        return o;
    };
    l.row_lo = take((size_t)(n + m) * 4);
    l.row_hi = take((size_t)(n + m) * 4);
    l.br_start = take((size_t)m * 4);
    l.br_end = take((size_t)m * 4);
    l.br_mask = take((size_t)m * 8);
    l.key_qend = take((size_t)n * 4);
    l.key_bq_begin = take((size_t)n * 4);
    l.key_bq_end = take((size_t)n * 4);
    l.status = take(4);
    l.pairs = take(8);
    l.total = off;
    return l;
}

struct PlanArgs {
    int64_t n, m;
    int32_t b, a, kind, uniform_len;
    const int32_t *cu, *anchor, *offs, *parent;
    int32_t *row_lo, *row_hi, *br_start, *br_end, *key_qend, *key_bq_begin, *key_bq_end;
    uint64_t *br_mask;
    int32_t *status;
    unsigned long long *pairs;
};

// Token offset of branch b.  With no branches (A = 0) there is no offsets array
// to read -- the caller may have passed NULL -- and every offset is 0.
__device__ __forceinline__ int32_t branch_offset(const PlanArgs &p, int32_t b) {
    if (p.uniform_len > 0) return b * p.uniform_len;
    if (p.a == 0 || p.offs == nullptr) return 0;
    return p.offs[b];
}

// Largest s in [0, B) with cu[s] <= i and cu[s+1] > i (the non-empty sequence
// holding i); clamped to [0, B-1] on bad input.
__device__ __forceinline__ int32_t seq_of(const PlanArgs &p, int32_t i) {
    int32_t lo = 0, hi = p.b;  // first s with cu[s+1] > i
    while (lo < hi) {
        int32_t mid = (lo + hi) >> 1;
        if (p.cu[mid + 1] > i) hi = mid; else lo = mid + 1;
    }
    return min(lo, max(p.b - 1, 0));
}

// First branch whose anchor is >= x.
__device__ __forceinline__ int32_t first_anchor_ge(const PlanArgs &p, int32_t x) {
    int32_t lo = 0, hi = p.a;
    while (lo < hi) {
        int32_t mid = (lo + hi) >> 1;
        if (p.anchor[mid] >= x) hi = mid; else lo = mid + 1;
    }
    return lo;
}

__global__ void plan_validate_kernel(PlanArgs p) {
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    const int64_t tid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    bool bad = false;
    if (tid == 0) {
        if (p.cu[0] != 0 || (int64_t)p.cu[p.b] != p.n) bad = true;
        if (branch_offset(p, 0) != 0 || (int64_t)branch_offset(p, p.a) != p.m) bad = true;
    }
    for (int64_t s = tid; s < p.b; s += stride)
        if (p.cu[s + 1] < p.cu[s]) bad = true;
    for (int64_t b = tid; b < p.a; b += stride) {
        const int32_t a = p.anchor[b];
        if (a < 0 || (int64_t)a >= p.n) bad = true;
        if (b > 0 && p.anchor[b - 1] > a) bad = true;
        const int32_t len = branch_offset(p, (int32_t)b + 1) - branch_offset(p, (int32_t)b);
        if (len < 0 || len > 64) bad = true;
    }
    if (bad) atomicExch(p.status, 1);
}

__global__ void plan_main_rows_kernel(PlanArgs p) {
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    unsigned long long local_pairs = 0;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < p.n; i += stride) {
        const int32_t s = seq_of(p, (int32_t)i);
        const int32_t lo = p.cu[s], end = p.cu[s + 1];
        p.row_lo[i] = lo;
        p.row_hi[i] = (int32_t)i;
        p.key_qend[i] = end;
        p.key_bq_begin[i] = branch_offset(p, first_anchor_ge(p, (int32_t)i));
        p.key_bq_end[i] = branch_offset(p, first_anchor_ge(p, end));
        local_pairs += (unsigned long long)max((int32_t)i - lo + 1, 0);
    }
    for (int o = 16; o; o >>= 1) local_pairs += __shfl_xor_sync(0xffffffffu, local_pairs, o);
    if ((threadIdx.x & 31) == 0 && local_pairs) atomicAdd(p.pairs, local_pairs);
}

__global__ void plan_branch_rows_kernel(PlanArgs p) {
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    unsigned long long local_pairs = 0;
    bool bad = false;
    for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < p.m; t += stride) {
        // branch holding token t
        int32_t b;
        if (p.uniform_len > 0) {
            b = (int32_t)(t / p.uniform_len);
        } else {
            int32_t lo = 0, hi = p.a;  // first b with offs[b+1] > t
            while (lo < hi) {
                int32_t mid = (lo + hi) >> 1;
                if (p.offs[mid + 1] > t) hi = mid; else lo = mid + 1;
            }
            b = min(lo, p.a - 1);
        }
        const int32_t start = branch_offset(p, b), end = branch_offset(p, b + 1);
        const int32_t i = (int32_t)t - start;
        const int32_t len = end - start;
        int32_t a = p.anchor[b];
        a = max(0, min(a, (int32_t)p.n - 1));
        const int32_t s = seq_of(p, a);
        uint64_t mask = 0;
        if (i < 0 || i >= 64 || len > 64) {
            bad = true;
        } else if (p.kind == BA_MASK_CHAIN) {
            mask = (i == 63) ? ~0ull : ((2ull << i) - 1ull);
        } else if (p.kind == BA_MASK_BLOCK) {
            mask = (len >= 64) ? ~0ull : ((1ull << len) - 1ull);
        } else {
            int32_t node = i;
            for (int step = 0; step < 64 && node >= 0; ++step) {
                mask |= 1ull << node;
                const int32_t par = p.parent[start + node];
                if (par >= node || par < -1) { bad = true; break; }
                node = par;
            }
        }
        p.row_lo[p.n + t] = p.cu[s];
        p.row_hi[p.n + t] = a;
        p.br_start[t] = start;
        p.br_end[t] = end;
        p.br_mask[t] = mask;
        local_pairs += (unsigned long long)max(a - p.cu[s] + 1, 0) + (unsigned long long)__popcll(mask);
    }
    if (bad) atomicExch(p.status, 1);
    for (int o = 16; o; o >>= 1) local_pairs += __shfl_xor_sync(0xffffffffu, local_pairs, o);
    if ((threadIdx.x & 31) == 0 && local_pairs) atomicAdd(p.pairs, local_pairs);
}

int grid_for(int64_t n, int block) {
    int64_t g = (n + block - 1) / block;
    if (g < 1) g = 1;
    if (g > 148 * 16) g = 148 * 16;
    return (int)g;
}

}  // namespace

extern "C" const char *ba_status_string(int status) {
    switch (status) {
        case BA_OK: return "ok";
        case BA_EINVAL: return "invalid argument";
        case BA_EUNSUPPORTED: return "unsupported dtype, head_dim or branch length";
        case BA_EWORKSPACE: return "plan memory or workspace too small or misaligned";
        case BA_EMETA: return "metadata failed device-side validation";
        case BA_ECUDA: return "CUDA runtime error";
        case BA_ETIMEOUT: return "bounded device-side wait expired";
        default: return "unknown status";
    }
}

extern "C" int ba_last_cuda_error(void) { return g_ba_last_cuda_error; }

static int check_sizes(const ba_problem_t *p) {
    if (!p) return BA_EINVAL;
    if (p->n_main < 0 || p->n_branch < 0 || p->num_seqs < 0 || p->num_branches < 0) return BA_EINVAL;
    if (p->n_main + p->n_branch >= (int64_t)1 << 31) return BA_EUNSUPPORTED;
    if (p->h_q <= 0 || p->h_kv <= 0 || p->h_q % p->h_kv != 0) return BA_EINVAL;
    if (p->head_dim != 64 && p->head_dim != 128) return BA_EUNSUPPORTED;
    if (p->dtype != BA_BF16 && p->dtype != BA_FP32) return BA_EUNSUPPORTED;
    if (p->mask_kind < BA_MASK_CHAIN || p->mask_kind > BA_MASK_TREE) return BA_EINVAL;
    if (p->uniform_len < 0 || p->uniform_len > 64) return BA_EUNSUPPORTED;
    if (p->impl < BA_IMPL_AUTO || p->impl > BA_IMPL_TC) return BA_EINVAL;
    if (p->n_main > 0 && p->num_seqs == 0) return BA_EINVAL;
    if (p->n_branch > 0 && (p->num_branches == 0 || p->n_main == 0)) return BA_EINVAL;
    if (p->uniform_len > 0 && (int64_t)p->uniform_len * p->num_branches != p->n_branch) return BA_EINVAL;
    if (!(p->softmax_scale >= 0.0f) || isinf(p->softmax_scale)) return BA_EINVAL;
    return BA_OK;
}

extern "C" size_t ba_plan_bytes(const ba_problem_t *p) {
    if (check_sizes(p) != BA_OK) return 0;
    return plan_layout(p->n_main, p->n_branch).total;
}

extern "C" int ba_plan_create(const ba_problem_t *p, void *plan_mem, size_t plan_bytes, void *stream,
                              ba_plan_t **out) {
    if (!out) return BA_EINVAL;
    *out = nullptr;
    int rc = check_sizes(p);
    if (rc != BA_OK) return rc;
    if (p->num_seqs > 0 && !p->cu_seqlens) return BA_EINVAL;
    if (p->num_branches > 0 && (!p->anchor_idx || (p->uniform_len == 0 && !p->branch_offsets))) return BA_EINVAL;
    if (p->mask_kind == BA_MASK_TREE && p->n_branch > 0 && !p->parent) return BA_EINVAL;
    if (p->impl == BA_IMPL_TC && !ba_tc_supported(p)) return BA_EUNSUPPORTED;
    const PlanLayout l = plan_layout(p->n_main, p->n_branch);
    if (!plan_mem || plan_bytes < l.total || ((uintptr_t)plan_mem & (kAlign - 1))) return BA_EWORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    char *base = (char *)plan_mem;

    PlanArgs a;
    a.n = p->n_main; a.m = p->n_branch; a.b = p->num_seqs; a.a = p->num_branches;
    a.kind = p->mask_kind; a.uniform_len = p->uniform_len;
    a.cu = p->cu_seqlens;
    // A = 0: the branch arrays are never read, whatever the caller passed for them
    a.anchor = p->num_branches > 0 ? p->anchor_idx : nullptr;
    a.offs = (p->num_branches > 0 && p->uniform_len == 0) ? p->branch_offsets : nullptr;
    a.parent = (p->mask_kind == BA_MASK_TREE && p->n_branch > 0) ? p->parent : nullptr;
    a.row_lo = (int32_t *)(base + l.row_lo); a.row_hi = (int32_t *)(base + l.row_hi);
    a.br_start = (int32_t *)(base + l.br_start); a.br_end = (int32_t *)(base + l.br_end);
    a.br_mask = (uint64_t *)(base + l.br_mask);
    a.key_qend = (int32_t *)(base + l.key_qend);
    a.key_bq_begin = (int32_t *)(base + l.key_bq_begin);
    a.key_bq_end = (int32_t *)(base + l.key_bq_end);
    a.status = (int32_t *)(base + l.status);
    a.pairs = (unsigned long long *)(base + l.pairs);

    BA_CUDA_CHECK(cudaMemsetAsync(a.status, 0, 4, st));
    BA_CUDA_CHECK(cudaMemsetAsync(a.pairs, 0, 8, st));
    int32_t status_host = 0;
    unsigned long long pairs_host = 0;
    if (p->num_seqs > 0) {
        const int64_t work = p->num_seqs > p->num_branches ? p->num_seqs : p->num_branches;
        plan_validate_kernel<<<grid_for(work, 256), 256, 0, st>>>(a);
        if ((rc = ba_check_launch()) != BA_OK) return rc;
        // stop here on bad top-level metadata: the row kernels index with it
        BA_CUDA_CHECK(cudaMemcpyAsync(&status_host, a.status, 4, cudaMemcpyDeviceToHost, st));
        BA_CUDA_CHECK(cudaStreamSynchronize(st));
        if (status_host != 0) return BA_EMETA;
        if (p->n_main > 0) {
            plan_main_rows_kernel<<<grid_for(p->n_main, 256), 256, 0, st>>>(a);
            if ((rc = ba_check_launch()) != BA_OK) return rc;
        }
        if (p->n_branch > 0) {
            plan_branch_rows_kernel<<<grid_for(p->n_branch, 256), 256, 0, st>>>(a);
            if ((rc = ba_check_launch()) != BA_OK) return rc;
        }
        BA_CUDA_CHECK(cudaMemcpyAsync(&status_host, a.status, 4, cudaMemcpyDeviceToHost, st));
        BA_CUDA_CHECK(cudaMemcpyAsync(&pairs_host, a.pairs, 8, cudaMemcpyDeviceToHost, st));
    }
    int32_t *host_offsets = nullptr;
    if (p->uniform_len == 0 && p->num_branches > 0) {
        host_offsets = (int32_t *)malloc(sizeof(int32_t) * ((size_t)p->num_branches + 1));
        if (!host_offsets) return BA_EINVAL;
        cudaError_t e = cudaMemcpyAsync(host_offsets, p->branch_offsets,
                                        sizeof(int32_t) * ((size_t)p->num_branches + 1),
                                        cudaMemcpyDeviceToHost, st);
        if (e != cudaSuccess) { free(host_offsets); g_ba_last_cuda_error = (int)e; return BA_ECUDA; }
    }
    {
        cudaError_t e = cudaStreamSynchronize(st);
        if (e != cudaSuccess) { free(host_offsets); g_ba_last_cuda_error = (int)e; return BA_ECUDA; }
    }
    if (status_host != 0) { free(host_offsets); return BA_EMETA; }

    ba_plan *pl = (ba_plan *)calloc(1, sizeof(ba_plan));
    if (!pl) { free(host_offsets); return BA_EINVAL; }
    pl->prob = *p;
    pl->prob.cu_seqlens = pl->prob.anchor_idx = pl->prob.branch_offsets = pl->prob.parent = nullptr;
    pl->meta.n_main = p->n_main; pl->meta.n_branch = p->n_branch;
    pl->meta.row_lo = a.row_lo; pl->meta.row_hi = a.row_hi;
    pl->meta.br_start = a.br_start; pl->meta.br_end = a.br_end; pl->meta.br_mask = a.br_mask;
    pl->meta.key_qend = a.key_qend; pl->meta.key_bq_begin = a.key_bq_begin;
    pl->meta.key_bq_end = a.key_bq_end;
    pl->scale = p->softmax_scale > 0.0f ? p->softmax_scale : 1.0f / sqrtf((float)p->head_dim);
    pl->impl = p->impl == BA_IMPL_AUTO ? (ba_tc_supported(p) ? BA_IMPL_TC : BA_IMPL_SIMT) : p->impl;
    pl->pairs = (int64_t)pairs_host;
    pl->row_pitch = ba_row_pitch(p->n_main + p->n_branch);
    pl->host_offsets = host_offsets;
    pl->dev_status = a.status;
    *out = pl;
    return BA_OK;
}

extern "C" int ba_plan_destroy(ba_plan_t *plan) {
    if (!plan) return BA_EINVAL;
    free(plan->host_offsets);
    free(plan);
    return BA_OK;
}

extern "C" int64_t ba_plan_pairs(const ba_plan_t *plan) { return plan ? plan->pairs : -1; }

extern "C" int ba_plan_impl(const ba_plan_t *plan) { return plan ? plan->impl : BA_EINVAL; }

extern "C" int ba_plan_check(ba_plan_t *plan, void *stream) {
    if (!plan) return BA_EINVAL;
    cudaStream_t st = (cudaStream_t)stream;
    int32_t status = 0;
    BA_CUDA_CHECK(cudaMemcpyAsync(&status, plan->dev_status, 4, cudaMemcpyDeviceToHost, st));
    BA_CUDA_CHECK(cudaMemsetAsync(plan->dev_status, 0, 4, st));
    BA_CUDA_CHECK(cudaStreamSynchronize(st));
    return status == 0 ? BA_OK : BA_ETIMEOUT;
}
