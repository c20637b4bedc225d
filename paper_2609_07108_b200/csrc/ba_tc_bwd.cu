// Tensor-core backward (sm_100a, bf16, head_dim 128): dQ kernel and dK/dV kernel.
//
// Gradients of the attention of paper Section 3.2, accumulated over key chunks
// ("replays the same K/V ring and accumulates gradients locally").  With the
// final log-sum-exp l and delta = <dO, O> of each row:
//   P = exp(scale * Q K^T - l),  dP = dO V^T,  dS = P o (dP - delta),
//   dQ = scale * dS K,  dK = scale * dS^T Q,  dV = P^T dO.
// Every output element has exactly one owning CTA, so sums are deterministic.
//
// dQ kernel (query-stationary, same work split as the forward): per 128-key
// tile S -> TMEM, softmax warps turn it into P (kept in registers as bf16),
// the same TMEM columns then receive dP, the warps form dS (bf16, written over
// those columns) and the tensor core adds dS K into the dQ accumulator.
//   TMEM: R_0 [0,128) R_1 [128,256) (S, then dP, then dS)  dQ_0 [256,384) dQ_1 [384,512)
#include <limits.h>
#include <string.h>

#include "ba_common.cuh"
#include "ba_sm100.cuh"

using namespace sm100;

namespace {

constexpr int kTile = 128;
constexpr uint32_t kTileBytes = 32768;
constexpr float kLog2e = 1.4426950408889634f;

__device__ __forceinline__ uint64_t bit_range(int lo, int hi) {
    lo = max(lo, 0);
    hi = min(hi, 63);
    if (lo > hi) return 0ull;
    return (~0ull >> (63 - hi)) & (~0ull << lo);
}

// ============================================================================
// dQ
// ============================================================================
constexpr int kDqThreads = 320;

struct DqSmem {
    alignas(1024) uint8_t q[2][kTileBytes];
    alignas(1024) uint8_t go[2][kTileBytes];
    alignas(1024) uint8_t kbuf[2][kTileBytes];
    alignas(1024) uint8_t vbuf[kTileBytes];
    alignas(8) uint64_t q_full;
    uint64_t k_full[2], k_empty[2], v_full, v_empty;
    uint64_t s_full[2], a_done[2], dp_full[2], b_done[2], dq_full[2];
    uint32_t tmem_base;
    int abort_flag;
    int lo_min, hi_max, lo_max, hi_min, bs_min, be_max;
};

struct TcBwdParams {
    BaMeta meta;
    BaRange r;
    const float *lse, *delta;
    void *dq_main, *dq_branch, *dk, *dv;
    int h_q, h_kv, group, pairs_per_group;
    float scale, scale_log2;
    int accumulate;
    int has_main_q;
    int main_tiles, total_tiles;      // dQ kernel: query row tiles
    int main_key_tiles, total_key_tiles;  // dK/dV kernel: key tiles
    int *status;
};

template <bool ACC_F32>
__device__ __forceinline__ void store_grad_chunk(void *dst, size_t elem_off, const uint32_t (&r)[32], float mul) {
    if (ACC_F32) {
        float4 *d4 = reinterpret_cast<float4 *>((float *)dst + elem_off);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            float4 old = d4[i];
            old.x += __uint_as_float(r[4 * i]) * mul;
            old.y += __uint_as_float(r[4 * i + 1]) * mul;
            old.z += __uint_as_float(r[4 * i + 2]) * mul;
            old.w += __uint_as_float(r[4 * i + 3]) * mul;
            d4[i] = old;
        }
    } else {
        uint4 *d4 = reinterpret_cast<uint4 *>((__nv_bfloat16 *)dst + elem_off);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            uint4 v;
            v.x = pack_bf16(__uint_as_float(r[8 * i]) * mul, __uint_as_float(r[8 * i + 1]) * mul);
            v.y = pack_bf16(__uint_as_float(r[8 * i + 2]) * mul, __uint_as_float(r[8 * i + 3]) * mul);
            v.z = pack_bf16(__uint_as_float(r[8 * i + 4]) * mul, __uint_as_float(r[8 * i + 5]) * mul);
            v.w = pack_bf16(__uint_as_float(r[8 * i + 6]) * mul, __uint_as_float(r[8 * i + 7]) * mul);
            d4[i] = v;
        }
    }
}

__global__ void __launch_bounds__(kDqThreads, 1)
tc_dq_kernel(const __grid_constant__ CUtensorMap tm_q_main, const __grid_constant__ CUtensorMap tm_q_branch,
             const __grid_constant__ CUtensorMap tm_go, const __grid_constant__ CUtensorMap tm_k,
             const __grid_constant__ CUtensorMap tm_v, const TcBwdParams p) {
    extern __shared__ uint8_t smem_raw[];
    DqSmem &sm = *reinterpret_cast<DqSmem *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    volatile int *abort_flag = &sm.abort_flag;

    const int per_tile = p.h_kv * p.pairs_per_group;
    const int tile = p.total_tiles - 1 - (int)(blockIdx.x / per_tile);
    const int inner = (int)(blockIdx.x % per_tile);
    const int g = inner / p.pairs_per_group, hp = inner % p.pairs_per_group;
    const int h0 = g * p.group + 2 * hp;
    const bool second_head = 2 * hp + 1 < p.group;
    const int h1 = second_head ? h0 + 1 : h0;
    const bool is_main = tile < p.main_tiles;
    const int64_t n = p.meta.n_main;
    const int64_t row0 = is_main ? p.r.qm_begin + (int64_t)tile * kTile
                                 : p.r.tok_begin + (int64_t)(tile - p.main_tiles) * kTile;
    const int64_t row_end = is_main ? p.r.qm_end : p.r.tok_end;
    const int64_t grow0 = is_main ? row0 : n + row0;  // row in the [N + M] numbering (dO, LSE, delta)

    if (tid == 0) {
        mbar_init(&sm.q_full, 1);
        mbar_init(&sm.v_full, 1);
        mbar_init(&sm.v_empty, 1);
        for (int i = 0; i < 2; ++i) {
            mbar_init(&sm.k_full[i], 1);
            mbar_init(&sm.k_empty[i], 1);
            mbar_init(&sm.s_full[i], 1);
            mbar_init(&sm.a_done[i], 128);
            mbar_init(&sm.dp_full[i], 1);
            mbar_init(&sm.b_done[i], 128);
            mbar_init(&sm.dq_full[i], 1);
        }
        sm.abort_flag = 0;
        sm.lo_min = INT_MAX; sm.hi_max = -1; sm.lo_max = -1; sm.hi_min = INT_MAX;
        sm.bs_min = INT_MAX; sm.be_max = -1;
        fence_barrier_init();
    }
    if (warp == 8) {
        tmem_alloc(&sm.tmem_base, 512);
        tmem_relinquish();
    }
    __syncthreads();

    int lo = 1, hi = 0, bstart = 0;
    uint64_t bmask = 0;
    bool valid = false;
    int64_t my_row = 0;
    if (warp < 8) {
        my_row = row0 + (tid & 127);
        valid = my_row < row_end;
        if (valid) {
            const int64_t grow = is_main ? my_row : n + my_row;
            if (p.r.parts & BA_PART_MAIN) {
                lo = max(p.meta.row_lo[grow], (int)p.r.kv_begin);
                hi = min(p.meta.row_hi[grow], (int)p.r.kv_end - 1);
                if (hi < lo) { lo = 1; hi = 0; }
            }
            if (!is_main && (p.r.parts & BA_PART_BRANCH)) {
                bstart = p.meta.br_start[my_row];
                bmask = p.meta.br_mask[my_row];
            }
            if (warp < 4) {
                if (hi >= lo) {
                    atomicMin(&sm.lo_min, lo); atomicMax(&sm.hi_max, hi);
                    atomicMax(&sm.lo_max, lo); atomicMin(&sm.hi_min, hi);
                } else {
                    atomicMax(&sm.lo_max, INT_MAX); atomicMin(&sm.hi_min, -1);
                }
                if (!is_main && (p.r.parts & BA_PART_BRANCH)) {
                    atomicMin(&sm.bs_min, bstart);
                    atomicMax(&sm.be_max, p.meta.br_end[my_row]);
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = sm.tmem_base;

    int kt0 = 0, n_main_tiles = 0, n_br = 0;
    if (sm.hi_max >= sm.lo_min) {
        kt0 = sm.lo_min / kTile;
        n_main_tiles = sm.hi_max / kTile - kt0 + 1;
    }
    const int bs = sm.bs_min;
    if (sm.be_max > bs) n_br = (sm.be_max - bs + kTile - 1) / kTile;
    const int T = n_main_tiles + n_br;
    const int full_lo = sm.lo_max, full_hi = sm.hi_min;

    if (warp == 9) {
        // ================================================= TMA producer
        if (lane == 0 && T > 0) {
            const CUtensorMap *tq = is_main ? &tm_q_main : &tm_q_branch;
            mbar_expect_tx(&sm.q_full, 4 * kTileBytes);
            for (int half = 0; half < 2; ++half) {
                tma_load_3d(sm.q[0] + half * 16384, tq, half * 64, h0, (int)row0, &sm.q_full);
                tma_load_3d(sm.q[1] + half * 16384, tq, half * 64, h1, (int)row0, &sm.q_full);
                tma_load_3d(sm.go[0] + half * 16384, &tm_go, half * 64, h0, (int)grow0, &sm.q_full);
                tma_load_3d(sm.go[1] + half * 16384, &tm_go, half * 64, h1, (int)grow0, &sm.q_full);
            }
            bool ok = true;
            int k_issued = 0, v_issued = 0;
            for (int j = 0; j < T && ok; ++j) {
                const int krow = j < n_main_tiles ? (kt0 + j) * kTile : (int)n + bs + (j - n_main_tiles) * kTile;
                const int kb = j & 1;
                if (j >= 2) ok = mbar_wait(&sm.k_empty[kb], ((j >> 1) - 1) & 1, abort_flag);
                if (!ok) break;
                mbar_expect_tx(&sm.k_full[kb], kTileBytes);
                tma_load_3d(sm.kbuf[kb], &tm_k, 0, g, krow, &sm.k_full[kb]);
                tma_load_3d(sm.kbuf[kb] + 16384, &tm_k, 64, g, krow, &sm.k_full[kb]);
                k_issued = j + 1;
                if (j >= 1) ok = mbar_wait(&sm.v_empty, (j - 1) & 1, abort_flag);
                if (!ok) break;
                mbar_expect_tx(&sm.v_full, kTileBytes);
                tma_load_3d(sm.vbuf, &tm_v, 0, g, krow, &sm.v_full);
                tma_load_3d(sm.vbuf + 16384, &tm_v, 64, g, krow, &sm.v_full);
                v_issued = j + 1;
            }
            if (!ok) {
                for (int j = max(k_issued - 2, 0); j < k_issued; ++j) {
                    uint32_t spins = 0;
                    while (!mbar_try_wait(&sm.k_full[j & 1], (j >> 1) & 1) && ++spins < (1u << 22)) {}
                }
                if (v_issued > 0) {
                    uint32_t spins = 0;
                    while (!mbar_try_wait(&sm.v_full, (v_issued - 1) & 1) && ++spins < (1u << 22)) {}
                }
            }
        }
    } else if (warp == 8) {
        // ================================================= MMA issuer
        if (lane == 0 && T > 0) {
            constexpr uint32_t IDESC_KMAJ = idesc_bf16(128, 128, 0);  // S = Q K^T, dP = dO V^T
            constexpr uint32_t IDESC_MN = idesc_bf16(128, 128, 1);    // dQ += dS K
            const uint32_t q_addr[2] = {smem_u32(sm.q[0]), smem_u32(sm.q[1])};
            const uint32_t go_addr[2] = {smem_u32(sm.go[0]), smem_u32(sm.go[1])};
            auto issue_kmajor = [&](uint32_t d_tmem, uint32_t a_addr, uint32_t b_addr) {
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    const uint32_t off = (ks >> 2) * 16384 + (ks & 3) * 32;
                    mma_ss(d_tmem, smem_desc_sw128(a_addr + off, 16, 1024), smem_desc_sw128(b_addr + off, 16, 1024),
                           IDESC_KMAJ, ks > 0);
                }
            };
            auto issue_dq = [&](int i, uint32_t k_addr, bool accumulate) {
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)
                    mma_ts(tmem + 256 + i * 128, tmem + i * 128 + ks * 8,
                           smem_desc_sw128(k_addr + ks * 2048, 16384, 1024), IDESC_MN, accumulate || ks > 0);
            };
            bool ok = mbar_wait(&sm.q_full, 0, abort_flag);
            ok = ok && mbar_wait(&sm.k_full[0], 0, abort_flag);
            if (ok) {
                tc_fence_after();
                issue_kmajor(tmem + 0, q_addr[0], smem_u32(sm.kbuf[0])); tc_commit(&sm.s_full[0]);
                issue_kmajor(tmem + 128, q_addr[1], smem_u32(sm.kbuf[0])); tc_commit(&sm.s_full[1]);
            }
            for (int j = 0; j < T && ok; ++j) {
                const int kb = j & 1;
                const uint32_t k_addr = smem_u32(sm.kbuf[kb]);
                for (int i = 0; i < 2 && ok; ++i) {
                    ok = mbar_wait(&sm.a_done[i], j & 1, abort_flag);
                    if (ok && i == 0) ok = mbar_wait(&sm.v_full, j & 1, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    issue_kmajor(tmem + i * 128, go_addr[i], smem_u32(sm.vbuf));
                    tc_commit(&sm.dp_full[i]);
                    if (i == 1) tc_commit(&sm.v_empty);
                }
                for (int i = 0; i < 2 && ok; ++i) {
                    ok = mbar_wait(&sm.b_done[i], j & 1, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    issue_dq(i, k_addr, j > 0);
                    if (i == 1) tc_commit(&sm.k_empty[kb]);
                    if (j + 1 < T) {
                        if (i == 0) {
                            ok = mbar_wait(&sm.k_full[kb ^ 1], ((j + 1) >> 1) & 1, abort_flag);
                            if (!ok) break;
                            tc_fence_after();
                        }
                        issue_kmajor(tmem + i * 128, q_addr[i], smem_u32(sm.kbuf[kb ^ 1]));
                        tc_commit(&sm.s_full[i]);
                    } else {
                        tc_commit(&sm.dq_full[i]);
                    }
                }
            }
        }
    } else {
        // ================================================= P / dS warps + epilogue
        const int i = warp >> 2;
        const int h = i == 0 ? h0 : h1;
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t r_addr = tmem + lane_base + i * 128;
        const uint32_t dq_addr = tmem + lane_base + 256 + i * 128;
        const float sl2 = p.scale_log2;
        float neg_lse2 = -INFINITY, dlt = 0.f;  // dead rows: P = exp2(-inf) = 0
        if (valid) {
            const int64_t grow = is_main ? my_row : n + my_row;
            neg_lse2 = -p.lse[grow * p.h_q + h] * kLog2e;
            dlt = p.delta[grow * p.h_q + h];
        }
        bool ok = true;
        for (int j = 0; j < T; ++j) {
            bool masked;
            uint64_t vis[2] = {~0ull, ~0ull};
            if (j < n_main_tiles) {
                const int kj = (kt0 + j) * kTile;
                masked = !(kj >= full_lo && kj + kTile - 1 <= full_hi);
                if (masked) {
                    vis[0] = bit_range(lo - kj, hi - kj);
                    vis[1] = bit_range(lo - kj - 64, hi - kj - 64);
                }
            } else {
                masked = true;
                const int off = bs + (j - n_main_tiles) * kTile - bstart;
                const uint64_t mk = valid ? bmask : 0ull;
                if (off >= 0) {
                    vis[0] = off < 64 ? mk >> off : 0ull;
                    vis[1] = 0ull;
                } else {
                    const int sh = -off;
                    if (sh < 64) { vis[0] = mk << sh; vis[1] = mk >> (64 - sh); }
                    else if (sh < 128) { vis[0] = 0ull; vis[1] = mk << (sh - 64); }
                    else { vis[0] = 0ull; vis[1] = 0ull; }
                }
            }
            // --- phase A: P = exp2(scale_log2 * S - lse2), kept as bf16 pairs
            ok = mbar_wait(&sm.s_full[i], j & 1, abort_flag);
            if (!ok) break;
            tc_fence_after();
            uint32_t pr[64];
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint32_t r[32];
                tmem_ld32(r_addr + c * 32, r);
                tmem_wait_ld();
                const uint32_t mk = masked ? (uint32_t)(vis[c >> 1] >> ((c & 1) * 32)) : 0xffffffffu;
#pragma unroll
                for (int e = 0; e < 32; e += 2) {
                    float p0 = exp2f(fmaf(__uint_as_float(r[e]), sl2, neg_lse2));
                    float p1 = exp2f(fmaf(__uint_as_float(r[e + 1]), sl2, neg_lse2));
                    if (masked) {
                        p0 = ((mk >> e) & 1u) ? p0 : 0.f;
                        p1 = ((mk >> (e + 1)) & 1u) ? p1 : 0.f;
                    }
                    pr[c * 16 + (e >> 1)] = pack_bf16(p0, p1);
                }
            }
            tc_fence_before();
            mbar_arrive(&sm.a_done[i]);
            // --- phase B: dS = P o (dP - delta), bf16, over the first 64 columns
            ok = mbar_wait(&sm.dp_full[i], j & 1, abort_flag);
            if (!ok) break;
            tc_fence_after();
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint32_t r[32], pk[16];
                tmem_ld32(r_addr + c * 32, r);
                tmem_wait_ld();
#pragma unroll
                for (int e = 0; e < 32; e += 2) {
                    const uint32_t pp = pr[c * 16 + (e >> 1)];
                    const float p0 = __uint_as_float(pp << 16), p1 = __uint_as_float(pp & 0xffff0000u);
                    pk[e >> 1] = pack_bf16(p0 * (__uint_as_float(r[e]) - dlt), p1 * (__uint_as_float(r[e + 1]) - dlt));
                }
                tmem_st16(r_addr + c * 16, pk);
            }
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(&sm.b_done[i]);
        }
        // --- epilogue: dQ = scale * accumulator
        if (ok && T > 0) ok = mbar_wait(&sm.dq_full[i], 0, abort_flag);
        tc_fence_after();
        const bool do_store = ok && valid && (i == 0 || second_head);
        void *dst = is_main ? p.dq_main : p.dq_branch;
        const size_t base = ((size_t)my_row * p.h_q + h) * 128;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            uint32_t r[32];
            if (T > 0 && ok) {
                tmem_ld32(dq_addr + c * 32, r);
                tmem_wait_ld();
            } else {
#pragma unroll
                for (int e = 0; e < 32; ++e) r[e] = 0u;
            }
            if (do_store) {
                if (p.accumulate) store_grad_chunk<true>(dst, base + c * 32, r, p.scale);
                else store_grad_chunk<false>(dst, base + c * 32, r, p.scale);
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 8) tmem_dealloc(tmem, 512);
    if (tid == 0 && sm.abort_flag) atomicExch(p.status, BA_ETIMEOUT);
}

}  // namespace

int ba_tc_bwd(const ba_plan *pl, const BaRange &r, const void *q_main, const void *q_branch, const void *k,
              const void *v, const float *lse, const float *delta, const void *d_o, int accumulate,
              void *dq_main, void *dq_branch, void *dk, void *dv, cudaStream_t st) {
    static bool attr_set = false;
    const size_t dq_smem = sizeof(DqSmem) + 1024;
    if (!attr_set) {
        BA_CUDA_CHECK(cudaFuncSetAttribute(tc_dq_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dq_smem));
        attr_set = true;
    }
    const ba_problem_t &pr = pl->prob;
    TcBwdParams p;
    memset(&p, 0, sizeof p);
    p.meta = pl->meta;
    p.r = r;
    p.lse = lse;
    p.delta = delta;
    p.dq_main = dq_main; p.dq_branch = dq_branch; p.dk = dk; p.dv = dv;
    p.h_q = pr.h_q; p.h_kv = pr.h_kv;
    p.group = pr.h_q / pr.h_kv;
    p.pairs_per_group = (p.group + 1) / 2;
    p.scale = pl->scale;
    p.scale_log2 = pl->scale * kLog2e;
    p.accumulate = accumulate;
    p.has_main_q = q_main != nullptr;
    p.status = pl->dev_status;
    const int64_t mt = q_main ? (r.qm_end - r.qm_begin + kTile - 1) / kTile : 0;
    const int64_t bt = (r.tok_end - r.tok_begin + kTile - 1) / kTile;
    p.main_tiles = (int)mt;
    p.total_tiles = (int)(mt + bt);

    CUtensorMap tq_main, tq_branch, tgo, tk, tv;
    const uint64_t all_rows = (uint64_t)(pr.n_main + pr.n_branch);
    if (!make_tmap_rhd(&tk, k, all_rows, pr.h_kv, 128, kTile) || !make_tmap_rhd(&tv, v, all_rows, pr.h_kv, 128, kTile) ||
        !make_tmap_rhd(&tgo, d_o, all_rows, pr.h_q, 128, kTile))
        return BA_EINVAL;
    const void *qm = q_main ? q_main : q_branch;
    const void *qb = (q_branch && pr.n_branch > 0) ? q_branch : q_main;
    const uint64_t qm_rows = q_main ? (uint64_t)pr.n_main : (uint64_t)pr.n_branch;
    const uint64_t qb_rows = (q_branch && pr.n_branch > 0) ? (uint64_t)pr.n_branch : (uint64_t)pr.n_main;
    if (!make_tmap_rhd(&tq_main, qm, qm_rows, pr.h_q, 128, kTile) ||
        !make_tmap_rhd(&tq_branch, qb, qb_rows, pr.h_q, 128, kTile))
        return BA_EINVAL;

    if (p.total_tiles > 0) {
        const int64_t grid = (int64_t)p.total_tiles * pr.h_kv * p.pairs_per_group;
        if (grid > INT_MAX) return BA_EUNSUPPORTED;
        tc_dq_kernel<<<(unsigned)grid, kDqThreads, dq_smem, st>>>(tq_main, tq_branch, tgo, tk, tv, p);
        int rc = ba_check_launch();
        if (rc != BA_OK) return rc;
    }
    // dK / dV: plain-FMA kernel until the tensor-core one lands
    return ba_simt_bwd_dkdv(pl, r, q_main, q_branch, k, v, lse, delta, d_o, accumulate, dk, dv, st);
}
