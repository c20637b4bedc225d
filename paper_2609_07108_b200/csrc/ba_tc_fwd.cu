// Tensor-core forward (sm_100a, bf16, head_dim 128).
//
// One CTA = 128 query rows x two query heads of one KV head (both heads see the
// same rows, hence the same key tiles and masks) -- or, when the group has an
// odd head left over, that head twice with the second copy discarded.  Both
// key sets of the paper's Section 3.2 (causal main prefix, own-branch keys) are
// walked as 128-key tiles in ONE online-softmax pass, which is Eq. (lse-merge)
// applied tile by tile; tiles no row can see are never visited, tiles every row
// sees entirely take a mask-free path.
//
// Warp roles (320 threads):
//   warps 0-3 / 4-7  softmax of query tile 0 / 1: one thread per row, scores read
//                    from TMEM, P written back to TMEM as bf16 over the scores
//   warp 8           issues tcgen05.mma: S_i = Q_i K^T, O_i += P_i V
//   warp 9           TMA producer: Q once, then K_j, V_j through a 4-stage ring
// The two query tiles ping-pong: while the softmax warps of tile 0 work on S_0,
// the tensor core runs tile 1's P V and next Q K^T, and vice versa.
// TMEM (512 columns): S_0 [0,128) S_1 [128,256) O_0 [256,384) O_1 [384,512);
// P_i occupies the first 64 columns of S_i.
#include <limits.h>
#include <string.h>

#include "ba_common.cuh"
#include "ba_sm100.cuh"

using namespace sm100;

namespace {

constexpr int kTile = 128;
constexpr int kStages = 4;
constexpr int kThreads = 320;
constexpr uint32_t kTileBytes = 32768;  // 128 rows x 128 bf16
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr float kRescaleThreshold = 8.0f;  // in log2 units: P stays below 2^8

struct FwdSmem {
    alignas(1024) uint8_t q[2][kTileBytes];
    alignas(1024) uint8_t kv[kStages][kTileBytes];
    alignas(8) uint64_t q_full;
    uint64_t kv_full[kStages], kv_empty[kStages];
    uint64_t s_full[2], p_half[2], p_full[2], o_full[2];
    uint32_t tmem_base;
    int abort_flag;
    int lo_min, hi_max, lo_max, hi_min, bs_min, be_max;
};

struct TcFwdParams {
    BaMeta meta;
    BaRange r;
    void *o;
    float *lse;
    int h_q, h_kv, group, pairs_per_group;
    float scale_log2;
    int partial_out;
    int main_tiles, total_tiles;
    // Step-major (per-depth) call: depth > 0.  The query rows are the depth-`depth` tokens of
    // branches [tok_begin, tok_end) (r.tok_* hold BRANCH indices then), the query tensor and the
    // outputs are indexed by branch, and the branch keys are stored depth-major after the main
    // rows: token (depth j + 1, branch b) is key row N + j * num_branches + b.
    int depth, num_branches, branch_len;
    int *status;
};

// bits [lo, hi] of a 64-bit word (empty if lo > hi)
__device__ __forceinline__ uint64_t bit_range(int lo, int hi) {
    lo = max(lo, 0);
    hi = min(hi, 63);
    if (lo > hi) return 0ull;
    return (~0ull >> (63 - hi)) & (~0ull << lo);
}

// Eq. (lse-merge) on one 32-column chunk of an fp32 row: dst = dst * w_old + r * w_new
// (dst is not read when w_old is 0: it may be uninitialised then)
__device__ __forceinline__ void merge_row_chunk(void *o, size_t elem_off, const uint32_t (&r)[32], float w_new,
                                                float w_old) {
    float4 *dst = reinterpret_cast<float4 *>((float *)o + elem_off);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
        if (w_old != 0.f) a = dst[i];
        a.x = a.x * w_old + __uint_as_float(r[4 * i]) * w_new;
        a.y = a.y * w_old + __uint_as_float(r[4 * i + 1]) * w_new;
        a.z = a.z * w_old + __uint_as_float(r[4 * i + 2]) * w_new;
        a.w = a.w * w_old + __uint_as_float(r[4 * i + 3]) * w_new;
        dst[i] = a;
    }
}

template <bool OUT_F32>
__device__ __forceinline__ void store_row_chunk(void *o, size_t elem_off, const uint32_t (&r)[32], float inv) {
    if (OUT_F32) {
        float4 *dst = reinterpret_cast<float4 *>((float *)o + elem_off);
#pragma unroll
        for (int i = 0; i < 8; ++i)
            dst[i] = make_float4(__uint_as_float(r[4 * i]) * inv, __uint_as_float(r[4 * i + 1]) * inv,
                                 __uint_as_float(r[4 * i + 2]) * inv, __uint_as_float(r[4 * i + 3]) * inv);
    } else {
        uint4 *dst = reinterpret_cast<uint4 *>((__nv_bfloat16 *)o + elem_off);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            uint4 v;
            v.x = pack_bf16(__uint_as_float(r[8 * i]) * inv, __uint_as_float(r[8 * i + 1]) * inv);
            v.y = pack_bf16(__uint_as_float(r[8 * i + 2]) * inv, __uint_as_float(r[8 * i + 3]) * inv);
            v.z = pack_bf16(__uint_as_float(r[8 * i + 4]) * inv, __uint_as_float(r[8 * i + 5]) * inv);
            v.w = pack_bf16(__uint_as_float(r[8 * i + 6]) * inv, __uint_as_float(r[8 * i + 7]) * inv);
            dst[i] = v;
        }
    }
}

// max over one 32-column chunk of scores (masked columns count as -inf)
template <bool MASKED>
__device__ __forceinline__ float chunk_max(const uint32_t (&r)[32], uint32_t mk, float m) {
    float m0 = m, m1 = -INFINITY, m2 = -INFINITY, m3 = -INFINITY;
#pragma unroll
    for (int e = 0; e < 32; e += 4) {
        float a = __uint_as_float(r[e]), b = __uint_as_float(r[e + 1]);
        float c = __uint_as_float(r[e + 2]), d = __uint_as_float(r[e + 3]);
        if (MASKED) {
            a = ((mk >> e) & 1u) ? a : -INFINITY;
            b = ((mk >> (e + 1)) & 1u) ? b : -INFINITY;
            c = ((mk >> (e + 2)) & 1u) ? c : -INFINITY;
            d = ((mk >> (e + 3)) & 1u) ? d : -INFINITY;
        }
        m0 = fmaxf(m0, a); m1 = fmaxf(m1, b); m2 = fmaxf(m2, c); m3 = fmaxf(m3, d);
    }
    return fmaxf(fmaxf(m0, m1), fmaxf(m2, m3));
}

// p = 2^(s * sl2 + neg_ms) for one 32-column chunk -> 16 packed bf16 pairs; the
// row sum is kept as two partial sums (packed fp32 add)
template <bool MASKED>
__device__ __forceinline__ void chunk_exp(const uint32_t (&r)[32], uint32_t mk, float sl2, float neg_ms,
                                          float2 &lsum, uint32_t (&pk)[16]) {
    const float2 s2 = make_float2(sl2, sl2), n2 = make_float2(neg_ms, neg_ms);
#pragma unroll
    for (int e = 0; e < 32; e += 2) {
        const float2 x = ffma2(make_float2(__uint_as_float(r[e]), __uint_as_float(r[e + 1])), s2, n2);
        float2 pp = make_float2(ex2(x.x), ex2(x.y));
        if (MASKED) {
            pp.x = ((mk >> e) & 1u) ? pp.x : 0.f;
            pp.y = ((mk >> (e + 1)) & 1u) ? pp.y : 0.f;
        }
        lsum = fadd2(lsum, pp);
        pk[e >> 1] = pack_bf16(pp.x, pp.y);
    }
}

__global__ void __launch_bounds__(kThreads, 1)
tc_fwd_kernel(const __grid_constant__ CUtensorMap tm_q_main, const __grid_constant__ CUtensorMap tm_q_branch,
              const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
              const TcFwdParams p) {
    extern __shared__ uint8_t smem_raw[];
    FwdSmem &sm = *reinterpret_cast<FwdSmem *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    volatile int *abort_flag = &sm.abort_flag;

    // ---- work item: later (longer-prefix) row tiles first; the CTAs of one row
    // tile (all KV heads and head pairs) are adjacent so they share K/V in L2
    const int per_tile = p.h_kv * p.pairs_per_group;
    const int tile = p.total_tiles - 1 - (int)(blockIdx.x / per_tile);
    const int inner = (int)(blockIdx.x % per_tile);
    const int g = inner / p.pairs_per_group, hp = inner % p.pairs_per_group;
    const int h0 = g * p.group + 2 * hp;
    const bool second_head = 2 * hp + 1 < p.group;
    const int h1 = second_head ? h0 + 1 : h0;
    const bool is_main = tile < p.main_tiles;
    const int64_t n = p.meta.n_main;
    // first row of the tile inside its tensor (q_main rows / q_branch tokens)
    const int64_t row0 = is_main ? p.r.qm_begin + (int64_t)tile * kTile
                                 : p.r.tok_begin + (int64_t)(tile - p.main_tiles) * kTile;
    const int64_t row_end = is_main ? p.r.qm_end : p.r.tok_end;

    if (tid == 0) {
        mbar_init(&sm.q_full, 1);
        for (int s = 0; s < kStages; ++s) { mbar_init(&sm.kv_full[s], 1); mbar_init(&sm.kv_empty[s], 1); }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&sm.s_full[i], 1);
            mbar_init(&sm.p_half[i], 128);
            mbar_init(&sm.p_full[i], 128);
            mbar_init(&sm.o_full[i], 1);
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
    if (warp == 9 && lane == 0) {
        tma_prefetch_desc(is_main ? &tm_q_main : &tm_q_branch);
        tma_prefetch_desc(&tm_k);
        tma_prefetch_desc(&tm_v);
    }
    __syncthreads();

    // ---- per-row metadata (softmax threads: row = tid % 128)
    int lo = 1, hi = 0, bstart = 0;
    uint64_t bmask = 0;
    bool valid = false;
    int64_t my_row = 0;
    if (warp < 8) {
        my_row = row0 + (tid & 127);
        valid = my_row < row_end;
        if (valid) {
            // depth mode: my_row is a branch index; all tokens of a branch share the causal prefix
            const int64_t grow = is_main ? my_row : n + (p.depth ? my_row * p.branch_len : my_row);
            if (p.r.parts & BA_PART_MAIN) {
                lo = max(p.meta.row_lo[grow], (int)p.r.kv_begin);
                hi = min(p.meta.row_hi[grow], (int)p.r.kv_end - 1);
                if (hi < lo) { lo = 1; hi = 0; }
            }
            if (!is_main && (p.r.parts & BA_PART_BRANCH) && !p.depth) {
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
                if (!is_main && (p.r.parts & BA_PART_BRANCH) && !p.depth) {
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

    // ---- key tiles: aligned 128-key main tiles [kt0, kt0 + n_main), then the
    // own-branch keys [bs, be) as n_br tiles starting at bs
    int kt0 = 0, n_main_tiles = 0, n_br = 0;
    if (sm.hi_max >= sm.lo_min) {
        kt0 = sm.lo_min / kTile;
        n_main_tiles = sm.hi_max / kTile - kt0 + 1;
    }
    const int bs = sm.bs_min;
    if (sm.be_max > bs) n_br = (sm.be_max - bs + kTile - 1) / kTile;
    // depth mode: one key tile per depth 1 .. depth, holding the tokens of this tile's own branches
    // in branch order, so row i sees exactly column i of each of them
    if (p.depth && (p.r.parts & BA_PART_BRANCH)) n_br = p.depth;
    const int T = n_main_tiles + n_br;
    const int full_lo = sm.lo_max, full_hi = sm.hi_min;

    if (warp == 9) {
        // ================================================= TMA producer
        if (lane == 0 && T > 0) {
            const CUtensorMap *tq = is_main ? &tm_q_main : &tm_q_branch;
            mbar_expect_tx(&sm.q_full, 2 * kTileBytes);
            for (int half = 0; half < 2; ++half) {
                tma_load_3d(sm.q[0] + half * 16384, tq, half * 64, h0, (int)row0, &sm.q_full);
                tma_load_3d(sm.q[1] + half * 16384, tq, half * 64, h1, (int)row0, &sm.q_full);
            }
            int issued = 0;
            bool ok = true;
            for (int it = 0; it < 2 * T && ok; ++it) {
                const int j = it >> 1, s = it % kStages;
                if (it >= kStages) ok = mbar_wait(&sm.kv_empty[s], ((it / kStages) - 1) & 1, abort_flag);
                if (!ok) break;
                const int krow = j < n_main_tiles ? (kt0 + j) * kTile
                                 : p.depth ? (int)n + (j - n_main_tiles) * p.num_branches + (int)row0
                                           : (int)n + bs + (j - n_main_tiles) * kTile;
                const CUtensorMap *tkv = (it & 1) ? &tm_v : &tm_k;
                mbar_expect_tx(&sm.kv_full[s], kTileBytes);
                tma_load_3d(sm.kv[s], tkv, 0, g, krow, &sm.kv_full[s]);
                tma_load_3d(sm.kv[s] + 16384, tkv, 64, g, krow, &sm.kv_full[s]);
                issued = it + 1;
            }
            if (!ok) {
                // leave no copy in flight behind: wait (bounded) for what was issued
                for (int it = max(issued - kStages, 0); it < issued; ++it) {
                    uint32_t spins = 0;
                    while (!mbar_try_wait(&sm.kv_full[it % kStages], (it / kStages) & 1) && ++spins < (1u << 22)) {}
                }
            }
        }
    } else if (warp == 8) {
        // ================================================= MMA issuer
        // The whole warp runs this code and an elected lane issues each MMA and commit: with
        // warp-uniform control flow the descriptors stay in uniform registers, which halves what
        // a tcgen05.mma costs its thread.  Every lane waits, and all agree on the outcome.
        if (T > 0) {
            constexpr uint32_t IDESC_QK = idesc_bf16(128, 128, 0);
            constexpr uint32_t IDESC_PV = idesc_bf16(128, 128, 1);
            // low descriptor words (the issuing thread advances them with one add per MMA)
            const uint32_t q_km[2] = {smem_desc_lo(smem_u32(sm.q[0]), 16), smem_desc_lo(smem_u32(sm.q[1]), 16)};
            const uint32_t kv_km0 = smem_desc_lo(smem_u32(sm.kv[0]), 16), kv_mn0 = smem_desc_lo(smem_u32(sm.kv[0]), 16384);
            constexpr uint32_t kStageStep = kTileBytes >> 4;
            auto issue_qk = [&](int i, int stage) {
                const uint32_t k_km = kv_km0 + stage * kStageStep;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)
                    if (elect_one()) mma_ss_lh(tmem + i * 128, q_km[i] + desc_step_kmajor(ks), k_km + desc_step_kmajor(ks), IDESC_QK, ks > 0);
            };
            auto issue_pv = [&](int i, int stage, bool accumulate, int ks0) {   // K steps ks0 .. ks0 + 3
                const uint32_t v_mn = kv_mn0 + stage * kStageStep;
#pragma unroll
                for (int ks = ks0; ks < ks0 + 4; ++ks)
                    if (elect_one()) mma_ts_lh(tmem + 256 + i * 128, tmem + i * 128 + ks * 8, v_mn + desc_step_mnmajor(ks), IDESC_PV,
                              accumulate || ks > 0);
            };
            bool ok = __all_sync(0xffffffffu, mbar_wait(&sm.q_full, 0, abort_flag));
            ok = ok && __all_sync(0xffffffffu, mbar_wait(&sm.kv_full[0], 0, abort_flag));
            if (ok) {
                tc_fence_after();
                issue_qk(0, 0); if (elect_one()) tc_commit(&sm.s_full[0]);
                issue_qk(1, 0); if (elect_one()) tc_commit(&sm.s_full[1]);
                if (elect_one()) tc_commit(&sm.kv_empty[0]);
            }
            for (int j = 0; j < T && ok; ++j) {
                const int it_v = 2 * j + 1, sv = it_v % kStages;
                const int it_k = 2 * j + 2, sk = it_k % kStages;
                for (int i = 0; i < 2 && ok; ++i) {
                    ok = __all_sync(0xffffffffu, mbar_wait(&sm.p_half[i], j & 1, abort_flag));
                    if (ok && i == 0) ok = __all_sync(0xffffffffu, mbar_wait(&sm.kv_full[sv], (it_v / kStages) & 1, abort_flag));
                    if (!ok) break;
                    tc_fence_after();
                    issue_pv(i, sv, j > 0, 0);            // keys 0-63 while the softmax warps finish keys 64-127
                    ok = __all_sync(0xffffffffu, mbar_wait(&sm.p_full[i], j & 1, abort_flag));
                    if (!ok) break;
                    tc_fence_after();
                    issue_pv(i, sv, true, 4);
                    if (i == 1) if (elect_one()) tc_commit(&sm.kv_empty[sv]);
                    if (j + 1 < T) {
                        if (i == 0) {
                            ok = __all_sync(0xffffffffu, mbar_wait(&sm.kv_full[sk], (it_k / kStages) & 1, abort_flag));
                            if (!ok) break;
                            tc_fence_after();
                        }
                        issue_qk(i, sk); if (elect_one()) tc_commit(&sm.s_full[i]);
                        if (i == 1) if (elect_one()) tc_commit(&sm.kv_empty[sk]);
                    } else {
                        if (elect_one()) tc_commit(&sm.o_full[i]);
                    }
                }
            }
        }
    } else {
        // ================================================= softmax + epilogue
        const int i = warp >> 2;                                   // query tile 0 / 1
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t s_addr = tmem + lane_base + i * 128;
        const uint32_t o_addr = tmem + lane_base + 256 + i * 128;
        const float sl2 = p.scale_log2;
        float m_run = -INFINITY, l_run = 0.f;
        bool ok = true;
        for (int j = 0; j < T; ++j) {
            ok = mbar_wait(&sm.s_full[i], j & 1, abort_flag);
            if (!ok) break;
            tc_fence_after();
            // --- visibility of this tile's 128 key columns for my row
            bool masked;
            uint64_t vis[2] = {~0ull, ~0ull};
            if (j < n_main_tiles) {
                const int kj = (kt0 + j) * kTile;
                masked = !(kj >= full_lo && kj + kTile - 1 <= full_hi);
                if (masked) {
                    vis[0] = bit_range(lo - kj, hi - kj);
                    vis[1] = bit_range(lo - kj - 64, hi - kj - 64);
                }
            } else if (p.depth) {
                masked = true;
                const int c = tid & 127;     // depth mode: column c is the same branch as row c
                vis[0] = (valid && c < 64) ? 1ull << c : 0ull;
                vis[1] = (valid && c >= 64) ? 1ull << (c - 64) : 0ull;
            } else {
                masked = true;
                // column c is branch token bs + 128 (j - n_main_tiles) + c; bit c = bmask bit (c + off)
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
            const uint32_t mk0 = (uint32_t)vis[0], mk1 = (uint32_t)(vis[0] >> 32);
            const uint32_t mk2 = (uint32_t)vis[1], mk3 = (uint32_t)(vis[1] >> 32);
            // --- pass 1: row maximum (chunks 2, 3, then 0, 1, which stay in registers)
            uint32_t ra[32], rb[32];
            float m_tile;
            tmem_ld32(s_addr + 64, ra);
            tmem_ld32(s_addr + 96, rb);
            tmem_wait_ld();
            if (masked) {
                m_tile = chunk_max<true>(ra, mk2, -INFINITY);
                tmem_ld32(s_addr, ra);
                m_tile = chunk_max<true>(rb, mk3, m_tile);
                tmem_ld32(s_addr + 32, rb);
                tmem_wait_ld();
                m_tile = chunk_max<true>(ra, mk0, m_tile);
                m_tile = chunk_max<true>(rb, mk1, m_tile);
            } else {
                m_tile = chunk_max<false>(ra, 0u, -INFINITY);
                tmem_ld32(s_addr, ra);
                m_tile = chunk_max<false>(rb, 0u, m_tile);
                tmem_ld32(s_addr + 32, rb);
                tmem_wait_ld();
                m_tile = chunk_max<false>(ra, 0u, m_tile);
                m_tile = chunk_max<false>(rb, 0u, m_tile);
            }
            // --- running maximum; O and l are rescaled only when it grew a lot
            const float m_new = fmaxf(m_run, m_tile);
            float alpha = 1.0f;
            const bool grow = m_new > m_run && (m_run == -INFINITY || (m_new - m_run) * sl2 > kRescaleThreshold);
            if (grow) {
                alpha = ex2((m_run - m_new) * sl2);  // m_run = -inf gives 0
                l_run *= alpha;
                m_run = m_new;
            }
            if (j > 0 && __any_sync(0xffffffffu, grow)) {
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    uint32_t r[32];
                    tmem_ld32(o_addr + c * 32, r);
                    tmem_wait_ld();
#pragma unroll
                    for (int e = 0; e < 32; ++e) r[e] = __float_as_uint(__uint_as_float(r[e]) * alpha);
                    tmem_st32(o_addr + c * 32, r);
                }
            }
            const float neg_ms = m_run == -INFINITY ? 0.f : -m_run * sl2;
            // --- pass 2: P = exp2(s * scale_log2 - m), bf16, over the first 64 score columns
            float2 l2 = make_float2(0.f, 0.f);
            uint32_t pk[16];
            if (masked) {
                chunk_exp<true>(ra, mk0, sl2, neg_ms, l2, pk);
                tmem_st16(s_addr, pk);
                tmem_ld32(s_addr + 64, ra);
                chunk_exp<true>(rb, mk1, sl2, neg_ms, l2, pk);
                tmem_st16(s_addr + 16, pk);
                tmem_ld32(s_addr + 96, rb);
                tmem_wait_st();
                tc_fence_before();
                mbar_arrive(&sm.p_half[i]);       // P of keys 0-63 is in place: P V may start
                tmem_wait_ld();
                chunk_exp<true>(ra, mk2, sl2, neg_ms, l2, pk);
                tmem_st16(s_addr + 32, pk);
                chunk_exp<true>(rb, mk3, sl2, neg_ms, l2, pk);
                tmem_st16(s_addr + 48, pk);
            } else {
                chunk_exp<false>(ra, 0u, sl2, neg_ms, l2, pk);
                tmem_st16(s_addr, pk);
                tmem_ld32(s_addr + 64, ra);
                chunk_exp<false>(rb, 0u, sl2, neg_ms, l2, pk);
                tmem_st16(s_addr + 16, pk);
                tmem_ld32(s_addr + 96, rb);
                tmem_wait_st();
                tc_fence_before();
                mbar_arrive(&sm.p_half[i]);       // P of keys 0-63 is in place: P V may start
                tmem_wait_ld();
                chunk_exp<false>(ra, 0u, sl2, neg_ms, l2, pk);
                tmem_st16(s_addr + 32, pk);
                chunk_exp<false>(rb, 0u, sl2, neg_ms, l2, pk);
                tmem_st16(s_addr + 48, pk);
            }
            const float l_add = l2.x + l2.y;
            l_run += l_add;
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(&sm.p_full[i]);
        }
        // --- epilogue: O / l and LSE
        if (ok && T > 0) ok = mbar_wait(&sm.o_full[i], 0, abort_flag);
        tc_fence_after();
        {
            const bool do_store = ok && valid && (i == 0 || second_head);
            const int h = i == 0 ? h0 : h1;
            int64_t orow = is_main ? my_row : n + my_row;
            if (p.depth) orow = my_row;              // outputs of a per-depth call are indexed by branch
            else if (p.partial_out)
                orow = is_main ? my_row - p.r.qm_begin : (p.r.qm_end - p.r.qm_begin) + (my_row - p.r.tok_begin);
            const float inv = l_run > 0.f ? 1.0f / l_run : 0.f;
            const size_t base = ((size_t)orow * p.h_q + h) * 128;
            const float lse_p = l_run > 0.f ? (m_run * sl2 + log2f(l_run)) * kLn2 : -INFINITY;
            float w_new = inv, w_old = 0.f;   // partial_out == 2: weights of Eq. (lse-merge)
            if (do_store) {
                float lse_out = lse_p;
                if (p.partial_out == 2) {
                    const float lse_a = p.lse[orow * p.h_q + h];
                    const float mx = fmaxf(lse_a, lse_p);
                    if (mx == -INFINITY) {
                        lse_out = -INFINITY; w_new = 0.f;
                    } else {
                        const float ea = expf(lse_a - mx), ep = expf(lse_p - mx), s = ea + ep;
                        lse_out = mx + logf(s);
                        w_old = ea / s;
                        w_new = ep / s * inv;
                    }
                }
                p.lse[orow * p.h_q + h] = lse_out;
            }
            // every lane runs the (warp-collective) TMEM loads; only live rows store
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint32_t r[32];
                if (T > 0 && ok) {
                    tmem_ld32(o_addr + c * 32, r);
                    tmem_wait_ld();
                } else {
#pragma unroll
                    for (int e = 0; e < 32; ++e) r[e] = 0u;
                }
                if (do_store) {
                    if (p.partial_out == 2) merge_row_chunk(p.o, base + c * 32, r, w_new, w_old);
                    else if (p.partial_out) store_row_chunk<true>(p.o, base + c * 32, r, inv);
                    else store_row_chunk<false>(p.o, base + c * 32, r, inv);
                }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 8) tmem_dealloc(tmem, 512);
    if (tid == 0 && sm.abort_flag) atomicExch(p.status, BA_ETIMEOUT);
}

}  // namespace

bool ba_tc_supported(const ba_problem_t *p) {
    return p->dtype == BA_BF16 && p->head_dim == 128 && encode_tiled_fn() != nullptr;
}

int ba_tc_fwd(const ba_plan *pl, const BaRange &r, const void *q_main, const void *q_branch, const void *k,
              const void *v, void *o, float *lse, int partial_out, cudaStream_t st, int depth) {
    // the dynamic shared-memory limit is a per-device attribute of the kernel
    static bool attr_set[64] = {};
    int dev = 0;
    BA_CUDA_CHECK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return BA_EUNSUPPORTED;
    const size_t smem = sizeof(FwdSmem) + 1024;
    if (!attr_set[dev]) {
        BA_CUDA_CHECK(cudaFuncSetAttribute(tc_fwd_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        attr_set[dev] = true;
    }
    const ba_problem_t &pr = pl->prob;
    TcFwdParams p;
    memset(&p, 0, sizeof p);
    p.meta = pl->meta;
    p.r = r;
    p.o = o;
    p.lse = lse;
    p.h_q = pr.h_q;
    p.h_kv = pr.h_kv;
    p.group = pr.h_q / pr.h_kv;
    p.pairs_per_group = (p.group + 1) / 2;
    p.scale_log2 = pl->scale * kLog2e;
    p.partial_out = partial_out;   // 0 final layout, 1 compact fp32, 2 compact fp32 merged in place
    p.status = pl->dev_status;
    p.depth = depth;
    p.num_branches = pr.num_branches;
    p.branch_len = pr.uniform_len;
    const int64_t mt = q_main ? (r.qm_end - r.qm_begin + kTile - 1) / kTile : 0;
    const int64_t bt = (r.tok_end - r.tok_begin + kTile - 1) / kTile;
    p.main_tiles = (int)mt;
    p.total_tiles = (int)(mt + bt);
    if (p.total_tiles == 0) return BA_OK;

    CUtensorMap tq_main, tq_branch, tk, tv;
    // depth mode: only the key rows of depths <= depth exist yet; rows beyond them read as zero
    const uint64_t kv_rows = depth ? (uint64_t)(pr.n_main + (int64_t)depth * pr.num_branches)
                                   : (uint64_t)(pr.n_main + pr.n_branch);
    if (!make_tmap_rhd(&tk, k, kv_rows, pr.h_kv, 128, kTile) || !make_tmap_rhd(&tv, v, kv_rows, pr.h_kv, 128, kTile))
        return BA_EINVAL;
    // an absent query tensor still needs a valid map object: alias the other one
    const void *qm = q_main ? q_main : q_branch;
    const void *qb = (q_branch && pr.n_branch > 0) ? q_branch : q_main;
    const uint64_t qm_rows = depth ? (uint64_t)pr.num_branches : q_main ? (uint64_t)pr.n_main : (uint64_t)pr.n_branch;
    uint64_t qb_rows = (q_branch && pr.n_branch > 0) ? (uint64_t)pr.n_branch : (uint64_t)pr.n_main;
    if (depth) qb_rows = (uint64_t)pr.num_branches;     // the queries of one depth: one row per branch
    if (!make_tmap_rhd(&tq_main, qm, qm_rows, pr.h_q, 128, kTile) ||
        !make_tmap_rhd(&tq_branch, qb, qb_rows, pr.h_q, 128, kTile))
        return BA_EINVAL;
    const int64_t grid = (int64_t)p.total_tiles * pr.h_kv * p.pairs_per_group;
    if (grid > INT_MAX) return BA_EUNSUPPORTED;
    tc_fwd_kernel<<<(unsigned)grid, kThreads, smem, st>>>(tq_main, tq_branch, tk, tv, p);
    return ba_check_launch();
}
