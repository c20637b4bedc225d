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
#include "ba_tc_bwd.cuh"

using namespace sm100;

namespace {

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

// P = 2^(s * sl2 + neg_lse2) for one 32-column chunk, as 16 packed bf16 pairs
template <bool MASKED>
__device__ __forceinline__ void chunk_p(const uint32_t (&r)[32], uint32_t mk, float sl2, float neg_lse2,
                                        uint32_t *pr) {
    const float2 s2 = make_float2(sl2, sl2), n2 = make_float2(neg_lse2, neg_lse2);
#pragma unroll
    for (int e = 0; e < 32; e += 2) {
        const float2 x = ffma2(make_float2(__uint_as_float(r[e]), __uint_as_float(r[e + 1])), s2, n2);
        float p0 = ex2(x.x), p1 = ex2(x.y);
        if (MASKED) {
            p0 = ((mk >> e) & 1u) ? p0 : 0.f;
            p1 = ((mk >> (e + 1)) & 1u) ? p1 : 0.f;
        }
        pr[e >> 1] = pack_bf16(p0, p1);
    }
}

// dS = P o (dP - delta) for one 32-column chunk (P given as packed bf16 pairs)
__device__ __forceinline__ void chunk_ds(const uint32_t (&r)[32], const uint32_t *pr, float dlt,
                                         uint32_t (&pk)[16]) {
    const float2 nd = make_float2(-dlt, -dlt);
#pragma unroll
    for (int e = 0; e < 32; e += 2) {
        const uint32_t pp = pr[e >> 1];
        const float2 pf = make_float2(__uint_as_float(pp << 16), __uint_as_float(pp & 0xffff0000u));
        const float2 d = fmul2(pf, fadd2(make_float2(__uint_as_float(r[e]), __uint_as_float(r[e + 1])), nd));
        pk[e >> 1] = pack_bf16(d.x, d.y);
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
        // the whole warp runs this code, an elected lane issues each MMA and commit (descriptors
        // then stay in uniform registers); every lane waits and all agree on the outcome
        if (T > 0) {
            constexpr uint32_t IDESC_KMAJ = idesc_bf16(128, 128, 0);  // S = Q K^T, dP = dO V^T
            constexpr uint32_t IDESC_MN = idesc_bf16(128, 128, 1);    // dQ += dS K
            // low descriptor words (the issuing thread advances them with one add per MMA)
            const uint32_t q_addr[2] = {smem_desc_lo(smem_u32(sm.q[0]), 16), smem_desc_lo(smem_u32(sm.q[1]), 16)};
            const uint32_t go_addr[2] = {smem_desc_lo(smem_u32(sm.go[0]), 16), smem_desc_lo(smem_u32(sm.go[1]), 16)};
            const uint32_t k_km[2] = {smem_desc_lo(smem_u32(sm.kbuf[0]), 16), smem_desc_lo(smem_u32(sm.kbuf[1]), 16)};
            const uint32_t k_mn[2] = {smem_desc_lo(smem_u32(sm.kbuf[0]), 16384), smem_desc_lo(smem_u32(sm.kbuf[1]), 16384)};
            const uint32_t v_km = smem_desc_lo(smem_u32(sm.vbuf), 16);
            auto issue_kmajor = [&](uint32_t d_tmem, uint32_t a_km, uint32_t b_km) {
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)
                    if (elect_one()) mma_ss_lh(d_tmem, a_km + desc_step_kmajor(ks), b_km + desc_step_kmajor(ks), IDESC_KMAJ, ks > 0);
            };
            auto issue_dq = [&](int i, uint32_t kmn, bool accumulate) {
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)
                    if (elect_one()) mma_ts_lh(tmem + 256 + i * 128, tmem + i * 128 + ks * 8, kmn + desc_step_mnmajor(ks), IDESC_MN,
                              accumulate || ks > 0);
            };
            bool ok = __all_sync(0xffffffffu, mbar_wait(&sm.q_full, 0, abort_flag));
            ok = ok && __all_sync(0xffffffffu, mbar_wait(&sm.k_full[0], 0, abort_flag));
            if (ok) {
                tc_fence_after();
                issue_kmajor(tmem + 0, q_addr[0], k_km[0]); if (elect_one()) tc_commit(&sm.s_full[0]);
                issue_kmajor(tmem + 128, q_addr[1], k_km[0]); if (elect_one()) tc_commit(&sm.s_full[1]);
            }
            for (int j = 0; j < T && ok; ++j) {
                const int kb = j & 1;
                for (int i = 0; i < 2 && ok; ++i) {
                    ok = __all_sync(0xffffffffu, mbar_wait(&sm.a_done[i], j & 1, abort_flag));
                    if (ok && i == 0) ok = __all_sync(0xffffffffu, mbar_wait(&sm.v_full, j & 1, abort_flag));
                    if (!ok) break;
                    tc_fence_after();
                    issue_kmajor(tmem + i * 128, go_addr[i], v_km);
                    if (elect_one()) tc_commit(&sm.dp_full[i]);
                    if (i == 1) if (elect_one()) tc_commit(&sm.v_empty);
                }
                for (int i = 0; i < 2 && ok; ++i) {
                    ok = __all_sync(0xffffffffu, mbar_wait(&sm.b_done[i], j & 1, abort_flag));
                    if (!ok) break;
                    tc_fence_after();
                    issue_dq(i, k_mn[kb], j > 0);
                    if (i == 1) if (elect_one()) tc_commit(&sm.k_empty[kb]);
                    if (j + 1 < T) {
                        if (i == 0) {
                            ok = __all_sync(0xffffffffu, mbar_wait(&sm.k_full[kb ^ 1], ((j + 1) >> 1) & 1, abort_flag));
                            if (!ok) break;
                            tc_fence_after();
                        }
                        issue_kmajor(tmem + i * 128, q_addr[i], k_km[kb ^ 1]);
                        if (elect_one()) tc_commit(&sm.s_full[i]);
                    } else {
                        if (elect_one()) tc_commit(&sm.dq_full[i]);
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
            neg_lse2 = p.nlse2_t[(size_t)h * p.row_pitch + grow];
            dlt = p.delta_t[(size_t)h * p.row_pitch + grow];
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
            const uint32_t mk0 = (uint32_t)vis[0], mk1 = (uint32_t)(vis[0] >> 32);
            const uint32_t mk2 = (uint32_t)vis[1], mk3 = (uint32_t)(vis[1] >> 32);
            uint32_t pr[64], ra[32], rb[32];
            tmem_ld32(r_addr, ra);
            tmem_ld32(r_addr + 32, rb);
            tmem_wait_ld();
            if (masked) {
                chunk_p<true>(ra, mk0, sl2, neg_lse2, &pr[0]);
                tmem_ld32(r_addr + 64, ra);
                chunk_p<true>(rb, mk1, sl2, neg_lse2, &pr[16]);
                tmem_ld32(r_addr + 96, rb);
                tmem_wait_ld();
                chunk_p<true>(ra, mk2, sl2, neg_lse2, &pr[32]);
                chunk_p<true>(rb, mk3, sl2, neg_lse2, &pr[48]);
            } else {
                chunk_p<false>(ra, 0u, sl2, neg_lse2, &pr[0]);
                tmem_ld32(r_addr + 64, ra);
                chunk_p<false>(rb, 0u, sl2, neg_lse2, &pr[16]);
                tmem_ld32(r_addr + 96, rb);
                tmem_wait_ld();
                chunk_p<false>(ra, 0u, sl2, neg_lse2, &pr[32]);
                chunk_p<false>(rb, 0u, sl2, neg_lse2, &pr[48]);
            }
            tc_fence_before();
            mbar_arrive(&sm.a_done[i]);
            // --- phase B: dS = P o (dP - delta), bf16, over the first 64 columns
            ok = mbar_wait(&sm.dp_full[i], j & 1, abort_flag);
            if (!ok) break;
            tc_fence_after();
            {
                uint32_t pk[16];
                tmem_ld32(r_addr, ra);
                tmem_ld32(r_addr + 32, rb);
                tmem_wait_ld();
                chunk_ds(ra, &pr[0], dlt, pk);
                tmem_st16(r_addr, pk);
                tmem_ld32(r_addr + 64, ra);
                chunk_ds(rb, &pr[16], dlt, pk);
                tmem_st16(r_addr + 16, pk);
                tmem_ld32(r_addr + 96, rb);
                tmem_wait_ld();
                chunk_ds(ra, &pr[32], dlt, pk);
                tmem_st16(r_addr + 32, pk);
                chunk_ds(rb, &pr[48], dlt, pk);
                tmem_st16(r_addr + 48, pk);
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


// ============================================================================
// dK / dV
// ============================================================================
// Key-stationary: one CTA owns 128 key rows of one KV head, keeps K_j, V_j in
// shared memory and dK_j, dV_j (fp32) in TMEM, and walks the query rows that
// can see those keys -- all query heads of the KV head -- as 64-row sub-tiles.
// Everything is computed transposed so that the key index is the TMEM lane:
//   S^T = K_j Q^T, dP^T = V_j dO^T        (128 keys x 64 query rows)
//   P^T = exp2(scale_log2 S^T - lse2[col]),  dS^T = P^T o (dP^T - delta[col])
//   dV_j += P^T dO,  dK_j += dS^T Q          (P^T, dS^T are TMEM A operands)
// Two sub-tiles are in flight (sets 0 / 1, one softmax warpgroup each).
//   TMEM: dK [0,128) dV [128,256); set b: XS_b = 256 + 128 b (64 cols: S^T, its
//   first 32 columns then hold P^T), XD_b = XS_b + 64 (dP^T, then dS^T)
constexpr int kKvThreads = 320;
constexpr int kSub = 64;           // query rows per sub-tile
constexpr int kQStages = 4;
constexpr uint32_t kSubBytes = 16384;  // 64 rows x 128 bf16

struct SubMeta {
    float neg_lse2[kSub];
    float delta[kSub];
    int bstart[kSub];
    unsigned long long mask[kSub];
};

struct KvSmem {
    alignas(1024) uint8_t k[kTileBytes];
    alignas(1024) uint8_t v[kTileBytes];
    alignas(1024) uint8_t qs[kQStages][2 * kSubBytes];  // Q sub-tile, then dO sub-tile
    alignas(16) SubMeta meta[kQStages];
    alignas(8) uint64_t kv_full;
    uint64_t q_full[kQStages], q_empty[kQStages];
    uint64_t sd_full[2], pd_done[2], acc_full;
    uint32_t tmem_base;
    int abort_flag;
    int qend_max, bq0_min, bq1_max;
};

// 16 columns of the transposed tile: P^T and dS^T as 8 packed bf16 pairs each;
// nl / dl point at the columns' -lse2 and delta in shared memory
template <bool MASKED>
__device__ __forceinline__ void quarter_pds(const uint32_t (&rs)[16], const uint32_t (&rd)[16], uint32_t mk,
                                            float sl2, const float *nl, const float *dl, uint32_t (&pk)[8],
                                            uint32_t (&dk8)[8]) {
    const float2 s2 = make_float2(sl2, sl2);
    const float4 *nl4 = reinterpret_cast<const float4 *>(nl);
    const float4 *dl4 = reinterpret_cast<const float4 *>(dl);
#pragma unroll
    for (int e = 0; e < 16; e += 4) {
        const float4 nv = nl4[e >> 2], dv = dl4[e >> 2];
        const float2 x0 = ffma2(make_float2(__uint_as_float(rs[e]), __uint_as_float(rs[e + 1])), s2,
                                make_float2(nv.x, nv.y));
        const float2 x1 = ffma2(make_float2(__uint_as_float(rs[e + 2]), __uint_as_float(rs[e + 3])), s2,
                                make_float2(nv.z, nv.w));
        float2 p0 = make_float2(ex2(x0.x), ex2(x0.y)), p1 = make_float2(ex2(x1.x), ex2(x1.y));
        if (MASKED) {
            p0.x = ((mk >> e) & 1u) ? p0.x : 0.f;
            p0.y = ((mk >> (e + 1)) & 1u) ? p0.y : 0.f;
            p1.x = ((mk >> (e + 2)) & 1u) ? p1.x : 0.f;
            p1.y = ((mk >> (e + 3)) & 1u) ? p1.y : 0.f;
        }
        float2 d0 = fmul2(p0, fadd2(make_float2(__uint_as_float(rd[e]), __uint_as_float(rd[e + 1])),
                                    make_float2(-dv.x, -dv.y)));
        float2 d1 = fmul2(p1, fadd2(make_float2(__uint_as_float(rd[e + 2]), __uint_as_float(rd[e + 3])),
                                    make_float2(-dv.z, -dv.w)));
        if (MASKED) {  // the scalars of invisible columns may be anything, even NaN
            d0.x = ((mk >> e) & 1u) ? d0.x : 0.f;
            d0.y = ((mk >> (e + 1)) & 1u) ? d0.y : 0.f;
            d1.x = ((mk >> (e + 2)) & 1u) ? d1.x : 0.f;
            d1.y = ((mk >> (e + 3)) & 1u) ? d1.y : 0.f;
        }
        pk[e >> 1] = pack_bf16(p0.x, p0.y);
        pk[(e >> 1) + 1] = pack_bf16(p1.x, p1.y);
        dk8[e >> 1] = pack_bf16(d0.x, d0.y);
        dk8[(e >> 1) + 1] = pack_bf16(d1.x, d1.y);
    }
}

__global__ void __launch_bounds__(kKvThreads, 1)
tc_dkdv_kernel(const __grid_constant__ CUtensorMap tm_q_main, const __grid_constant__ CUtensorMap tm_q_branch,
               const __grid_constant__ CUtensorMap tm_go, const __grid_constant__ CUtensorMap tm_k,
               const __grid_constant__ CUtensorMap tm_v, const TcBwdParams p) {
    extern __shared__ uint8_t smem_raw[];
    KvSmem &sm = *reinterpret_cast<KvSmem *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    volatile int *abort_flag = &sm.abort_flag;

    // KV-head-major order: the CTAs resident at one time belong to one or two KV
    // heads and stream the same query rows, so that stream is read from HBM about
    // once per head instead of once per wave of CTAs
    const int g = (int)(blockIdx.x / p.total_key_tiles);
    const int tile = (int)(blockIdx.x % p.total_key_tiles);
    const bool main_keys = tile < p.main_key_tiles;
    const int64_t n = p.meta.n_main;
    // first key of the tile: main key index, or branch token index
    const int64_t key0 = main_keys ? p.r.kv_begin + (int64_t)tile * kTile
                                   : p.r.tok_begin + (int64_t)(tile - p.main_key_tiles) * kTile;
    const int64_t key_end = main_keys ? p.r.kv_end : p.r.tok_end;
    const int64_t gkey0 = main_keys ? key0 : n + key0;

    if (tid == 0) {
        mbar_init(&sm.kv_full, 1);
        for (int s = 0; s < kQStages; ++s) { mbar_init(&sm.q_full[s], 2); mbar_init(&sm.q_empty[s], 1); }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&sm.sd_full[b], 1);
            mbar_init(&sm.pd_done[b], 128);
        }
        mbar_init(&sm.acc_full, 1);
        sm.abort_flag = 0;
        sm.qend_max = -1; sm.bq0_min = INT_MAX; sm.bq1_max = -1;
        fence_barrier_init();
    }
    if (warp == 8) {
        tmem_alloc(&sm.tmem_base, 512);
        tmem_relinquish();
    }
    __syncthreads();

    // ---- my key row (threads of both warpgroups: key = tid % 128)
    bool kvalid = false;
    int my_key = 0, my_qend = 0, my_bq0 = 0, my_bq1 = 0;
    if (warp < 8) {
        const int64_t kk = key0 + (tid & 127);
        kvalid = kk < key_end;
        my_key = (int)kk;
        if (kvalid) {
            if (main_keys) {
                my_qend = p.meta.key_qend[kk];
                my_bq0 = p.meta.key_bq_begin[kk];
                my_bq1 = p.meta.key_bq_end[kk];
            } else {
                my_bq0 = p.meta.br_start[kk];
                my_bq1 = p.meta.br_end[kk];
            }
            if (warp < 4) {
                if (main_keys) atomicMax(&sm.qend_max, my_qend);
                atomicMin(&sm.bq0_min, my_bq0);
                atomicMax(&sm.bq1_max, my_bq1);
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = sm.tmem_base;

    // ---- query segments: main rows [m0, m1), branch tokens [b0, b1).  Sub-tiles
    // start at ma / ba: the segment starts moved back (by < 4 rows) so that every
    // sub-tile's first row is a multiple of 4 in the [N + M] row numbering; this
    // keeps the bulk copies of the per-row scalars 16-byte aligned.  The extra
    // leading rows are masked like any other invisible row.
    int64_t m0 = 0, m1 = 0, b0 = 0, b1 = 0;
    if (main_keys && p.has_main_q) {
        m0 = max(key0, p.r.qm_begin);
        m1 = min((int64_t)sm.qend_max, p.r.qm_end);
    }
    if (sm.bq1_max > sm.bq0_min) {
        b0 = max((int64_t)sm.bq0_min, p.r.tok_begin);
        b1 = min((int64_t)sm.bq1_max, p.r.tok_end);
    }
    const int64_t ma = m0 & ~(int64_t)3;
    const int64_t ba = ((n + b0) & ~(int64_t)3) - n;   // may be as low as -3
    const int n_sub_main = m1 > m0 ? (int)((m1 - ma + kSub - 1) / kSub) : 0;
    const int n_sub_br = b1 > b0 ? (int)((b1 - ba + kSub - 1) / kSub) : 0;
    const int n_sub = n_sub_main + n_sub_br;
    const int n_iter = n_sub * p.group;

    if (warp == 9) {
        // ================================================= producer (whole warp)
        if (n_iter > 0) {
            if (lane == 0) {
                mbar_expect_tx(&sm.kv_full, 2 * kTileBytes);
                for (int half = 0; half < 2; ++half) {
                    tma_load_3d(sm.k + half * 16384, &tm_k, half * 64, g, (int)gkey0, &sm.kv_full);
                    tma_load_3d(sm.v + half * 16384, &tm_v, half * 64, g, (int)gkey0, &sm.kv_full);
                }
            }
            bool ok = true;
            int issued = 0;
            int hh = 0, s = 0;  // t = hh * n_sub + s
            // the query stream comes from HBM: ask for sub-tile t + kPrefetch to be
            // brought into L2 while sub-tile t is loaded
            constexpr int kPrefetch = 16;
            int ph = 0, ps = 0;
            for (int i = 0; i < kPrefetch; ++i)
                if (++ps == n_sub) { ps = 0; ++ph; }
            for (int t = 0; t < n_iter; ++t) {
                const int st = t % kQStages;
                if (t >= kQStages) ok = mbar_wait(&sm.q_empty[st], ((t / kQStages) - 1) & 1, abort_flag);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                const int h = g * p.group + hh;
                const bool seg_main = s < n_sub_main;
                const int64_t r0 = seg_main ? ma + (int64_t)s * kSub : ba + (int64_t)(s - n_sub_main) * kSub;
                const int64_t grow0 = seg_main ? r0 : n + r0;
                SubMeta &mt = sm.meta[st];
                if (lane == 0) {
                    const CUtensorMap *tq = seg_main ? &tm_q_main : &tm_q_branch;
                    mbar_expect_tx(&sm.q_full[st], 2 * kSubBytes + 2 * kSub * 4);
                    for (int half = 0; half < 2; ++half) {
                        tma_load_3d(sm.qs[st] + half * 8192, tq, half * 64, h, (int)r0, &sm.q_full[st]);
                        tma_load_3d(sm.qs[st] + kSubBytes + half * 8192, &tm_go, half * 64, h, (int)grow0,
                                    &sm.q_full[st]);
                    }
                    const size_t off = (size_t)h * p.row_pitch + grow0;
                    bulk_load(mt.neg_lse2, p.nlse2_t + off, kSub * 4, &sm.q_full[st]);
                    bulk_load(mt.delta, p.delta_t + off, kSub * 4, &sm.q_full[st]);
                    if (t + kPrefetch < n_iter) {
                        const int h2 = g * p.group + ph;
                        const bool main2 = ps < n_sub_main;
                        const int64_t r2 = main2 ? ma + (int64_t)ps * kSub : ba + (int64_t)(ps - n_sub_main) * kSub;
                        const int64_t g2 = main2 ? r2 : n + r2;
                        const CUtensorMap *tq2 = main2 ? &tm_q_main : &tm_q_branch;
                        for (int half = 0; half < 2; ++half) {
                            tma_prefetch_3d(tq2, half * 64, h2, (int)r2);
                            tma_prefetch_3d(&tm_go, half * 64, h2, (int)g2);
                        }
                        const size_t off2 = (size_t)h2 * p.row_pitch + g2;
                        bulk_prefetch(p.nlse2_t + off2, kSub * 4);
                        bulk_prefetch(p.delta_t + off2, kSub * 4);
                    }
                }
                if (++ps == n_sub) { ps = 0; ++ph; }
                if (!main_keys) {
                    // own-branch tiles (rare, tiny): branch start and mask of each query token
                    for (int c = lane; c < kSub; c += 32) {
                        const int64_t tok = r0 + c;
                        const bool live = tok >= b0 && tok < b1;
                        mt.bstart[c] = live ? p.meta.br_start[tok] : 0;
                        mt.mask[c] = live ? p.meta.br_mask[tok] : 0ull;
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&sm.q_full[st]);  // second arrival: plain stores are in place
                issued = t + 1;
                if (++s == n_sub) { s = 0; ++hh; }
            }
            if (!ok && lane == 0) {
                for (int t = max(issued - kQStages, 0); t < issued; ++t) {
                    uint32_t spins = 0;
                    while (!mbar_try_wait(&sm.q_full[t % kQStages], (t / kQStages) & 1) && ++spins < (1u << 22)) {}
                }
                uint32_t spins = 0;
                while (!mbar_try_wait(&sm.kv_full, 0) && ++spins < (1u << 22)) {}
            }
        }
    } else if (warp == 8) {
        // ================================================= MMA issuer
        // the whole warp runs this code, an elected lane issues each MMA and commit
        if (n_iter > 0) {
            constexpr uint32_t IDESC_T = idesc_bf16(128, kSub, 0);   // 128 keys x 64 rows, K = d
            constexpr uint32_t IDESC_ACC = idesc_bf16(128, 128, 1);  // 128 keys x 128 d, K = 64 rows
            // low descriptor words (the issuing thread advances them with one add per MMA);
            // a stage holds the Q sub-tile, then the dO sub-tile, each two 64-column halves of 8 KB
            const uint32_t k_km = smem_desc_lo(smem_u32(sm.k), 16), v_km = smem_desc_lo(smem_u32(sm.v), 16);
            const uint32_t qs_km0 = smem_desc_lo(smem_u32(sm.qs[0]), 16), qs_mn0 = smem_desc_lo(smem_u32(sm.qs[0]), 8192);
            constexpr uint32_t kStageStep = (2 * kSubBytes) >> 4, kHalfStage = kSubBytes >> 4;
            auto issue_t = [&](uint32_t d_tmem, uint32_t a_km, uint32_t b_km) {
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)
                    if (elect_one()) mma_ss_lh(d_tmem, a_km + desc_step_kmajor(ks), b_km + (uint32_t)((ks >> 2) * 512 + (ks & 3) * 2),
                              IDESC_T, ks > 0);
            };
            auto issue_acc = [&](uint32_t d_tmem, uint32_t a_tmem, uint32_t b_mn, bool accumulate) {
#pragma unroll
                for (int ks = 0; ks < 4; ++ks)
                    if (elect_one()) mma_ts_lh(d_tmem, a_tmem + ks * 8, b_mn + desc_step_mnmajor(ks), IDESC_ACC, accumulate || ks > 0);
            };
            bool ok = __all_sync(0xffffffffu, mbar_wait(&sm.kv_full, 0, abort_flag));
            for (int b = 0; b < 2 && ok; ++b) {
                if (b >= n_iter) break;
                ok = __all_sync(0xffffffffu, mbar_wait(&sm.q_full[b], 0, abort_flag));
                if (!ok) break;
                tc_fence_after();
                issue_t(tmem + 256 + b * 128, k_km, qs_km0 + b * kStageStep);                    // S^T = K Q^T
                issue_t(tmem + 256 + b * 128 + 64, v_km, qs_km0 + b * kStageStep + kHalfStage);  // dP^T = V dO^T
                if (elect_one()) tc_commit(&sm.sd_full[b]);
            }
            for (int t = 0; t < n_iter && ok; ++t) {
                const int b = t & 1;
                const uint32_t stage_mn = qs_mn0 + (t % kQStages) * kStageStep;
                ok = __all_sync(0xffffffffu, mbar_wait(&sm.pd_done[b], (t >> 1) & 1, abort_flag));
                if (!ok) break;
                tc_fence_after();
                issue_acc(tmem + 128, tmem + 256 + b * 128, stage_mn + kHalfStage, t > 0);   // dV += P^T dO
                issue_acc(tmem + 0, tmem + 256 + b * 128 + 64, stage_mn, t > 0);             // dK += dS^T Q
                if (elect_one()) tc_commit(&sm.q_empty[t % kQStages]);
                const int t2 = t + 2;
                if (t2 < n_iter) {
                    const uint32_t next_km = qs_km0 + (t2 % kQStages) * kStageStep;
                    ok = __all_sync(0xffffffffu, mbar_wait(&sm.q_full[t2 % kQStages], (t2 / kQStages) & 1, abort_flag));
                    if (!ok) break;
                    tc_fence_after();
                    issue_t(tmem + 256 + b * 128, k_km, next_km);
                    issue_t(tmem + 256 + b * 128 + 64, v_km, next_km + kHalfStage);
                    if (elect_one()) tc_commit(&sm.sd_full[b]);
                }
            }
            if (ok) if (elect_one()) tc_commit(&sm.acc_full);
        }
    } else {
        // ================================================= P^T / dS^T warps + epilogue
        const int b = warp >> 2;
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t xs_addr = tmem + lane_base + 256 + b * 128;
        const uint32_t xd_addr = xs_addr + 64;
        const float sl2 = p.scale_log2;
        bool ok = true;
        for (int t = b; t < n_iter; t += 2) {
            const int st = t % kQStages;
            const int s = t % n_sub;
            const bool seg_main = s < n_sub_main;
            const int64_t r0 = seg_main ? ma + (int64_t)s * kSub : ba + (int64_t)(s - n_sub_main) * kSub;
            const int64_t rbeg = seg_main ? m0 : b0, rend = seg_main ? m1 : b1;
            const SubMeta &mt = sm.meta[st];
            // --- which of the 64 query rows (columns) see my key (needs only the
            // stage's scalars, so it runs while the MMAs are still in flight)
            ok = mbar_wait(&sm.q_full[st], (t / kQStages) & 1, abort_flag);
            if (!ok) break;
            uint64_t vis = 0ull;
            if (kvalid) {
                if (main_keys) {
                    if (seg_main)  // same sequence, causal: key <= row < end of the key's sequence
                        vis = bit_range((int)(max((int64_t)my_key, rbeg) - r0), (int)(min((int64_t)my_qend, rend) - 1 - r0));
                    else           // branch tokens anchored at or after the key, inside its sequence
                        vis = bit_range((int)(max((int64_t)my_bq0, rbeg) - r0), (int)(min((int64_t)my_bq1, rend) - 1 - r0));
                } else {
                    // own-branch tokens whose mask has my bit
                    const int lo_c = max((int)(max((int64_t)my_bq0, rbeg) - r0), 0);
                    const int hi_c = min((int)(min((int64_t)my_bq1, rend) - 1 - r0), kSub - 1);
                    for (int c = lo_c; c <= hi_c; ++c) {
                        const int rel = my_key - mt.bstart[c];
                        if (rel >= 0 && rel < 64 && ((mt.mask[c] >> rel) & 1ull)) vis |= 1ull << c;
                    }
                }
            }
            const bool masked = !__all_sync(0xffffffffu, vis == ~0ull);
            ok = mbar_wait(&sm.sd_full[b], (t >> 1) & 1, abort_flag);
            if (!ok) break;
            tc_fence_after();
            // --- P^T = exp2(scale_log2 S^T - lse2[col]), dS^T = P^T o (dP^T - delta[col]),
            // 16 columns at a time, the next pair of loads in flight behind the math
            {
                uint32_t sa[16], da[16], sb[16], db[16], pk[8], dk8[8];
                tmem_ld16(xs_addr, sa);
                tmem_ld16(xd_addr, da);
                tmem_ld16(xs_addr + 16, sb);
                tmem_ld16(xd_addr + 16, db);
                tmem_wait_ld();
                if (masked) {
                    quarter_pds<true>(sa, da, (uint32_t)vis & 0xffffu, sl2, mt.neg_lse2, mt.delta, pk, dk8);
                    tmem_st8(xs_addr, pk); tmem_st8(xd_addr, dk8);
                    tmem_ld16(xs_addr + 32, sa); tmem_ld16(xd_addr + 32, da);
                    quarter_pds<true>(sb, db, (uint32_t)(vis >> 16) & 0xffffu, sl2, mt.neg_lse2 + 16, mt.delta + 16, pk, dk8);
                    tmem_st8(xs_addr + 8, pk); tmem_st8(xd_addr + 8, dk8);
                    tmem_ld16(xs_addr + 48, sb); tmem_ld16(xd_addr + 48, db);
                    tmem_wait_ld();
                    quarter_pds<true>(sa, da, (uint32_t)(vis >> 32) & 0xffffu, sl2, mt.neg_lse2 + 32, mt.delta + 32, pk, dk8);
                    tmem_st8(xs_addr + 16, pk); tmem_st8(xd_addr + 16, dk8);
                    quarter_pds<true>(sb, db, (uint32_t)(vis >> 48) & 0xffffu, sl2, mt.neg_lse2 + 48, mt.delta + 48, pk, dk8);
                    tmem_st8(xs_addr + 24, pk); tmem_st8(xd_addr + 24, dk8);
                } else {
                    quarter_pds<false>(sa, da, 0u, sl2, mt.neg_lse2, mt.delta, pk, dk8);
                    tmem_st8(xs_addr, pk); tmem_st8(xd_addr, dk8);
                    tmem_ld16(xs_addr + 32, sa); tmem_ld16(xd_addr + 32, da);
                    quarter_pds<false>(sb, db, 0u, sl2, mt.neg_lse2 + 16, mt.delta + 16, pk, dk8);
                    tmem_st8(xs_addr + 8, pk); tmem_st8(xd_addr + 8, dk8);
                    tmem_ld16(xs_addr + 48, sb); tmem_ld16(xd_addr + 48, db);
                    tmem_wait_ld();
                    quarter_pds<false>(sa, da, 0u, sl2, mt.neg_lse2 + 32, mt.delta + 32, pk, dk8);
                    tmem_st8(xs_addr + 16, pk); tmem_st8(xd_addr + 16, dk8);
                    quarter_pds<false>(sb, db, 0u, sl2, mt.neg_lse2 + 48, mt.delta + 48, pk, dk8);
                    tmem_st8(xs_addr + 24, pk); tmem_st8(xd_addr + 24, dk8);
                }
            }
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(&sm.pd_done[b]);
        }
        // --- epilogue: warpgroup 0 writes dK (x scale), warpgroup 1 writes dV
        if (ok && n_iter > 0) ok = mbar_wait(&sm.acc_full, 0, abort_flag);
        tc_fence_after();
        const uint32_t acc_addr = tmem + lane_base + b * 128;
        void *dst = b == 0 ? p.dk : p.dv;
        const float mul = b == 0 ? p.scale : 1.0f;
        const size_t base = ((size_t)(gkey0 + (tid & 127)) * p.h_kv + g) * 128;
        const bool do_store = ok && kvalid;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            uint32_t r[32];
            if (n_iter > 0 && ok) {
                tmem_ld32(acc_addr + c * 32, r);
                tmem_wait_ld();
            } else {
#pragma unroll
                for (int e = 0; e < 32; ++e) r[e] = 0u;
            }
            if (do_store) {
                if (p.accumulate) store_grad_chunk<true>(dst, base + c * 32, r, mul);
                else store_grad_chunk<false>(dst, base + c * 32, r, mul);
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
              void *dq_main, void *dq_branch, void *dk, void *dv, cudaStream_t st, int stages) {
    // the dynamic shared-memory limit is a per-device attribute of the kernel
    static bool attr_set[64] = {};
    int dev = 0;
    BA_CUDA_CHECK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return BA_EUNSUPPORTED;
    const size_t dq_smem = sizeof(DqSmem) + 1024;
    const size_t kv_smem = sizeof(KvSmem) + 1024;
    if (!attr_set[dev]) {
        BA_CUDA_CHECK(cudaFuncSetAttribute(tc_dq_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dq_smem));
        BA_CUDA_CHECK(cudaFuncSetAttribute(tc_dkdv_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kv_smem));
        attr_set[dev] = true;
    }
    const ba_problem_t &pr = pl->prob;
    TcBwdParams p;
    memset(&p, 0, sizeof p);
    p.meta = pl->meta;
    p.r = r;
    (void)lse;
    p.delta_t = delta;
    p.nlse2_t = delta + (size_t)pl->row_pitch * pr.h_q;
    p.row_pitch = pl->row_pitch;
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

    if (p.total_tiles > 0 && (stages & BA_STAGE_DQ)) {
        const int64_t grid = (int64_t)p.total_tiles * pr.h_kv * p.pairs_per_group;
        if (grid > INT_MAX) return BA_EUNSUPPORTED;
        tc_dq_kernel<<<(unsigned)grid, kDqThreads, dq_smem, st>>>(tq_main, tq_branch, tgo, tk, tv, p);
        int rc = ba_check_launch();
        if (rc != BA_OK) return rc;
    }
    // dK / dV
    const int64_t kmt = (r.parts & BA_PART_MAIN) ? (r.kv_end - r.kv_begin + kTile - 1) / kTile : 0;
    const int64_t kbt = (r.parts & BA_PART_BRANCH) ? (r.tok_end - r.tok_begin + kTile - 1) / kTile : 0;
    p.main_key_tiles = (int)kmt;
    p.total_key_tiles = (int)(kmt + kbt);
    if (p.total_key_tiles > 0 && (stages & BA_STAGE_DKDV)) {
        CUtensorMap tq_main64, tq_branch64, tgo64;
        if (!make_tmap_rhd(&tq_main64, qm, qm_rows, pr.h_q, 128, kSub) ||
            !make_tmap_rhd(&tq_branch64, qb, qb_rows, pr.h_q, 128, kSub) ||
            !make_tmap_rhd(&tgo64, d_o, all_rows, pr.h_q, 128, kSub))
            return BA_EINVAL;
        const int64_t grid = (int64_t)p.total_key_tiles * pr.h_kv;
        if (grid > INT_MAX) return BA_EUNSUPPORTED;
        tc_dkdv_kernel<<<(unsigned)grid, kKvThreads, kv_smem, st>>>(tq_main64, tq_branch64, tgo64, tk, tv, p);
        int rc = ba_check_launch();
        if (rc != BA_OK) return rc;
    }
    return BA_OK;
}
