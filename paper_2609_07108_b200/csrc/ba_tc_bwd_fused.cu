// Tensor-core backward in ONE kernel (sm_100a, bf16, head_dim 128): dQ, dK, dV.
//
// Same mathematics as the split kernels (paper Section 3.2: gradients are
// accumulated over key chunks), but S and dP are formed once per (key tile,
// query tile, head) instead of once in a dQ kernel and once in a dK/dV kernel:
// 10 D flop per visible pair instead of 14 D.  The price: dQ rows are shared by
// all key tiles, so they are summed with fp32 atomic adds into an accumulator (the
// caller's in `accumulate` mode, one in the workspace otherwise) and their
// rounding depends on the arrival order; dK and dV still have one owning CTA and
// stay bit-reproducible.
//
// Key-stationary: one CTA owns 128 key rows of one KV head, keeps K_j, V_j in
// shared memory and dK_j, dV_j (fp32) in TMEM, and walks the query rows that can
// see those keys -- every query head of the KV head -- as 128-row tiles.  All
// tiles are transposed (TMEM lane = key, or head dimension for dQ):
//   S^T  = K_j Q^T,  dP^T = V_j dO^T                    (128 keys x 128 rows)
//   P^T  = exp2(scale_log2 S^T - lse2[col])             -> TMEM, bf16, over S^T
//   dS^T = P^T o (dP^T - delta[col])                    -> shared memory, bf16
//   dV_j += P^T dO,  dK_j += dS^T Q,  dQ^T = K_j^T dS^T (dS^T: A operand of one,
//                                                        B operand of the other)
//   TMEM: dK [0,128)  dV [128,256)  S^T / P^T [256,384)  X [384,512): dP^T, then dQ^T
// dQ^T (lane = head dimension, column = query row) is read back and added to the
// accumulator with one 128-byte reduction per warp and row.
//
// Warps 0-3 / 4-7 work on query columns [0,64) / [64,128) of every tile: A(t) P^T
// from S^T, then B(t) dS^T from dP^T.  Warps 8-11 read dQ^T out of X (R(t)) and
// issue the reductions, warp 13 runs the copies, one thread each of warps 12 and 14
// issues MMAs:  warp 12: dP(t) [after R(t-1)], dQ(t) dK(t) [after B(t)]
//               warp 14: dV(t) [after A(t)], S(t+1)
// The warpgroups re-split the register file (setmaxnreg) for their roles.
#include "ba_tc_bwd.cuh"

using namespace sm100;

namespace {

constexpr int kFusedThreads = 512;   // four warpgroups: P^T/dS^T (2), dQ^T readers, MMA + copies
// Registers per thread after the warpgroups re-split the register file.  The
// kernel starts with 128 each; what the increases take must have been given up
// by the decrease, or the increase waits forever.
constexpr int kRegsCompute = 152, kRegsReduce = 136, kRegsIssue = 72;
static_assert(2 * 128 * kRegsCompute + 128 * kRegsReduce + 128 * kRegsIssue <= kFusedThreads * 128,
              "register re-split exceeds what the CTA owns");

struct FusedSmem {
    alignas(1024) uint8_t k[kTileBytes];
    alignas(1024) uint8_t v[kTileBytes];
    alignas(1024) uint8_t q[2][kTileBytes];
    alignas(1024) uint8_t go[2][kTileBytes];
    alignas(1024) uint8_t ds[kTileBytes];     // dS^T: 128 keys x 128 rows, two 64-row halves
    alignas(16) float neg_lse2[2][kTile];
    alignas(16) float delta[2][kTile];
    alignas(8) uint64_t kv_full;
    uint64_t q_full[2], q_empty[2];
    uint64_t s_full, a_done, dp_full, b_done, dq_full, r_done, dk_done, acc_full;
    uint32_t tmem_base;
    int abort_flag;
    int qend_max, bq0_min, bq1_max;
};
static_assert(sizeof(FusedSmem) <= 232448, "shared memory of the fused backward kernel");

// P^T of 32 query columns: 2^(s * sl2 + nl[c]) as 16 packed bf16 pairs (invisible -> 0)
template <bool MASKED>
__device__ __forceinline__ void chunk_pt(const uint32_t (&r)[32], uint32_t mk, float sl2, const float *nl,
                                         uint32_t *pr) {
    const float2 s2 = make_float2(sl2, sl2);
    const float4 *nl4 = reinterpret_cast<const float4 *>(nl);
#pragma unroll
    for (int e = 0; e < 32; e += 4) {
        const float4 nv = nl4[e >> 2];
        const float2 x0 = ffma2(make_float2(__uint_as_float(r[e]), __uint_as_float(r[e + 1])), s2,
                                make_float2(nv.x, nv.y));
        const float2 x1 = ffma2(make_float2(__uint_as_float(r[e + 2]), __uint_as_float(r[e + 3])), s2,
                                make_float2(nv.z, nv.w));
        float p0 = ex2(x0.x), p1 = ex2(x0.y), p2 = ex2(x1.x), p3 = ex2(x1.y);
        if (MASKED) {  // the scalars of invisible columns may be anything, even NaN
            p0 = ((mk >> e) & 1u) ? p0 : 0.f;
            p1 = ((mk >> (e + 1)) & 1u) ? p1 : 0.f;
            p2 = ((mk >> (e + 2)) & 1u) ? p2 : 0.f;
            p3 = ((mk >> (e + 3)) & 1u) ? p3 : 0.f;
        }
        pr[e >> 1] = pack_bf16(p0, p1);
        pr[(e >> 1) + 1] = pack_bf16(p2, p3);
    }
}

// dS^T of 32 query columns: P o (dP - dl[c]) as 16 packed bf16 pairs (invisible -> 0)
template <bool MASKED>
__device__ __forceinline__ void chunk_dst(const uint32_t (&r)[32], const uint32_t *pr, uint32_t mk,
                                          const float4 *dl4, uint32_t (&pk)[16]) {
#pragma unroll
    for (int e = 0; e < 32; e += 4) {
        const float4 dv = dl4[e >> 2];
        const uint32_t pa = pr[e >> 1], pb = pr[(e >> 1) + 1];
        const float2 fa = make_float2(__uint_as_float(pa << 16), __uint_as_float(pa & 0xffff0000u));
        const float2 fb = make_float2(__uint_as_float(pb << 16), __uint_as_float(pb & 0xffff0000u));
        // dP - delta as one packed fma (delta * -1 + dP): no separate negations
        const float2 m1 = make_float2(-1.f, -1.f);
        float2 d0 = fmul2(fa, ffma2(make_float2(dv.x, dv.y), m1,
                                    make_float2(__uint_as_float(r[e]), __uint_as_float(r[e + 1]))));
        float2 d1 = fmul2(fb, ffma2(make_float2(dv.z, dv.w), m1,
                                    make_float2(__uint_as_float(r[e + 2]), __uint_as_float(r[e + 3]))));
        if (MASKED) {
            d0.x = ((mk >> e) & 1u) ? d0.x : 0.f;
            d0.y = ((mk >> (e + 1)) & 1u) ? d0.y : 0.f;
            d1.x = ((mk >> (e + 2)) & 1u) ? d1.x : 0.f;
            d1.y = ((mk >> (e + 3)) & 1u) ? d1.y : 0.f;
        }
        pk[e >> 1] = pack_bf16(d0.x, d0.y);
        pk[(e >> 1) + 1] = pack_bf16(d1.x, d1.y);
    }
}

__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
template <int N> __device__ __forceinline__ void reg_inc() {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N));
}
template <int N> __device__ __forceinline__ void reg_dec() {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N));
}
__device__ __forceinline__ void red_add_f32(float *ptr, float v) {
    asm volatile("red.global.add.f32 [%0], %1;" ::"l"(ptr), "f"(v) : "memory");
}
// the same, predicated inside the instruction: no branch, and `ptr` is not touched when `on` is false
__device__ __forceinline__ void red_add_f32_if(float *ptr, float v, bool on) {
    asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %2, 0;\n@p red.global.add.f32 [%0], %1;\n}\n"
                 ::"l"(ptr), "f"(v), "r"((int)on) : "memory");
}

__global__ void __launch_bounds__(kFusedThreads, 1)
tc_bwd_fused_kernel(const __grid_constant__ CUtensorMap tm_q_main, const __grid_constant__ CUtensorMap tm_q_branch,
                    const __grid_constant__ CUtensorMap tm_go, const __grid_constant__ CUtensorMap tm_k,
                    const __grid_constant__ CUtensorMap tm_v, const TcBwdParams p) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    FusedSmem &sm = *reinterpret_cast<FusedSmem *>(smem_raw);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    volatile int *abort_flag = &sm.abort_flag;
    if (smem_u32(smem_raw) & 1023u) {   // the swizzled tiles need 1024-byte alignment
        if (tid == 0) atomicExch(p.status, BA_EUNSUPPORTED);
        return;
    }

    // KV-head-major order: the CTAs resident at one time stream the same query rows
    const int g = (int)(blockIdx.x / p.total_key_tiles);
    const int tile = (int)(blockIdx.x % p.total_key_tiles);
    const bool main_keys = tile < p.main_key_tiles;
    const int64_t n = p.meta.n_main;
    // depth mode: branch key tile = (depth j + 1, 128 consecutive branches)
    const int btile = tile - p.main_key_tiles;
    const int kdepth = (p.depth && !main_keys) ? btile / p.branch_tiles_per_depth : 0;
    // first key of the tile: main key index, or branch token index (depth mode: branch index)
    const int64_t key0 = main_keys ? p.r.kv_begin + (int64_t)tile * kTile
                         : p.depth ? p.r.tok_begin + (int64_t)(btile % p.branch_tiles_per_depth) * kTile
                                   : p.r.tok_begin + (int64_t)btile * kTile;
    const int64_t key_end = main_keys ? p.r.kv_end : p.r.tok_end;
    const int64_t gkey0 = main_keys ? key0 : p.depth ? n + (int64_t)kdepth * p.num_branches + key0 : n + key0;
    // global row number of branch query 0 (rows of dO and of the per-row scalars): branch rows
    // follow the main rows, except in depth mode, where those tensors hold one row per branch
    const int64_t qbase = p.depth ? 0 : n;

    if (tid == 0) {
        mbar_init(&sm.kv_full, 1);
        for (int s = 0; s < 2; ++s) { mbar_init(&sm.q_full[s], 1); mbar_init(&sm.q_empty[s], 2); }
        mbar_init(&sm.s_full, 1);
        mbar_init(&sm.a_done, 256);
        mbar_init(&sm.dp_full, 1);
        mbar_init(&sm.b_done, 256);
        mbar_init(&sm.dq_full, 1);
        mbar_init(&sm.r_done, 128);
        mbar_init(&sm.dk_done, 1);
        mbar_init(&sm.acc_full, 2);
        sm.abort_flag = 0;
        sm.qend_max = -1; sm.bq0_min = INT_MAX; sm.bq1_max = -1;
        fence_barrier_init();
    }
    if (warp == 12) {
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
                if (p.depth) {   // token ranges -> branch ranges (every branch has branch_len tokens)
                    my_bq0 /= p.branch_len;
                    my_bq1 /= p.branch_len;
                }
            } else if (p.depth) {
                my_bq0 = (int)kk;          // seen by the query of its own branch only
                my_bq1 = (int)kk + 1;
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

    // ---- query segments: main rows [m0, m1), branch tokens [b0, b1).  Tiles start
    // at ma / ba: the segment starts moved back (by < 4 rows) so that every tile's
    // first row is a multiple of 4 in the [N + M] row numbering, which keeps the
    // bulk copies of the per-row scalars 16-byte aligned.  The extra leading rows
    // are masked like any other invisible row.
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
    const int64_t ba = ((qbase + b0) & ~(int64_t)3) - qbase;   // may be as low as -3
    const int n_sub_main = m1 > m0 ? (int)((m1 - ma + kTile - 1) / kTile) : 0;
    const int n_sub_br = b1 > b0 ? (int)((b1 - ba + kTile - 1) / kTile) : 0;
    const int n_sub = n_sub_main + n_sub_br;
    // t = head_in_group * n_sub + s, and step s works on tile n_sub - 1 - s: every key tile's query
    // range ends where its sequence (or the call's query range) ends, so CTAs that start together
    // walk the same tiles at the same time from that common end and share them through L2,
    // whereas their first tiles differ (causal: key tile k starts at row tile k)
    const int n_iter = n_sub * p.group;

    if (warp >= 12) {
      reg_dec<kRegsIssue>();
      if (warp == 13) {
        // ================================================= copies (one thread)
        if (lane == 0 && n_iter > 0) {
            mbar_expect_tx(&sm.kv_full, 2 * kTileBytes);
            for (int half = 0; half < 2; ++half) {
                tma_load_3d(sm.k + half * 16384, &tm_k, half * 64, g, (int)gkey0, &sm.kv_full);
                tma_load_3d(sm.v + half * 16384, &tm_v, half * 64, g, (int)gkey0, &sm.kv_full);
            }
            bool ok = true;
            int issued = 0;
            int hh = 0, s = 0;
            // the query stream comes from HBM: ask for tile t + kPrefetch to be brought
            // into L2 while tile t is loaded
            constexpr int kPrefetch = 8;
            int ph = 0, ps = 0;
            for (int i = 0; i < kPrefetch; ++i)
                if (++ps == n_sub) { ps = 0; ++ph; }
            for (int t = 0; t < n_iter; ++t) {
                const int st = t & 1;
                if (t >= 2) ok = mbar_wait(&sm.q_empty[st], ((t >> 1) - 1) & 1, abort_flag);
                if (!ok) break;
                const int h = g * p.group + hh;
                const int u = n_sub - 1 - s;   // tiles are walked from the last one down (see n_iter)
                const bool seg_main = u < n_sub_main;
                const int64_t r0 = seg_main ? ma + (int64_t)u * kTile : ba + (int64_t)(u - n_sub_main) * kTile;
                const int64_t grow0 = seg_main ? r0 : qbase + r0;
                const CUtensorMap *tq = seg_main ? &tm_q_main : &tm_q_branch;
                mbar_expect_tx(&sm.q_full[st], 2 * kTileBytes + 2 * kTile * 4);
                for (int half = 0; half < 2; ++half) {
                    tma_load_3d(sm.q[st] + half * 16384, tq, half * 64, h, (int)r0, &sm.q_full[st]);
                    tma_load_3d(sm.go[st] + half * 16384, &tm_go, half * 64, h, (int)grow0, &sm.q_full[st]);
                }
                const size_t off = (size_t)h * p.row_pitch + grow0;
                bulk_load(sm.neg_lse2[st], p.nlse2_t + off, kTile * 4, &sm.q_full[st]);
                bulk_load(sm.delta[st], p.delta_t + off, kTile * 4, &sm.q_full[st]);
                issued = t + 1;
                if (t + kPrefetch < n_iter) {
                    const int h2 = g * p.group + ph;
                    const int u2 = n_sub - 1 - ps;
                    const bool main2 = u2 < n_sub_main;
                    const int64_t r2 = main2 ? ma + (int64_t)u2 * kTile : ba + (int64_t)(u2 - n_sub_main) * kTile;
                    const int64_t g2 = main2 ? r2 : qbase + r2;
                    const CUtensorMap *tq2 = main2 ? &tm_q_main : &tm_q_branch;
                    for (int half = 0; half < 2; ++half) {
                        tma_prefetch_3d(tq2, half * 64, h2, (int)r2);
                        tma_prefetch_3d(&tm_go, half * 64, h2, (int)g2);
                    }
                    const size_t off2 = (size_t)h2 * p.row_pitch + g2;
                    bulk_prefetch(p.nlse2_t + off2, kTile * 4);
                    bulk_prefetch(p.delta_t + off2, kTile * 4);
                }
                if (++ps == n_sub) { ps = 0; ++ph; }
                if (++s == n_sub) { s = 0; ++hh; }
            }
            if (!ok) {
                // leave no copy in flight behind: wait (bounded) for what was issued
                for (int t = max(issued - 2, 0); t < issued; ++t) {
                    uint32_t spins = 0;
                    while (!mbar_try_wait(&sm.q_full[t & 1], (t >> 1) & 1) && ++spins < (1u << 22)) {}
                }
                uint32_t spins = 0;
                while (!mbar_try_wait(&sm.kv_full, 0) && ++spins < (1u << 22)) {}
            }
        }
      } else if (warp == 12 || warp == 14) {
        // ================================================= MMA issuers
        // Two issuing threads with independent streams, because one thread cannot feed the
        // tensor core here: a tcgen05.mma costs its thread about 53 clocks on an idle SM (a
        // 128x128x16 MMA runs 64) and several times that while the other warps of its
        // scheduler are busy.
        //   warp 12: dP^T(t) [after R(t-1)], dQ^T(t) and dK(t) [after B(t)]   -- X, dK
        //   warp 14: dV(t) [after A(t)], S^T(t+1)                             -- S^T / P^T, dV
        // No order is needed between the two streams; each keeps its own order by issuing
        // from one thread.  A Q / dO stage is released by both (q_empty counts 2).
        // The whole warp runs the code and an elected lane issues each MMA and commit: with
        // warp-uniform control flow the descriptors stay in uniform registers, which halves
        // the cost of a tcgen05.mma for its thread.
        if (n_iter > 0) {
            constexpr uint32_t IDESC_T = idesc_bf16_full(128, 128, 0, 0);    // S^T, dP^T: both operands K-major
            constexpr uint32_t IDESC_ACC = idesc_bf16_full(128, 128, 0, 1);  // dV, dK: B = dO / Q rows, MN-major
            constexpr uint32_t IDESC_DQ = idesc_bf16_full(128, 128, 1, 1);   // dQ^T: A = K_j rows, B = dS^T rows
            // low descriptor words of every operand tile; stage st of Q / dO is 2048 units further
            const uint32_t k_km = smem_desc_lo(smem_u32(sm.k), 16), k_mn = smem_desc_lo(smem_u32(sm.k), 16384);
            const uint32_t v_km = smem_desc_lo(smem_u32(sm.v), 16);
            const uint32_t ds_km = smem_desc_lo(smem_u32(sm.ds), 16), ds_mn = smem_desc_lo(smem_u32(sm.ds), 16384);
            const uint32_t q_km0 = smem_desc_lo(smem_u32(sm.q[0]), 16), q_mn0 = smem_desc_lo(smem_u32(sm.q[0]), 16384);
            const uint32_t go_km0 = smem_desc_lo(smem_u32(sm.go[0]), 16), go_mn0 = smem_desc_lo(smem_u32(sm.go[0]), 16384);
            constexpr uint32_t kStageStep = kTileBytes >> 4;
            const uint32_t t_dk = tmem, t_dv = tmem + 128, t_s = tmem + 256, t_x = tmem + 384;
            // D[128 x 128] = A B^T, A and B tiles of 128 rows x 128 bf16 (K = the 128 columns)
            auto issue_t = [&](uint32_t d_tmem, uint32_t a_km, uint32_t b_km) {
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)
                    if (elect_one()) mma_ss_lh(d_tmem, a_km + desc_step_kmajor(ks), b_km + desc_step_kmajor(ks), IDESC_T, ks > 0);
            };
            // every lane waits (and all agree on the outcome, so the warp stays converged)
            auto wait = [&](uint64_t *bar, uint32_t parity) {
                return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag));
            };
            bool ok = wait(&sm.kv_full, 0);
            ok = ok && wait(&sm.q_full[0], 0);
            if (warp == 12) {
                if (ok) {
                    tc_fence_after();
                    issue_t(t_x, v_km, go_km0);  if (elect_one()) tc_commit(&sm.dp_full);   // dP^T(0)
                }
                for (int t = 0; t < n_iter && ok; ++t) {
                    const int st = t & 1;
                    const uint32_t q_mn = q_mn0 + st * kStageStep, go_km = go_km0 + st * kStageStep;
                    // --- dP^T(t) into X once dQ^T(t-1) has been read out of it
                    if (t > 0) {
                        ok = wait(&sm.r_done, (t - 1) & 1);
                        if (ok) ok = wait(&sm.q_full[st], (t >> 1) & 1);
                        if (!ok) break;
                        tc_fence_after();
                        issue_t(t_x, v_km, go_km);
                        if (elect_one()) tc_commit(&sm.dp_full);
                    }
                    // --- dQ^T(t) = K_j^T dS^T into X, dK += dS^T Q
                    ok = wait(&sm.b_done, t & 1);
                    if (!ok) break;
                    tc_fence_after();
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks)
                        if (elect_one()) mma_ss_lh(t_x, k_mn + desc_step_mnmajor(ks), ds_mn + desc_step_mnmajor(ks), IDESC_DQ, ks > 0);
                    if (elect_one()) tc_commit(&sm.dq_full);
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks)
                        if (elect_one()) mma_ss_lh(t_dk, ds_km + desc_step_kmajor(ks), q_mn + desc_step_mnmajor(ks), IDESC_ACC,
                                  t > 0 || ks > 0);
                    if (elect_one()) tc_commit(&sm.dk_done);
                    if (elect_one()) tc_commit(&sm.q_empty[st]);
                }
            } else {
                if (ok) {
                    tc_fence_after();
                    issue_t(t_s, k_km, q_km0);   if (elect_one()) tc_commit(&sm.s_full);    // S^T(0)
                }
                for (int t = 0; t < n_iter && ok; ++t) {
                    const int st = t & 1;
                    const uint32_t go_mn = go_mn0 + st * kStageStep, q_km_next = q_km0 + (st ^ 1) * kStageStep;
                    // --- dV += P^T dO  (P^T: bf16 pairs in columns [0,32) and [64,96) of the S^T region)
                    ok = wait(&sm.a_done, t & 1);
                    if (!ok) break;
                    tc_fence_after();
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks)
                        if (elect_one()) mma_ts_lh(t_dv, t_s + (ks >> 2) * 64 + (ks & 3) * 8, go_mn + desc_step_mnmajor(ks), IDESC_ACC,
                                  t > 0 || ks > 0);
                    if (elect_one()) tc_commit(&sm.q_empty[st]);
                    // --- S^T(t+1): P^T(t) is consumed by the dV MMAs queued above
                    if (t + 1 < n_iter) {
                        ok = wait(&sm.q_full[st ^ 1], ((t + 1) >> 1) & 1);
                        if (!ok) break;
                        tc_fence_after();
                        issue_t(t_s, k_km, q_km_next);
                        if (elect_one()) tc_commit(&sm.s_full);
                    }
                }
            }
            if (ok) if (elect_one()) tc_commit(&sm.acc_full);
        }
      }
    } else if (warp >= 8) {
        // ================================================= dQ^T readers (warps 8-11)
        // X -> registers (which frees X for the next dP^T), then one reduction per
        // query row and warp: 32 lanes = 32 consecutive floats of the row.  These
        // warps stall on the reductions when the L2 is busy; nothing waits for them.
        reg_inc<kRegsReduce>();
        const int dlane = tid & 127;                    // my TMEM lane: head dimension of dQ^T
        const uint32_t x_addr = tmem + ((uint32_t)((warp & 3) * 32) << 16) + 384;
        const size_t row_stride = (size_t)p.h_q * 128;
        const float sc = p.scale;
        int s = 0, hh = 0;                              // tile t = hh * n_sub + s
        for (int t = 0; t < n_iter; ++t) {
            const int u = n_sub - 1 - s;
            const bool seg_main = u < n_sub_main;
            const int r0 = seg_main ? (int)ma + u * kTile : (int)ba + (u - n_sub_main) * kTile;   // first query row
            const int rbeg = seg_main ? (int)m0 : (int)b0, rend = seg_main ? (int)m1 : (int)b1;
            const int c_lo = max(rbeg - r0, 0), c_hi = min(rend - r0, kTile);
            float *ptr = (float *)(seg_main ? p.dq_main : p.dq_branch) +
                         ((ptrdiff_t)r0 * p.h_q + (g * p.group + hh)) * 128 + dlane;
            if (!mbar_wait(&sm.dq_full, t & 1, abort_flag)) break;
            tc_fence_after();
            uint32_t r[4][32];
#pragma unroll
            for (int q4 = 0; q4 < 4; ++q4) tmem_ld32(x_addr + 32 * q4, r[q4]);
            tmem_wait_ld();
            tc_fence_before();
            mbar_arrive(&sm.r_done);
            // the pointer advances row by row (kept opaque so that 128 addresses are not formed ahead)
            if (c_lo == 0 && c_hi == kTile) {
#pragma unroll
                for (int q4 = 0; q4 < 4; ++q4)
#pragma unroll
                    for (int e = 0; e < 32; ++e) {
                        red_add_f32(ptr, __uint_as_float(r[q4][e]) * sc);
                        ptr += row_stride;
                        asm volatile("" : "+l"(ptr));
                    }
            } else {
#pragma unroll
                for (int q4 = 0; q4 < 4; ++q4)
#pragma unroll
                    for (int e = 0; e < 32; ++e) {
                        const int c = 32 * q4 + e;
                        red_add_f32_if(ptr, __uint_as_float(r[q4][e]) * sc, c >= c_lo && c < c_hi);
                        ptr += row_stride;
                        asm volatile("" : "+l"(ptr));
                    }
            }
            if (++s == n_sub) { s = 0; ++hh; }
        }
    } else {
        // ================================================= P^T / dS^T warps + epilogue (warps 0-7)
        reg_inc<kRegsCompute>();
        const int hf = warp >> 2;                       // my 64 query columns of every tile
        const int krow = tid & 127;                     // my TMEM lane: key (head dimension for dQ^T)
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t s_addr = tmem + lane_base + 256 + 64 * hf;   // my S^T columns; P^T goes over the first 32
        const uint32_t x_addr = tmem + lane_base + 384 + 64 * hf;   // my dP^T / dQ^T columns
        // my row of the dS^T tile: 128 bytes in half hf, 16-byte chunks swizzled by the row
        const uint32_t ds_row = smem_u32(sm.ds) + hf * 16384 + krow * 128;
        const uint32_t ds_xor = (uint32_t)(krow & 7);
        const float sl2 = p.scale_log2;
        bool ok = true;

        uint32_t pr[32];   // P^T of my 64 columns, bf16 pairs, kept from phase A to phase B
        int s = 0, hh = 0;                       // tile t = hh * n_sub + s
        const int ma_i = (int)ma + 64 * hf, ba_i = (int)ba + 64 * hf;
        for (int t = 0; t < n_iter; ++t) {
            const int st = t & 1;
            const int u = n_sub - 1 - s;
            const bool seg_main = u < n_sub_main;
            const int r0h = seg_main ? ma_i + u * kTile : ba_i + (u - n_sub_main) * kTile;   // my first query row
            const int rbeg = seg_main ? (int)m0 : (int)b0, rend = seg_main ? (int)m1 : (int)b1;
            // --- which of my 64 query rows (columns) see my key
            uint64_t vis = 0ull;
            if (kvalid) {
                if (main_keys) {
                    if (seg_main)  // same sequence, causal: key <= row < end of the key's sequence
                        vis = bit_range(max(my_key, rbeg) - r0h, min(my_qend, rend) - 1 - r0h);
                    else           // branch tokens anchored at or after the key, inside its sequence
                        vis = bit_range(max(my_bq0, rbeg) - r0h, min(my_bq1, rend) - 1 - r0h);
                } else if (p.depth) {
                    // my key is token (kdepth + 1) of branch my_key: seen by that branch's query
                    if (my_key >= rbeg && my_key < rend) vis = bit_range(my_key - r0h, my_key - r0h);
                } else {
                    // own-branch tokens whose mask has my bit (few, short tiles)
                    const int lo_c = max(max(my_bq0, rbeg) - r0h, 0);
                    const int hi_c = min(min(my_bq1, rend) - 1 - r0h, 63);
                    for (int c = lo_c; c <= hi_c; ++c) {
                        const int rel = my_key - p.meta.br_start[r0h + c];
                        if (rel >= 0 && rel < 64 && ((p.meta.br_mask[r0h + c] >> rel) & 1ull)) vis |= 1ull << c;
                    }
                }
            }
            const bool masked = !__all_sync(0xffffffffu, vis == ~0ull);
            const uint32_t mk0 = (uint32_t)vis, mk1 = (uint32_t)(vis >> 32);
            ok = mbar_wait(&sm.q_full[st], (t >> 1) & 1, abort_flag);   // the tile's scalars
            if (!ok) break;
            const float *nl = sm.neg_lse2[st] + 64 * hf, *dl = sm.delta[st] + 64 * hf;

            // --- phase A: P^T = exp2(scale_log2 S^T - lse2[col]) -> TMEM (bf16) and registers
            ok = mbar_wait(&sm.s_full, t & 1, abort_flag);
            if (!ok) break;
            tc_fence_after();
            {
                uint32_t ra[32], rb[32];
                tmem_ld32(s_addr, ra);
                tmem_ld32(s_addr + 32, rb);
                tmem_wait_ld();
                if (masked) {
                    chunk_pt<true>(ra, mk0, sl2, nl, &pr[0]);
                    chunk_pt<true>(rb, mk1, sl2, nl + 32, &pr[16]);
                } else {
                    chunk_pt<false>(ra, 0u, sl2, nl, &pr[0]);
                    chunk_pt<false>(rb, 0u, sl2, nl + 32, &pr[16]);
                }
                tmem_st32(s_addr, pr);
            }
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(&sm.a_done);
            // delta of my first 32 columns goes into registers while this warp would wait anyway
            // (phase B is on the critical chain and its shared-memory loads queue behind the SS MMAs)
            float4 d0[8];
#pragma unroll
            for (int i4 = 0; i4 < 8; ++i4) d0[i4] = reinterpret_cast<const float4 *>(dl)[i4];

            // --- phase B: dS^T = P^T o (dP^T - delta[col]) -> shared memory (bf16)
            ok = mbar_wait(&sm.dp_full, t & 1, abort_flag);
            if (ok && t > 0) ok = mbar_wait(&sm.dk_done, (t - 1) & 1, abort_flag);   // dS^T(t-1) no longer read
            if (!ok) break;
            tc_fence_after();
            {
                uint32_t ra[32], rb[32], pk[16];
                tmem_ld32(x_addr, ra);
                tmem_ld32(x_addr + 32, rb);
                tmem_wait_ld();
                if (masked) chunk_dst<true>(ra, &pr[0], mk0, d0, pk);
                else chunk_dst<false>(ra, &pr[0], 0u, d0, pk);
#pragma unroll
                for (int ch = 0; ch < 4; ++ch)
                    st_shared_v4(ds_row + (((uint32_t)ch ^ ds_xor) << 4), pk[4 * ch], pk[4 * ch + 1], pk[4 * ch + 2],
                                 pk[4 * ch + 3]);
                if (masked) chunk_dst<true>(rb, &pr[16], mk1, reinterpret_cast<const float4 *>(dl + 32), pk);
                else chunk_dst<false>(rb, &pr[16], 0u, reinterpret_cast<const float4 *>(dl + 32), pk);
#pragma unroll
                for (int ch = 0; ch < 4; ++ch)
                    st_shared_v4(ds_row + (((uint32_t)(ch + 4) ^ ds_xor) << 4), pk[4 * ch], pk[4 * ch + 1],
                                 pk[4 * ch + 2], pk[4 * ch + 3]);
            }
            fence_proxy_async();   // the MMAs read dS^T through the async proxy
            tc_fence_before();
            mbar_arrive(&sm.b_done);
            if (++s == n_sub) { s = 0; ++hh; }
        }
        // --- epilogue: warpgroup 0 writes dK (x scale), warpgroup 1 writes dV
        if (ok && n_iter > 0) ok = mbar_wait(&sm.acc_full, 0, abort_flag);
        tc_fence_after();
        const uint32_t acc_addr = tmem + lane_base + hf * 128;
        void *dst = hf == 0 ? p.dk : p.dv;
        const float mul = hf == 0 ? p.scale : 1.0f;
        const size_t base = ((size_t)(gkey0 + krow) * p.h_kv + g) * 128;
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
    if (warp == 12) tmem_dealloc(tmem, 512);
    if (tid == 0 && sm.abort_flag) atomicExch(p.status, BA_ETIMEOUT);
}

}  // namespace

int ba_tc_bwd_fused(const ba_plan *pl, const BaRange &r, const void *q_main, const void *q_branch, const void *k,
                    const void *v, const float *delta, const void *d_o, int accumulate, void *dq_main,
                    void *dq_branch, void *dk, void *dv, cudaStream_t st, int depth) {
    // dq_main / dq_branch are always fp32 accumulators (summed with atomic adds);
    // `accumulate` says whether dK / dV are fp32 accumulators too or written in bf16
    // the dynamic shared-memory limit is a per-device attribute of the kernel
    static bool attr_set[64] = {};
    int dev = 0;
    BA_CUDA_CHECK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return BA_EUNSUPPORTED;
    const size_t smem = sizeof(FusedSmem);
    if (!attr_set[dev]) {
        // The register re-split inside the kernel hands out what a launch with 128 registers per
        // thread owns.  A build that gave the kernel fewer (another compiler, a register cap, a debug
        // build) would leave setmaxnreg.inc waiting for registers nobody releases: refuse to launch.
        cudaFuncAttributes fa;
        BA_CUDA_CHECK(cudaFuncGetAttributes(&fa, tc_bwd_fused_kernel));
        if (fa.numRegs * kFusedThreads < 2 * 128 * kRegsCompute + 128 * kRegsReduce + 128 * kRegsIssue)
            return BA_EUNSUPPORTED;
        BA_CUDA_CHECK(cudaFuncSetAttribute(tc_bwd_fused_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        attr_set[dev] = true;
    }
    const ba_problem_t &pr = pl->prob;
    TcBwdParams p;
    memset(&p, 0, sizeof p);
    p.meta = pl->meta;
    p.r = r;
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
    const int64_t kmt = (r.parts & BA_PART_MAIN) ? (r.kv_end - r.kv_begin + kTile - 1) / kTile : 0;
    int64_t kbt = (r.parts & BA_PART_BRANCH) ? (r.tok_end - r.tok_begin + kTile - 1) / kTile : 0;
    p.depth = depth;
    p.num_branches = pr.num_branches;
    p.branch_len = pr.uniform_len;
    p.branch_tiles_per_depth = (int)kbt;
    if (depth) kbt *= depth;    // the tokens of depths 1 .. depth of the selected branches are keys
    p.main_key_tiles = (int)kmt;
    p.total_key_tiles = (int)(kmt + kbt);
    if (p.total_key_tiles == 0) return BA_OK;

    CUtensorMap tq_main, tq_branch, tgo, tk, tv;
    // depth mode: key rows of depths <= depth only (later rows read as zero); dO holds one row per branch
    const uint64_t all_rows = (uint64_t)(pr.n_main + pr.n_branch);
    const uint64_t kv_rows = depth ? (uint64_t)(pr.n_main + (int64_t)depth * pr.num_branches) : all_rows;
    const uint64_t go_rows = depth ? (uint64_t)pr.num_branches : all_rows;
    if (!make_tmap_rhd(&tk, k, kv_rows, pr.h_kv, 128, kTile) || !make_tmap_rhd(&tv, v, kv_rows, pr.h_kv, 128, kTile) ||
        !make_tmap_rhd(&tgo, d_o, go_rows, pr.h_q, 128, kTile))
        return BA_EINVAL;
    const void *qm = q_main ? q_main : q_branch;
    const void *qb = (q_branch && pr.n_branch > 0) ? q_branch : q_main;
    const uint64_t qm_rows = depth ? (uint64_t)pr.num_branches : q_main ? (uint64_t)pr.n_main : (uint64_t)pr.n_branch;
    uint64_t qb_rows = (q_branch && pr.n_branch > 0) ? (uint64_t)pr.n_branch : (uint64_t)pr.n_main;
    if (depth) qb_rows = (uint64_t)pr.num_branches;
    if (!make_tmap_rhd(&tq_main, qm, qm_rows, pr.h_q, 128, kTile) ||
        !make_tmap_rhd(&tq_branch, qb, qb_rows, pr.h_q, 128, kTile))
        return BA_EINVAL;
    const int64_t grid = (int64_t)p.total_key_tiles * pr.h_kv;
    if (grid > INT_MAX) return BA_EUNSUPPORTED;
    tc_bwd_fused_kernel<<<(unsigned)grid, kFusedThreads, smem, st>>>(tq_main, tq_branch, tgo, tk, tv, p);
    return ba_check_launch();
}
