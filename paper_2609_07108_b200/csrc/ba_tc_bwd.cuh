// Pieces shared by the tensor-core backward kernels (ba_tc_bwd.cu: split dQ and
// dK/dV kernels; ba_tc_bwd_fused.cu: one key-stationary kernel for all three).
#pragma once

#include <limits.h>
#include <string.h>

#include "ba_common.cuh"
#include "ba_sm100.cuh"

namespace {

constexpr int kTile = 128;
constexpr uint32_t kTileBytes = 32768;   // 128 rows x 128 bf16
constexpr float kLog2e = 1.4426950408889634f;

// bits [lo, hi] of a 64-bit word (empty if lo > hi)
__device__ __forceinline__ uint64_t bit_range(int lo, int hi) {
    lo = max(lo, 0);
    hi = min(hi, 63);
    if (lo > hi) return 0ull;
    return (~0ull >> (63 - hi)) & (~0ull << lo);
}

struct TcBwdParams {
    BaMeta meta;
    BaRange r;
    const float *nlse2_t, *delta_t;   // head-major [h_q, row_pitch]: -LSE log2(e), delta
    int64_t row_pitch;
    void *dq_main, *dq_branch, *dk, *dv;
    int h_q, h_kv, group, pairs_per_group;
    float scale, scale_log2;
    int accumulate;
    int has_main_q;
    int main_tiles, total_tiles;      // dQ kernel: query row tiles
    int main_key_tiles, total_key_tiles;  // dK/dV and fused kernels: key tiles
    // Step-major (per-depth) call of the one-kernel backward: depth > 0.  Query rows are the
    // depth-`depth` tokens of branches [r.tok_begin, r.tok_end) (branch indices), Q / dO / dQ and
    // the per-row scalars are indexed by branch, and branch keys are stored depth-major after the
    // main rows: token (depth j + 1, branch b) is key row N + j * num_branches + b.
    int depth, num_branches, branch_len, branch_tiles_per_depth;
    int *status;
};

// one 32-column chunk of a gradient row: fp32 accumulate (dst += r * mul) or bf16 store
template <bool ACC_F32>
__device__ __forceinline__ void store_grad_chunk(void *dst, size_t elem_off, const uint32_t (&r)[32], float mul) {
    using sm100::pack_bf16;
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

}  // namespace
