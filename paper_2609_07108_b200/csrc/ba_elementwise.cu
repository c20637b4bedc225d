// HBM-bound elementwise kernels: Eq. (lse-merge), the backward preprocess
// delta = rowsum(dO * O), and the fp32 -> output-dtype conversion of gradient
// accumulators.  All are grid-stride, 16-byte vectorised, one pass over memory.
#include "ba_common.cuh"

namespace {

constexpr int kThreads = 256;
constexpr int kBlocksPerSm = 8;
constexpr int kSms = 148;

inline int stream_grid(int64_t work_items) {
    int64_t g = (work_items + kThreads - 1) / kThreads;
    const int64_t cap = (int64_t)kSms * kBlocksPerSm;
    if (g > cap) g = cap;
    if (g < 1) g = 1;
    return (int)g;
}

__device__ __forceinline__ uint2 pack_bf16x4(float4 x) {
    __nv_bfloat162 lo = __floats2bfloat162_rn(x.x, x.y);
    __nv_bfloat162 hi = __floats2bfloat162_rn(x.z, x.w);
    uint2 r;
    r.x = *reinterpret_cast<uint32_t *>(&lo);
    r.y = *reinterpret_cast<uint32_t *>(&hi);
    return r;
}

// Eq. (lse-merge) in max-subtracted form.  LPI = lanes per (row, head) item,
// each lane owning one float4 of the d-vector; all lanes of an item sit in one
// warp so that in-place updates (O_out == O_a, LSE_out == LSE_a) are safe.
template <int LPI, bool OUT_BF16>
__global__ void __launch_bounds__(kThreads)
lse_merge_kernel(int64_t items, const float4 *oa, const float *lse_a,   // may alias o_out / lse_out: no __restrict__
                 const float4 *__restrict__ ob, const float *__restrict__ lse_b,
                 void *o_out, float *lse_out) {
    constexpr int IPW = 32 / LPI;  // items per warp
    const int lane = threadIdx.x & 31;
    const int sub = lane % LPI;
    const int64_t warp = ((int64_t)blockIdx.x * kThreads + threadIdx.x) >> 5;
    const int64_t warps = ((int64_t)gridDim.x * kThreads) >> 5;
    for (int64_t base = warp * IPW; base < items; base += warps * IPW) {
        const int64_t i = base + lane / LPI;
        const bool live = i < items;
        float la = -INFINITY, lb = -INFINITY;
        float4 a = make_float4(0.f, 0.f, 0.f, 0.f), b = a;
        if (live) {
            la = lse_a[i];
            lb = lse_b[i];
            a = oa[i * LPI + sub];
            b = ob[i * LPI + sub];
        }
        __syncwarp();
        const float m = fmaxf(la, lb);
        float wa = 0.f, wb = 0.f, l = -INFINITY;
        if (m != -INFINITY) {
            const float ea = expf(la - m), eb = expf(lb - m);
            const float s = ea + eb;
            l = m + logf(s);
            const float inv = 1.0f / s;
            wa = ea * inv;
            wb = eb * inv;
        }
        if (live) {
            float4 r;
            r.x = wa * a.x + wb * b.x;
            r.y = wa * a.y + wb * b.y;
            r.z = wa * a.z + wb * b.z;
            r.w = wa * a.w + wb * b.w;
            if (OUT_BF16)
                reinterpret_cast<uint2 *>(o_out)[i * LPI + sub] = pack_bf16x4(r);
            else
                reinterpret_cast<float4 *>(o_out)[i * LPI + sub] = r;
            if (sub == 0 && lse_out) lse_out[i] = l;
        }
    }
}

template <bool OUT_BF16>
int launch_merge(int lpi, int64_t items, const float *oa, const float *la, const float *ob,
                 const float *lb, void *oo, float *lo, cudaStream_t st) {
    const int grid = stream_grid(items * lpi);
#define BA_MERGE_CASE(L)                                                                          \
    case L:                                                                                       \
        lse_merge_kernel<L, OUT_BF16><<<grid, kThreads, 0, st>>>(                                 \
            items, (const float4 *)oa, la, (const float4 *)ob, lb, oo, lo);                       \
        break;
    switch (lpi) {
        BA_MERGE_CASE(1) BA_MERGE_CASE(2) BA_MERGE_CASE(4) BA_MERGE_CASE(8) BA_MERGE_CASE(16)
        BA_MERGE_CASE(32)
        default: return BA_EUNSUPPORTED;
    }
#undef BA_MERGE_CASE
    return ba_check_launch();
}

// delta_t[h, r] = sum_d dO[r, h, d] * O[r, h, d] and nlse2_t[h, r] = -LSE[r, h] log2(e),
// both head-major with `pitch` rows per head; one 16-byte chunk per lane.  The rows are
// two segments handled by one launch: [row_a, row_a + items_a / h_q), then rows from row_b
// (the main query rows and the branch rows of one call).
template <typename T, int LPI>
__global__ void __launch_bounds__(kThreads)
delta_kernel(int64_t items, int64_t items_a, const uint4 *__restrict__ o, const uint4 *__restrict__ d_o,
             const float *__restrict__ lse, float *__restrict__ delta_t, float *__restrict__ nlse2_t,
             int64_t row_a, int64_t row_b, int h_q, int64_t pitch) {
    constexpr int IPW = 32 / LPI;
    const int lane = threadIdx.x & 31;
    const int sub = lane % LPI;
    const int64_t warp = ((int64_t)blockIdx.x * kThreads + threadIdx.x) >> 5;
    const int64_t warps = ((int64_t)gridDim.x * kThreads) >> 5;
    for (int64_t base = warp * IPW; base < items; base += warps * IPW) {
        const int64_t i = base + lane / LPI;
        float acc = 0.f;
        int64_t r = 0;
        int h = 0;
        if (i < items) {
            const int64_t j = i < items_a ? i : i - items_a;
            r = (i < items_a ? row_a : row_b) + j / h_q;
            h = (int)(j % h_q);
            const int64_t e = (r * h_q + h) * LPI + sub;
            const uint4 x = o[e], y = d_o[e];
            if (sizeof(T) == 4) {
                const float *xf = reinterpret_cast<const float *>(&x);
                const float *yf = reinterpret_cast<const float *>(&y);
#pragma unroll
                for (int c = 0; c < 4; ++c) acc += xf[c] * yf[c];
            } else {
                const __nv_bfloat162 *xb = reinterpret_cast<const __nv_bfloat162 *>(&x);
                const __nv_bfloat162 *yb = reinterpret_cast<const __nv_bfloat162 *>(&y);
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const float2 xf = __bfloat1622float2(xb[c]), yf = __bfloat1622float2(yb[c]);
                    acc += xf.x * yf.x + xf.y * yf.y;
                }
            }
        }
#pragma unroll
        for (int off = LPI / 2; off; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
        if (i < items && sub == 0) {
            delta_t[h * pitch + r] = acc;
            nlse2_t[h * pitch + r] = -lse[r * h_q + h] * 1.4426950408889634f;
        }
    }
}

template <bool OUT_BF16>
__global__ void __launch_bounds__(kThreads)
finalize_kernel(int64_t chunks, int64_t count, const float *__restrict__ src, void *dst) {
    const int64_t stride = (int64_t)gridDim.x * kThreads;
    for (int64_t c = (int64_t)blockIdx.x * kThreads + threadIdx.x; c < chunks; c += stride) {
        const int64_t e = c * 4;
        if (e + 4 <= count) {
            const float4 x = *reinterpret_cast<const float4 *>(src + e);
            if (OUT_BF16)
                *reinterpret_cast<uint2 *>((__nv_bfloat16 *)dst + e) = pack_bf16x4(x);
            else
                *reinterpret_cast<float4 *>((float *)dst + e) = x;
        } else {
            for (int64_t j = e; j < count; ++j) {
                if (OUT_BF16) ((__nv_bfloat16 *)dst)[j] = __float2bfloat16_rn(src[j]);
                else ((float *)dst)[j] = src[j];
            }
        }
    }
}

}  // namespace

extern "C" int lse_merge(int64_t rows_heads, int d, const float *O_a, const float *LSE_a,
                         const float *O_b, const float *LSE_b, void *O_out, int out_dtype,
                         float *LSE_out, void *stream) {
    if (rows_heads < 0 || d <= 0) return BA_EINVAL;
    if (rows_heads == 0) return BA_OK;
    if (!O_a || !O_b || !LSE_a || !LSE_b || !O_out) return BA_EINVAL;
    if (d % 4 != 0 || 32 % (d / 4) != 0) return BA_EUNSUPPORTED;
    if (out_dtype != BA_FP32 && out_dtype != BA_BF16) return BA_EUNSUPPORTED;
    if (((uintptr_t)O_a | (uintptr_t)O_b | (uintptr_t)O_out) & 15) return BA_EINVAL;
    if (out_dtype == BA_BF16 && O_out == (const void *)O_a) return BA_EINVAL;
    cudaStream_t st = (cudaStream_t)stream;
    if (out_dtype == BA_BF16)
        return launch_merge<true>(d / 4, rows_heads, O_a, LSE_a, O_b, LSE_b, O_out, LSE_out, st);
    return launch_merge<false>(d / 4, rows_heads, O_a, LSE_a, O_b, LSE_b, O_out, LSE_out, st);
}

int ba_delta(const void *o, const void *d_o, const float *lse, float *delta_t, float *nlse2_t,
             int64_t row_pitch, int64_t row_a_begin, int64_t row_a_end, int64_t row_b_begin,
             int64_t row_b_end, int h_q, int d, int dtype, cudaStream_t st) {
    const int64_t items_a = row_a_end > row_a_begin ? (row_a_end - row_a_begin) * h_q : 0;
    const int64_t items_b = row_b_end > row_b_begin ? (row_b_end - row_b_begin) * h_q : 0;
    const int64_t items = items_a + items_b;
    if (items <= 0) return BA_OK;
    const size_t esz = dtype == BA_FP32 ? 4 : 2;
    const uint4 *op = (const uint4 *)o, *gp = (const uint4 *)d_o;
    const int lpi = (int)(d * esz / 16);
    const int grid = stream_grid(items * lpi);
#define BA_DELTA_LAUNCH(T, L)                                                                            \
    delta_kernel<T, L><<<grid, kThreads, 0, st>>>(items, items_a, op, gp, lse, delta_t, nlse2_t,        \
                                                  row_a_begin, row_b_begin, h_q, row_pitch)
    if (dtype == BA_FP32 && lpi == 16) BA_DELTA_LAUNCH(float, 16);
    else if (dtype == BA_FP32 && lpi == 32) BA_DELTA_LAUNCH(float, 32);
    else if (dtype == BA_BF16 && lpi == 8) BA_DELTA_LAUNCH(__nv_bfloat16, 8);
    else if (dtype == BA_BF16 && lpi == 16) BA_DELTA_LAUNCH(__nv_bfloat16, 16);
    else return BA_EUNSUPPORTED;
#undef BA_DELTA_LAUNCH
    return ba_check_launch();
}

extern "C" int ba_finalize_grads(const float *src, void *dst, int64_t count, int dst_dtype,
                                 void *stream) {
    if (count < 0) return BA_EINVAL;
    if (count == 0) return BA_OK;
    if (!src || !dst) return BA_EINVAL;
    if (dst_dtype != BA_FP32 && dst_dtype != BA_BF16) return BA_EUNSUPPORTED;
    if (((uintptr_t)src | (uintptr_t)dst) & 15) return BA_EINVAL;
    const int64_t chunks = (count + 3) / 4;
    const int grid = stream_grid(chunks);
    cudaStream_t st = (cudaStream_t)stream;
    if (dst_dtype == BA_BF16)
        finalize_kernel<true><<<grid, kThreads, 0, st>>>(chunks, count, src, dst);
    else
        finalize_kernel<false><<<grid, kThreads, 0, st>>>(chunks, count, src, dst);
    return ba_check_launch();
}
