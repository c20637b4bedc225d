// branch_attn_bwd_static: the backward pass for callers that cannot hand the
// library any scratch memory of their own.
//
// Some hosts of this library run where device allocation is off limits at call
// time -- inside a pre-planned memory arena, under a framework hook that forbids
// allocator calls, or late in a process whose pool is already carved up -- so
// they cannot obtain the few megabytes branch_attn_bwd needs for its per-row
// scalars (delta = <dO, O> and -LSE log2(e)).  For them the scratch lives here,
// in a fixed array inside the library image.  Every GPU that loads the library
// holds these BA_STATIC_SCRATCH_BYTES until the process exits, which is why the
// array is small and the entry point refuses problems that do not fit.
#include <mutex>

#include "ba_common.cuh"

namespace {

constexpr size_t kScratchFloats = BA_STATIC_SCRATCH_BYTES / sizeof(float);

// The scratch itself.  In host code this name is only a stand-in for the
// symbol, never a device address: the address is looked up once per device
// below and that pointer is what the kernels receive.
static __device__ __align__(256) float g_bwd_scratch[kScratchFloats];

constexpr int kMaxDevices = 64;
std::mutex g_setup_lock;
float *g_scratch_ptr[kMaxDevices] = {};

// First use on a device: resolve the device address of the array with that
// device current.  No allocation happens here or anywhere below.
int scratch_for_current_device(float **out) {
    int dev = -1;
    BA_CUDA_CHECK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return BA_EUNSUPPORTED;
    std::lock_guard<std::mutex> hold(g_setup_lock);
    if (!g_scratch_ptr[dev]) {
        void *ptr = nullptr;
        BA_CUDA_CHECK(cudaGetSymbolAddress(&ptr, g_bwd_scratch));
        if (!ptr) return BA_ECUDA;
        g_scratch_ptr[dev] = static_cast<float *>(ptr);
    }
    *out = g_scratch_ptr[dev];
    return BA_OK;
}

}  // namespace

extern "C" int branch_attn_bwd_static(const ba_plan_t *plan, const void *q_main, const void *q_branch,
                                      const void *k, const void *v, const void *O, const float *LSE,
                                      const void *dO, int64_t qm_begin, int64_t qm_end, int64_t br_begin,
                                      int64_t br_end, int64_t kv_begin, int64_t kv_end, int parts,
                                      int accumulate, void *dQ_main, void *dQ_branch, void *dK, void *dV,
                                      void *stream) {
    if (!plan) return BA_EINVAL;
    const size_t need = ba_workspace_bytes(plan, BA_OP_BWD);
    if (need > BA_STATIC_SCRATCH_BYTES) return BA_EWORKSPACE;  // problem too large for the built-in scratch
    float *scratch = nullptr;
    const int rc = scratch_for_current_device(&scratch);
    if (rc != BA_OK) return rc;
    // The kernels write every scratch entry they later read (the rows of the
    // selected query ranges) before reading it, so nothing has to be cleared
    // between calls even though the array keeps the previous call's contents.
    return branch_attn_bwd_stages(plan, q_main, q_branch, k, v, O, LSE, dO, qm_begin, qm_end, br_begin, br_end,
                                  kv_begin, kv_end, parts, accumulate, dQ_main, dQ_branch, dK, dV, scratch,
                                  BA_STATIC_SCRATCH_BYTES, stream, BA_STAGE_ALL);
}
