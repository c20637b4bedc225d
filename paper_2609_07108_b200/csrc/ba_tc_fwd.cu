// Tensor-core (tcgen05) forward: placeholder until the kernels land.
#include "ba_common.cuh"

bool ba_tc_supported(const ba_problem_t *) { return false; }

int ba_tc_fwd(const ba_plan *, const BaRange &, const void *, const void *, const void *, const void *,
              void *, float *, bool, cudaStream_t) {
    return BA_EUNSUPPORTED;
}

int ba_tc_bwd(const ba_plan *, const BaRange &, const void *, const void *, const void *, const void *,
              const float *, const float *, const void *, int, void *, void *, void *, void *,
              cudaStream_t) {
    return BA_EUNSUPPORTED;
}
