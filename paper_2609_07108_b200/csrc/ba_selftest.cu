// Self-test of the bounded device-side wait: the path every tensor-core kernel
// takes when a barrier it waits on is never signalled (give up, raise the CTA's
// abort flag, report BA_ETIMEOUT through the plan's status word, return).  The
// kernels' own waits only run out after about two seconds of a stalled pipeline,
// which no healthy run produces; here one small CTA waits, with a short limit,
// on a barrier that by construction nobody arrives at.  No copy is in flight, no
// tensor memory is held, and the kernel returns normally.
#include "ba_common.cuh"
#include "ba_sm100.cuh"

namespace {

__global__ void __launch_bounds__(32, 1) bounded_wait_probe_kernel(long long limit_cycles, int *status) {
    __shared__ alignas(8) uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        sm100::mbar_init(&bar, 1);
        abort_flag = 0;
        sm100::fence_barrier_init();
    }
    __syncwarp();
    bool ok = true;
    if (threadIdx.x == 0) ok = sm100::mbar_wait(&bar, 0, &abort_flag, limit_cycles);   // nobody arrives
    __syncwarp();
    if (threadIdx.x == 0 && (!ok || abort_flag)) atomicExch(status, BA_ETIMEOUT);
}

}  // namespace

extern "C" int ba_selftest_bounded_wait(ba_plan_t *plan, int64_t limit_cycles, void *stream) {
    if (!plan) return BA_EINVAL;
    // a short limit only: this entry point exists to make the wait run out, not to stall a GPU
    if (limit_cycles < 1 || limit_cycles > 100000000ll) return BA_EINVAL;
    bounded_wait_probe_kernel<<<1, 32, 0, (cudaStream_t)stream>>>((long long)limit_cycles, plan->dev_status);
    return ba_check_launch();
}
