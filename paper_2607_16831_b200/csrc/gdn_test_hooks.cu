// Test-only entry points (see gdn_test_hooks.h).
#include "gdn_test_hooks.h"

#include "gdn_prefill_ws.cuh"
#include "gdn_sm100.cuh"

namespace gdn {
using namespace sm100;

__global__ void __launch_bounds__(128) gdn_test_bounded_wait_kernel(int* status_word, long long* elapsed,
                                                                    long long limit_cycles) {
    __shared__ uint64_t bars[2];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_word;
    volatile int* abort_flag = &abort_word;
    const int tid = threadIdx.x, warp = tid >> 5;
    if (tid == 0) {
        mbar_init(bars + 0, 1);  // nobody ever arrives at either barrier
        mbar_init(bars + 1, 1);
        abort_word = 0;
        mbar_fence_init();
    }
    if (warp == 0) {
        __syncwarp();
        tmem_alloc(&tmem_slot, 32);
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = tmem_slot;

    if (warp == 1) {
        // the wait that runs out: short limit, raises the abort flag
        const long long t0 = clock64();
        const bool ok = mbar_wait_all(bars + 0, 0, abort_flag, limit_cycles);
        if (tid == 32 && elapsed) *elapsed = ok ? -1 : clock64() - t0;
    } else if (warp >= 2) {
        // two more roles parked on a barrier of their own with the normal limit: they leave because
        // the flag was raised, not because their own limit ran out
        (void)mbar_wait_all(bars + 1, 0, abort_flag);
    }
    // ---- the unwind every prefill kernel ends with
    unwind_after_abort(abort_flag, status_word, kStatusTimeout);
    if (warp == 0) {
        __syncwarp();
        tmem_dealloc(tmem_base, 32);
    }
}

}  // namespace gdn

extern "C" int gdn_test_bounded_wait(int* status_word, long long* elapsed, long long limit_cycles, void* stream) {
    if (!status_word) return GDN_ERR_NULL;
    if (limit_cycles < 0 || limit_cycles > 2000000000LL) return GDN_ERR_SHAPE;
    gdn::gdn_test_bounded_wait_kernel<<<1, 128, 0, (cudaStream_t)stream>>>(status_word, elapsed, limit_cycles);
    return cudaGetLastError() == cudaSuccess ? GDN_OK : GDN_ERR_CUDA;
}
