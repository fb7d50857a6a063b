// Self-test of the device-side time-out path, and the synchronous status check.
//
// Every wait inside the library's kernels is a bounded poll of an mbarrier; a wait that runs out
// bumps the pool's status word 1 and the block leaves without storing results.  That branch cannot
// be reached by valid inputs, so a one-block kernel whose barrier nobody ever completes stands in
// for it: same barrier type, same poll instruction, same bookkeeping, a small poll limit.
#include "common.cuh"

namespace lora {

__global__ void __launch_bounds__(32)
wait_expiry_kernel(int32_t *status, uint32_t polls, int32_t *witness) {
    __shared__ __align__(8) uint64_t bar;
    const uint32_t addr = (uint32_t)__cvta_generic_to_shared(&bar);
    if (threadIdx.x == 0) {
        // one arrival expected, none will come
        asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(addr), "r"(1u) : "memory");
    }
    __syncthreads();
    if (threadIdx.x != 0) return;
    bool done = false;
    for (uint32_t i = 0; i < polls && !done; ++i) {
        uint32_t ok;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(ok)
            : "r"(addr), "r"(0u)
            : "memory");
        done = ok != 0;
    }
    if (!done) {
        atomicAdd(&status[STATUS_TIMEOUTS], 1);   // what every kernel of the library does on expiry
        return;                                   // and no result is stored
    }
    if (witness) *witness = 1;   // only reached if the wait had succeeded
}

}  // namespace lora

using namespace lora;

extern "C" {

lora_status_t lora_pool_selftest_wait_expiry(lora_pool_t *pool, int32_t polls, int32_t *witness_dev,
                                             void *stream) {
    if (!pool || polls < 1 || polls > (1 << 20)) return LORA_ERR_INVALID_ARG;
    DeviceGuard guard(pool->device);
    if (!guard.ok) return cuda_fail(cudaErrorInvalidDevice);
    wait_expiry_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(pool->status_dev, (uint32_t)polls, witness_dev);
    return count_launch();
}

lora_status_t lora_pool_check_status(lora_pool_t *pool, void *stream, int32_t *words_out) {
    if (!pool) return LORA_ERR_INVALID_ARG;
    DeviceGuard guard(pool->device);
    if (!guard.ok) return cuda_fail(cudaErrorInvalidDevice);
    int32_t w[STATUS_WORDS] = {0, 0, 0, 0};
    LORA_CUDA_TRY(cudaMemcpyAsync(w, pool->status_dev, sizeof(w), cudaMemcpyDeviceToHost,
                                  (cudaStream_t)stream));
    LORA_CUDA_TRY(cudaStreamSynchronize((cudaStream_t)stream));
    if (words_out)
        for (int i = 0; i < STATUS_WORDS; ++i) words_out[i] = w[i];
    return w[STATUS_TIMEOUTS] != 0 ? LORA_ERR_TIMEOUT : LORA_OK;
}

}  // extern "C"
