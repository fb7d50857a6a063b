// lora_bgmv_apply_static: the decode apply for callers that cannot provide (or allocate) a
// workspace.  The scratch array, the look-up of its device address and the entry point live in
// this one file; the kernels are the two-phase CUDA-core kernels of apply_twophase.cu, which
// receive the looked-up address like any other workspace pointer.
#include "apply_common.cuh"

// ---------------------------------------------------------------------------------------------
// Decode apply without a caller workspace: the fp32 partial products live in a fixed array that
// is part of the loaded library image.
// ---------------------------------------------------------------------------------------------
namespace lora {

constexpr size_t STATIC_SCRATCH_BYTES = LORA_STATIC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_static_scratch[STATIC_SCRATCH_BYTES];

constexpr int MAX_DEVICES = 64;
static void *g_scratch_addr[MAX_DEVICES];     // device address of the array, per device
static std::atomic<int> g_scratch_state[MAX_DEVICES];   // 0 = unknown, 1 = resolved

// The array's name is only a handle on the host; the address a kernel can use has to be asked
// for, with the device in question current.
static lora_status_t static_scratch_ptr(int device, void **out) {
    if (device < 0 || device >= MAX_DEVICES) return LORA_ERR_INVALID_ARG;
    if (g_scratch_state[device].load(std::memory_order_acquire) != 1) {
        void *p = nullptr;
        LORA_CUDA_TRY(cudaGetSymbolAddress(&p, g_static_scratch));
        if (!p) return cuda_fail(cudaErrorInvalidSymbol);
        g_scratch_addr[device] = p;
        g_scratch_state[device].store(1, std::memory_order_release);
    }
    *out = g_scratch_addr[device];
    return LORA_OK;
}

lora_status_t check_apply_args(lora_pool_t *pool, int32_t target, const void *x, int64_t ldx,
                               const void *yb, int64_t ldyb, void *y, int64_t ldy, int32_t T);
void fill_apply_params(lora_pool_t *pool, ApplyParams &P, int32_t target, const void *x,
                       int64_t ldx, const void *yb, int64_t ldyb, void *y, int64_t ldy,
                       const int32_t *slot_idx_dev, int32_t T, const void *meta, int32_t tile_m);
}  // namespace lora

extern "C" lora_status_t lora_bgmv_apply_static(lora_pool_t *pool, int32_t target, const void *x,
                                                int64_t ldx, const void *y_base, int64_t ldyb,
                                                void *y, int64_t ldy, const int32_t *slot_idx_dev,
                                                int32_t T, const void *meta, void *stream) {
    using namespace lora;
    lora_status_t s = check_apply_args(pool, target, x, ldx, y_base, ldyb, y, ldy, T);
    if (s != LORA_OK || T == 0) return s;
    if (!meta && !slot_idx_dev) return LORA_ERR_INVALID_ARG;
    // the full eight-way split of the shrink phase must fit: 8 * T * bucket(r_max) floats
    const size_t need = (size_t)8 * (size_t)T * rank_bucket(pool->r_max) * sizeof(float);
    if (need > STATIC_SCRATCH_BYTES) return LORA_ERR_BUFFER_TOO_SMALL;
    int32_t tile_m = 1;
    if (meta && !pool->find_meta(meta, T, &tile_m)) return LORA_ERR_INVALID_ARG;
    DeviceGuard guard(pool->device);
    if (!guard.ok) return cuda_fail(cudaErrorInvalidDevice);
    void *scratch = nullptr;
    if ((s = static_scratch_ptr(pool->device, &scratch)) != LORA_OK) return s;
    ApplyParams P;
    fill_apply_params(pool, P, target, x, ldx, y_base, ldyb, y, ldy, slot_idx_dev, T, meta, tile_m);
    // every partial the expand phase reads is written by this call's shrink phase first, so
    // nothing left in the array by an earlier call needs clearing
    return launch_twophase(pool, P, scratch, STATIC_SCRATCH_BYTES, (cudaStream_t)stream);
}
