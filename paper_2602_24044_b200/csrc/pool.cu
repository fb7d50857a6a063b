// Slot pool: A_max preallocated slots of uniform footprint S_max (paper Section 2.2), and the
// side-stream swap-in of an adapter from pinned CPU memory (the adapter-cache stage of paper
// Section 5 whose cost Eq. 1 calls Lat_load).
#include <new>

#include "apply_common.cuh"

namespace lora {

thread_local int32_t g_last_cuda_error = 0;
std::atomic<int64_t> g_launch_count{0};

static inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

struct PoolLayout {
    size_t off_status, off_table, off_maps, off_staging, off_weights, bytes;
    size_t staging_elems;
    int64_t slot_stride;   // elements
};

static lora_status_t validate_desc(const lora_pool_desc_t *d) {
    if (!d || !d->targets) return LORA_ERR_INVALID_ARG;
    if (d->num_slots < 1 || d->num_slots > 8192 || d->num_targets < 1) return LORA_ERR_INVALID_ARG;
    if (d->r_max < 1 || d->r_max > 64) return LORA_ERR_RANK;
    for (int32_t p = 0; p < d->num_targets; ++p) {
        const lora_target_t &t = d->targets[p];
        if (t.d_in < 8 || t.d_out < 8 || (t.d_in % 8) || (t.d_out % 8)) return LORA_ERR_SHAPE;
    }
    return LORA_OK;
}

static PoolLayout pool_layout(const lora_pool_desc_t *d) {
    PoolLayout L;
    int64_t per_rank = 0;
    int32_t max_d_in = 0;
    for (int32_t p = 0; p < d->num_targets; ++p) {
        per_rank += (int64_t)d->targets[p].d_in + d->targets[p].d_out;
        if (d->targets[p].d_in > max_d_in) max_d_in = d->targets[p].d_in;
    }
    L.slot_stride = per_rank * d->r_max;
    L.staging_elems = (size_t)max_d_in * d->r_max;
    L.off_status = 0;
    L.off_table = 256;
    L.off_maps = align_up(L.off_table + sizeof(SlotEntry) * (size_t)d->num_slots, 256);
    L.off_staging = align_up(L.off_maps + (size_t)d->num_targets * 16 * sizeof(CUtensorMap), 256);
    L.off_weights = align_up(L.off_staging + L.staging_elems * 2, 256);
    // 256 bytes of slack after the last slot: tiled loads of 64-column blocks may start inside
    // the last row of the last matrix and run up to 126 bytes past its end
    L.bytes = L.off_weights + (size_t)L.slot_stride * 2 * (size_t)d->num_slots + 256;
    return L;
}

__global__ void set_slot_kernel(SlotEntry *table, int32_t slot, int32_t rank, float scale,
                                int32_t loaded) {
    if (threadIdx.x == 0 && blockIdx.x == 0) {
        SlotEntry e;
        e.rank = rank;
        e.scale = scale;
        e.loaded = loaded;
        e.reserved = 0;
        table[slot] = e;
    }
}

// in: [d_in, r] row-major (the formula's A); out: [r8, d_in] row-major, rows r..r8-1 zero
// (r8 = the slot's row capacity).
__global__ void transpose_a_kernel(const __nv_bfloat16 *__restrict__ in,
                                   __nv_bfloat16 *__restrict__ out, int32_t d_in, int32_t r,
                                   int32_t r8) {
    const int32_t d = blockIdx.x * blockDim.x + threadIdx.x;
    if (d >= d_in) return;
    const __nv_bfloat16 zero = __float2bfloat16(0.0f);
    for (int32_t k = 0; k < r8; ++k)
        out[(int64_t)k * d_in + d] = k < r ? in[(int64_t)d * r + k] : zero;
}

static bool is_pinned(const void *p) {
    cudaPointerAttributes a;
    cudaError_t e = cudaPointerGetAttributes(&a, p);
    if (e != cudaSuccess) {
        cudaGetLastError();
        return false;
    }
    return a.type == cudaMemoryTypeHost || a.type == cudaMemoryTypeManaged;
}

static lora_status_t fence_load_after_compute(lora_pool_t *pool, cudaStream_t load,
                                              cudaStream_t compute, bool have_compute) {
    if (!have_compute || load == compute) return LORA_OK;
    LORA_CUDA_TRY(cudaEventRecord(pool->fence, compute));
    LORA_CUDA_TRY(cudaStreamWaitEvent(load, pool->fence, 0));
    return LORA_OK;
}

struct CopyJob {
    char *dst;
    const char *src;
    size_t bytes;
};

}  // namespace lora

using namespace lora;

extern "C" {

lora_status_t lora_pool_bytes(const lora_pool_desc_t *desc, size_t *bytes) {
    if (!bytes) return LORA_ERR_INVALID_ARG;
    lora_status_t s = validate_desc(desc);
    if (s != LORA_OK) return s;
    *bytes = pool_layout(desc).bytes;
    return LORA_OK;
}

static void release_sync_objects(lora_pool_t *p) {
    if (p->fence) cudaEventDestroy(p->fence);
    if (p->ev_fork) cudaEventDestroy(p->ev_fork);
    if (p->ev_join) cudaEventDestroy(p->ev_join);
    if (p->side_stream) cudaStreamDestroy(p->side_stream);
    p->fence = p->ev_fork = p->ev_join = nullptr;
    p->side_stream = nullptr;
}

lora_status_t lora_pool_create(const lora_pool_desc_t *desc, lora_pool_t **out) {
    if (!out) return LORA_ERR_INVALID_ARG;
    *out = nullptr;
    lora_status_t s = validate_desc(desc);
    if (s != LORA_OK) return s;
    if (!desc->device_buf || ((uintptr_t)desc->device_buf & 255)) return LORA_ERR_INVALID_ARG;
    PoolLayout L = pool_layout(desc);
    if (desc->device_buf_bytes < L.bytes) return LORA_ERR_BUFFER_TOO_SMALL;

    DeviceGuard guard(desc->device);
    if (!guard.ok) return cuda_fail(cudaErrorInvalidDevice);
    lora_pool_t *p = new (std::nothrow) lora_pool();
    if (!p) return LORA_ERR_INVALID_ARG;
    p->device = desc->device;
    p->num_slots = desc->num_slots;
    p->r_max = desc->r_max;
    p->num_targets = desc->num_targets;
    p->targets.assign(desc->targets, desc->targets + desc->num_targets);
    p->base = (char *)desc->device_buf;
    p->bytes = L.bytes;
    p->status_dev = (int32_t *)(p->base + L.off_status);
    p->table_dev = (SlotEntry *)(p->base + L.off_table);
    p->maps_dev = (CUtensorMap *)(p->base + L.off_maps);
    p->staging_dev = (__nv_bfloat16 *)(p->base + L.off_staging);
    p->staging_elems = L.staging_elems;
    p->weights_dev = (__nv_bfloat16 *)(p->base + L.off_weights);
    p->slot_stride = L.slot_stride;
    int64_t off = 0;
    for (int32_t t = 0; t < p->num_targets; ++t) {
        TargetView tv;
        tv.d_in = p->targets[t].d_in;
        tv.d_out = p->targets[t].d_out;
        tv.off_a = off;
        off += (int64_t)p->r_max * tv.d_in;
        tv.off_b = off;
        off += (int64_t)p->r_max * tv.d_out;
        p->target_views.push_back(tv);
    }
    SlotEntry empty = {0, 0.0f, 0, 0};
    p->table_host.assign(p->num_slots, empty);
    p->ready.assign(p->num_slots, nullptr);
    cudaError_t e = cudaEventCreateWithFlags(&p->fence, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&p->ev_fork, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&p->ev_join, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&p->side_stream, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaMemset(p->base, 0, L.off_staging);   // status, table, tensor maps
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&p->sm_count, cudaDevAttrMultiProcessorCount,
                                                     desc->device);
    if (e != cudaSuccess) {
        release_sync_objects(p);
        delete p;
        return cuda_fail(e);
    }
    if ((s = build_fused_maps(p)) != LORA_OK) {
        release_sync_objects(p);
        delete p;
        return s;
    }
    *out = p;
    return LORA_OK;
}

lora_status_t lora_pool_destroy(lora_pool_t *pool) {
    if (!pool) return LORA_ERR_INVALID_ARG;
    DeviceGuard guard(pool->device);
    for (cudaEvent_t ev : pool->ready)
        if (ev) cudaEventDestroy(ev);
    release_sync_objects(pool);
    delete pool;
    return LORA_OK;
}

lora_status_t lora_pool_load_slot(lora_pool_t *pool, int32_t slot, const lora_adapter_host_t *ad,
                                  void *load_stream, void *compute_stream) {
    if (!pool || !ad || !ad->A || !ad->B) return LORA_ERR_INVALID_ARG;
    if (slot < 0 || slot >= pool->num_slots) return LORA_ERR_SLOT_RANGE;
    if (ad->rank < 1 || ad->rank > pool->r_max) return LORA_ERR_RANK;
    if (ad->a_layout != LORA_A_DIN_MAJOR && ad->a_layout != LORA_A_RANK_MAJOR &&
        ad->a_layout != LORA_PACKED)
        return LORA_ERR_INVALID_ARG;
    const bool packed = ad->a_layout == LORA_PACKED;
    // packed: A[0] is one buffer with every target's A [rank, d_in] and B [rank, d_out] in order
    std::vector<const char *> srcA(pool->num_targets), srcB(pool->num_targets);
    if (packed) {
        if (!ad->A[0] || ((uintptr_t)ad->A[0] & 15)) return LORA_ERR_INVALID_ARG;
        const char *p = (const char *)ad->A[0];
        for (int32_t t = 0; t < pool->num_targets; ++t) {
            srcA[t] = p;  p += (size_t)ad->rank * pool->targets[t].d_in * 2;
            srcB[t] = p;  p += (size_t)ad->rank * pool->targets[t].d_out * 2;
        }
    } else {
        for (int32_t t = 0; t < pool->num_targets; ++t) {
            if (!ad->A[t] || !ad->B[t]) return LORA_ERR_INVALID_ARG;
            if (((uintptr_t)ad->A[t] | (uintptr_t)ad->B[t]) & 1) return LORA_ERR_INVALID_ARG;
            srcA[t] = (const char *)ad->A[t];
            srcB[t] = (const char *)ad->B[t];
        }
    }
    DeviceGuard guard(pool->device);
    if (!guard.ok) return cuda_fail(cudaErrorInvalidDevice);
    if (!ad->trust_pinned) {
        if (packed) {
            if (!is_pinned(srcA[0]) || !is_pinned(srcB[pool->num_targets - 1])) return LORA_ERR_NOT_PINNED;
        } else {
            for (int32_t t = 0; t < pool->num_targets; ++t)
                if (!is_pinned(ad->A[t]) || !is_pinned(ad->B[t])) return LORA_ERR_NOT_PINNED;
        }
    }

    cudaStream_t ls = (cudaStream_t)load_stream, cs = (cudaStream_t)compute_stream;
    if (!pool->ready[slot])
        LORA_CUDA_TRY(cudaEventCreateWithFlags(&pool->ready[slot], cudaEventDisableTiming));
    lora_status_t s = fence_load_after_compute(pool, ls, cs, compute_stream != nullptr);
    if (s != LORA_OK) return s;

    const int32_t r = ad->rank, r8 = pool->r_max;   // padding rows r .. r_max-1 are zeroed
    __nv_bfloat16 *slot_base = pool->weights_dev + (int64_t)slot * pool->slot_stride;

    set_slot_kernel<<<1, 32, 0, ls>>>(pool->table_dev, slot, 0, 0.0f, 0);
    if ((s = count_launch()) != LORA_OK) return s;
    // from here on the slot is empty on the device; the host's view follows until the load is
    // queued completely (an error on the way leaves both sides saying "empty")
    pool->table_host[slot] = {0, 0.0f, 0, 0};

    // One DMA per matrix.  Neighbouring host matrices given as separate pointers are not merged
    // into one copy: two pinned allocations can be adjacent in the address space, and a copy must
    // not span both.  A caller that holds the adapter in one buffer says so with LORA_PACKED.
    std::vector<CopyJob> jobs;
    auto push = [&jobs](void *dst, const void *src, size_t bytes) {
        jobs.push_back({(char *)dst, (const char *)src, bytes});
    };
    if (packed && r == r8) {
        // a full-rank packed adapter has exactly the slot's layout: one DMA for the whole adapter
        push(slot_base, srcA[0], (size_t)pool->slot_stride * 2);
    } else {
        for (int32_t t = 0; t < pool->num_targets; ++t) {
            const TargetView &tv = pool->target_views[t];
            if (ad->a_layout != LORA_A_DIN_MAJOR)
                push(slot_base + tv.off_a, srcA[t], (size_t)r * tv.d_in * 2);
            push(slot_base + tv.off_b, srcB[t], (size_t)r * tv.d_out * 2);
        }
    }
    for (const CopyJob &j : jobs)
        LORA_CUDA_TRY(cudaMemcpyAsync(j.dst, j.src, j.bytes, cudaMemcpyHostToDevice, ls));

    for (int32_t t = 0; t < pool->num_targets; ++t) {
        const TargetView &tv = pool->target_views[t];
        __nv_bfloat16 *dA = slot_base + tv.off_a, *dB = slot_base + tv.off_b;
        if (ad->a_layout == LORA_A_DIN_MAJOR) {
            LORA_CUDA_TRY(cudaMemcpyAsync(pool->staging_dev, srcA[t], (size_t)r * tv.d_in * 2,
                                          cudaMemcpyHostToDevice, ls));
            transpose_a_kernel<<<(tv.d_in + 255) / 256, 256, 0, ls>>>(pool->staging_dev, dA,
                                                                      tv.d_in, r, r8);
            if ((s = count_launch()) != LORA_OK) return s;
        } else if (r8 > r) {
            LORA_CUDA_TRY(cudaMemsetAsync(dA + (int64_t)r * tv.d_in, 0,
                                          (size_t)(r8 - r) * tv.d_in * 2, ls));
        }
        if (r8 > r)
            LORA_CUDA_TRY(cudaMemsetAsync(dB + (int64_t)r * tv.d_out, 0,
                                          (size_t)(r8 - r) * tv.d_out * 2, ls));
    }
    set_slot_kernel<<<1, 32, 0, ls>>>(pool->table_dev, slot, r, ad->scale, 1);
    if ((s = count_launch()) != LORA_OK) return s;
    LORA_CUDA_TRY(cudaEventRecord(pool->ready[slot], ls));
    const int32_t rb = rank_bucket(r);
    pool->bucket_mask |= rb == 8 ? 1u : rb == 16 ? 2u : rb == 32 ? 4u : 8u;
    pool->table_host[slot].rank = r;
    pool->table_host[slot].scale = ad->scale;
    pool->table_host[slot].loaded = 1;
    return LORA_OK;
}

lora_status_t lora_pool_evict_slot(lora_pool_t *pool, int32_t slot, void *load_stream,
                                   void *compute_stream) {
    if (!pool) return LORA_ERR_INVALID_ARG;
    if (slot < 0 || slot >= pool->num_slots) return LORA_ERR_SLOT_RANGE;
    DeviceGuard guard(pool->device);
    if (!guard.ok) return cuda_fail(cudaErrorInvalidDevice);
    cudaStream_t ls = (cudaStream_t)load_stream, cs = (cudaStream_t)compute_stream;
    lora_status_t s = fence_load_after_compute(pool, ls, cs, compute_stream != nullptr);
    if (s != LORA_OK) return s;
    set_slot_kernel<<<1, 32, 0, ls>>>(pool->table_dev, slot, 0, 0.0f, 0);
    if ((s = count_launch()) != LORA_OK) return s;
    if (pool->ready[slot]) LORA_CUDA_TRY(cudaEventRecord(pool->ready[slot], ls));
    pool->table_host[slot] = {0, 0.0f, 0, 0};
    return LORA_OK;
}

lora_status_t lora_pool_acquire(lora_pool_t *pool, const int32_t *slots_host, int32_t n,
                                void *compute_stream) {
    if (!pool || (n > 0 && !slots_host) || n < 0) return LORA_ERR_INVALID_ARG;
    for (int32_t i = 0; i < n; ++i)
        if (slots_host[i] < 0 || slots_host[i] >= pool->num_slots) return LORA_ERR_SLOT_RANGE;
    DeviceGuard guard(pool->device);
    if (!guard.ok) return cuda_fail(cudaErrorInvalidDevice);
    for (int32_t i = 0; i < n; ++i) {
        cudaEvent_t ev = pool->ready[slots_host[i]];
        if (ev) LORA_CUDA_TRY(cudaStreamWaitEvent((cudaStream_t)compute_stream, ev, 0));
    }
    return LORA_OK;
}

lora_status_t lora_pool_read_slot(lora_pool_t *pool, int32_t slot, int32_t target, void *A_host,
                                  void *B_host, void *stream) {
    if (!pool) return LORA_ERR_INVALID_ARG;
    if (slot < 0 || slot >= pool->num_slots || target < 0 || target >= pool->num_targets)
        return LORA_ERR_SLOT_RANGE;
    DeviceGuard guard(pool->device);
    if (!guard.ok) return cuda_fail(cudaErrorInvalidDevice);
    const TargetView &tv = pool->target_views[target];
    const __nv_bfloat16 *sb = pool->weights_dev + (int64_t)slot * pool->slot_stride;
    if (A_host)
        LORA_CUDA_TRY(cudaMemcpyAsync(A_host, sb + tv.off_a, (size_t)pool->r_max * tv.d_in * 2,
                                      cudaMemcpyDeviceToHost, (cudaStream_t)stream));
    if (B_host)
        LORA_CUDA_TRY(cudaMemcpyAsync(B_host, sb + tv.off_b, (size_t)pool->r_max * tv.d_out * 2,
                                      cudaMemcpyDeviceToHost, (cudaStream_t)stream));
    return LORA_OK;
}

lora_status_t lora_pool_slot_info(const lora_pool_t *pool, int32_t slot, int32_t *rank,
                                  float *scale) {
    if (!pool) return LORA_ERR_INVALID_ARG;
    if (slot < 0 || slot >= pool->num_slots) return LORA_ERR_SLOT_RANGE;
    if (rank) *rank = pool->table_host[slot].loaded ? pool->table_host[slot].rank : 0;
    if (scale) *scale = pool->table_host[slot].scale;
    return LORA_OK;
}

lora_status_t lora_pool_poll_status(lora_pool_t *pool, int32_t *host_out, void *stream) {
    if (!pool || !host_out) return LORA_ERR_INVALID_ARG;
    DeviceGuard guard(pool->device);
    if (!guard.ok) return cuda_fail(cudaErrorInvalidDevice);
    LORA_CUDA_TRY(cudaMemcpyAsync(host_out, pool->status_dev, sizeof(int32_t) * STATUS_WORDS,
                                  cudaMemcpyDeviceToHost, (cudaStream_t)stream));
    return LORA_OK;
}

lora_status_t lora_pool_reset_status(lora_pool_t *pool, void *stream) {
    if (!pool) return LORA_ERR_INVALID_ARG;
    DeviceGuard guard(pool->device);
    if (!guard.ok) return cuda_fail(cudaErrorInvalidDevice);
    LORA_CUDA_TRY(cudaMemsetAsync(pool->status_dev, 0, sizeof(int32_t) * STATUS_WORDS,
                                  (cudaStream_t)stream));
    return LORA_OK;
}

lora_status_t lora_pool_set_tuning(lora_pool_t *pool, int32_t key, int32_t value) {
    if (!pool || key < 0 || key >= 16) return LORA_ERR_INVALID_ARG;
    pool->tuning[key] = value;
    return LORA_OK;
}

const char *lora_status_string(lora_status_t s) {
    switch (s) {
        case LORA_OK: return "ok";
        case LORA_ERR_INVALID_ARG: return "invalid argument";
        case LORA_ERR_SHAPE: return "bad shape (dimensions must be positive multiples of 8)";
        case LORA_ERR_SLOT_RANGE: return "slot or target index out of range";
        case LORA_ERR_RANK: return "rank outside 1..r_max";
        case LORA_ERR_NOT_LOADED: return "slot is empty";
        case LORA_ERR_BUSY: return "slot busy";
        case LORA_ERR_BUFFER_TOO_SMALL: return "caller buffer too small";
        case LORA_ERR_NOT_PINNED: return "host adapter memory is not pinned";
        case LORA_ERR_CUDA: return "CUDA runtime error";
        case LORA_ERR_TIMEOUT: return "device-side wait timed out";
    }
    return "unknown status";
}

int32_t lora_last_cuda_error(void) { return g_last_cuda_error; }
int64_t lora_launch_count(void) { return g_launch_count.load(std::memory_order_relaxed); }

}  // extern "C"
