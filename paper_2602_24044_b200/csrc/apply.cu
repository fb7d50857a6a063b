// C entry points of the LoRA forward y = y_base + s_i * (x . A_i) . B_i (paper Section 2.2) and
// the choice of kernel path.
#include "apply_common.cuh"

namespace lora {

static bool ranges_overlap(const void *a, size_t na, const void *b, size_t nb) {
    const char *pa = (const char *)a, *pb = (const char *)b;
    return pa < pb + nb && pb < pa + na;
}

lora_status_t check_apply_args(lora_pool_t *pool, int32_t target, const void *x, int64_t ldx,
                               const void *yb, int64_t ldyb, void *y, int64_t ldy, int32_t T) {
    if (!pool) return LORA_ERR_INVALID_ARG;
    if (target < 0 || target >= pool->num_targets) return LORA_ERR_SLOT_RANGE;
    if (T < 0) return LORA_ERR_SHAPE;
    if (T == 0) return LORA_OK;
    if (!x || !yb || !y) return LORA_ERR_INVALID_ARG;
    const lora_target_t &tg = pool->targets[target];
    if (ldx < tg.d_in || ldyb < tg.d_out || ldy < tg.d_out) return LORA_ERR_SHAPE;
    if ((ldx % 8) || (ldyb % 8) || (ldy % 8)) return LORA_ERR_SHAPE;
    if (((uintptr_t)x | (uintptr_t)yb | (uintptr_t)y) & 15) return LORA_ERR_INVALID_ARG;
    if (y != yb) {
        const size_t ny = ((size_t)(T - 1) * ldy + tg.d_out) * 2;
        const size_t nb = ((size_t)(T - 1) * ldyb + tg.d_out) * 2;
        if (ranges_overlap(y, ny, yb, nb)) return LORA_ERR_INVALID_ARG;
    } else if (ldy != ldyb) {
        return LORA_ERR_INVALID_ARG;
    }
    return LORA_OK;
}

void fill_apply_params(lora_pool_t *pool, ApplyParams &P, int32_t target, const void *x,
                       int64_t ldx, const void *yb, int64_t ldyb, void *y, int64_t ldy,
                       const int32_t *slot_idx_dev, int32_t T, const void *meta, int32_t tile_m) {
    P.pool = pool->view();
    P.tv = pool->target_views[target];
    P.x = (const __nv_bfloat16 *)x;
    P.yb = (const __nv_bfloat16 *)yb;
    P.y = (__nv_bfloat16 *)y;
    P.ldx = ldx; P.ldyb = ldyb; P.ldy = ldy;
    P.slot_idx = slot_idx_dev;
    P.meta = (const int32_t *)meta;
    P.ws = nullptr;
    P.T = T;
    P.RS = rank_bucket(pool->r_max);
    P.KS = P.JS = 1;
    P.tile_m = tile_m;
    P.meta_slots = pool->num_slots;
    P.in_place = (y == yb);
    P.units = meta ? meta_layout(T, pool->num_slots, tile_m).cap_tile : T;
    if (P.units < 1) P.units = 1;
    P.off_part = P.off_vpart = P.off_vh = P.off_vl = P.off_stage = 0;
    P.stage_bytes = P.n_stages = 0;
    P.moff_perm = P.moff_udesc = P.moff_uperm = 0;
    P.path_filter = 0;
    P.no_pdl = 0;
    P.early = 0;
    P.push = 0;
}

static lora_status_t apply_common(lora_pool_t *pool, int32_t target, const void *x, int64_t ldx,
                                  const void *yb, int64_t ldyb, void *y, int64_t ldy,
                                  const int32_t *slot_idx_dev, int32_t T, const void *meta,
                                  int32_t tile_m, void *workspace, size_t workspace_bytes,
                                  cudaStream_t stream, bool use_tc) {
    ApplyParams P;
    fill_apply_params(pool, P, target, x, ldx, yb, ldyb, y, ldy, slot_idx_dev, T, meta, tile_m);
    // the workspace contract holds on every path, whether or not the chosen kernels use it
    if (!workspace || workspace_bytes < (size_t)T * P.RS * sizeof(float))
        return LORA_ERR_BUFFER_TOO_SMALL;
    if (pool->tuning[0] == 1) return launch_twophase(pool, P, workspace, workspace_bytes, stream);
    // prefill batches: runs of consecutive tokens go to the tensor-core kernels (tuning key 4 = 1
    // keeps everything on the fused kernel)
    if (use_tc && pool->tuning[4] != 1) {
        bool applies = false;
        lora_status_t s = launch_tc_long_tiles(pool, P, workspace, workspace_bytes, stream, &applies, true);
        if (s != LORA_OK) return s;
        if (applies) {
            // The tiles those kernels leave over (short, ragged or scattered ones: a handful of
            // units whose chains take tens of microseconds but move few bytes) run beside them on
            // the pool's own stream, forked from and joined back into the caller's stream; the two
            // parts write disjoint rows of y.  Tuning key 6 = 1: one after the other.
            ApplyParams rest = P;
            rest.path_filter = 32;   // runs of >= 32 consecutive tokens are taken by the other path
            const bool beside = pool->side_stream && pool->tuning[6] != 1;
            lora_status_t s_rest = LORA_OK;
            if (beside) {
                LORA_CUDA_TRY(cudaEventRecord(pool->ev_fork, stream));
                LORA_CUDA_TRY(cudaStreamWaitEvent(pool->side_stream, pool->ev_fork, 0));
                rest.no_pdl = 1;
                s_rest = launch_fused(pool, rest, pool->side_stream);
                cudaError_t e = cudaEventRecord(pool->ev_join, pool->side_stream);
                if (e != cudaSuccess && s_rest == LORA_OK) s_rest = cuda_fail(e);
            }
            bool handled = false;
            s = launch_tc_long_tiles(pool, P, workspace, workspace_bytes, stream, &handled, false);
            if (beside) {
                // the join is made whatever happened above, so a capture of the caller's stream
                // never ends with the pool's stream still forked from it
                cudaError_t e = cudaStreamWaitEvent(stream, pool->ev_join, 0);
                if (e != cudaSuccess && s == LORA_OK) s = cuda_fail(e);
            } else if (s == LORA_OK) {
                s_rest = launch_fused(pool, rest, stream);
            }
            return s != LORA_OK ? s : s_rest;
        }
    }
    return launch_fused(pool, P, stream);
}
}  // namespace lora

using namespace lora;

extern "C" {

lora_status_t lora_workspace_bytes(const lora_pool_t *pool, int32_t T_max, size_t *bytes) {
    if (!pool || !bytes) return LORA_ERR_INVALID_ARG;
    if (T_max < 0) return LORA_ERR_SHAPE;
    // eight fp32 slabs for the partial v of the tensor-core shrink's pieces (and a little slack)
    const size_t T = (size_t)(T_max > 0 ? T_max : 1);
    *bytes = (size_t)8 * T * rank_bucket(pool->r_max) * sizeof(float) + ((T / 32 + 8) * sizeof(int32_t) + 15) / 16 * 16;
    return LORA_OK;
}

lora_status_t lora_bgmv_apply(lora_pool_t *pool, int32_t target, const void *x, int64_t ldx,
                              const void *y_base, int64_t ldyb, void *y, int64_t ldy,
                              const int32_t *slot_idx_dev, int32_t T, const void *meta,
                              void *workspace, size_t workspace_bytes, void *stream) {
    lora_status_t s = check_apply_args(pool, target, x, ldx, y_base, ldyb, y, ldy, T);
    if (s != LORA_OK || T == 0) return s;
    if (!meta && !slot_idx_dev) return LORA_ERR_INVALID_ARG;
    int32_t tile_m = 1;
    if (meta) {
        if (!pool->find_meta(meta, T, &tile_m)) return LORA_ERR_INVALID_ARG;
    }
    DeviceGuard guard(pool->device);
    if (!guard.ok) return cuda_fail(cudaErrorInvalidDevice);
    return apply_common(pool, target, x, ldx, y_base, ldyb, y, ldy, slot_idx_dev, T, meta, tile_m,
                        workspace, workspace_bytes, (cudaStream_t)stream, false);
}

lora_status_t lora_bgmv_apply_multi(lora_pool_t *pool, const lora_apply_item_t *items, int32_t n_items,
                                    const int32_t *slot_idx_dev, int32_t T, const void *meta,
                                    void *workspace, size_t workspace_bytes, void *stream) {
    if (!pool || !items || n_items < 1 || n_items > LORA_MULTI_MAX) return LORA_ERR_INVALID_ARG;
    if (T < 0) return LORA_ERR_SHAPE;
    for (int32_t i = 0; i < n_items; ++i) {
        const lora_apply_item_t &it = items[i];
        lora_status_t s = check_apply_args(pool, it.target, it.x, it.ldx, it.y_base, it.ldyb, it.y, it.ldy, T);
        if (s != LORA_OK) return s;
    }
    if (T == 0) return LORA_OK;
    if (!meta) return LORA_ERR_INVALID_ARG;
    int32_t tile_m = 1;
    if (!pool->find_meta(meta, T, &tile_m)) return LORA_ERR_INVALID_ARG;
    // independence: nothing an item writes may be read or written by another item
    for (int32_t i = 0; i < n_items; ++i) {
        const lora_target_t &ti = pool->targets[items[i].target];
        const size_t ny = ((size_t)(T - 1) * items[i].ldy + ti.d_out) * 2;
        for (int32_t j = 0; j < n_items; ++j) {
            if (j == i) continue;
            const lora_target_t &tj = pool->targets[items[j].target];
            if (ranges_overlap(items[i].y, ny, items[j].x, ((size_t)(T - 1) * items[j].ldx + tj.d_in) * 2) ||
                ranges_overlap(items[i].y, ny, items[j].y_base, ((size_t)(T - 1) * items[j].ldyb + tj.d_out) * 2) ||
                ranges_overlap(items[i].y, ny, items[j].y, ((size_t)(T - 1) * items[j].ldy + tj.d_out) * 2))
                return LORA_ERR_INVALID_ARG;
        }
    }
    if (!workspace || workspace_bytes < (size_t)T * rank_bucket(pool->r_max) * sizeof(float))
        return LORA_ERR_BUFFER_TOO_SMALL;
    DeviceGuard guard(pool->device);
    if (!guard.ok) return cuda_fail(cudaErrorInvalidDevice);
    ApplyParams P[LORA_MULTI_MAX];
    for (int32_t i = 0; i < n_items; ++i)
        fill_apply_params(pool, P[i], items[i].target, items[i].x, items[i].ldx, items[i].y_base,
                          items[i].ldyb, items[i].y, items[i].ldy, slot_idx_dev, T, meta, tile_m);
    if (pool->tuning[0] == 1) {   // the two-phase baseline has no multi-projection form
        for (int32_t i = 0; i < n_items; ++i) {
            lora_status_t s = launch_twophase(pool, P[i], workspace, workspace_bytes, (cudaStream_t)stream);
            if (s != LORA_OK) return s;
        }
        return LORA_OK;
    }
    return launch_fused_items(pool, P, n_items, (cudaStream_t)stream);
}

lora_status_t lora_sgmv_apply(lora_pool_t *pool, int32_t target, const void *x, int64_t ldx,
                              const void *y_base, int64_t ldyb, void *y, int64_t ldy,
                              const void *meta, int32_t T, void *workspace, size_t workspace_bytes,
                              void *stream) {
    lora_status_t s = check_apply_args(pool, target, x, ldx, y_base, ldyb, y, ldy, T);
    if (s != LORA_OK || T == 0) return s;
    if (!meta) return LORA_ERR_INVALID_ARG;
    int32_t tile_m = 1;
    if (!pool->find_meta(meta, T, &tile_m)) return LORA_ERR_INVALID_ARG;
    DeviceGuard guard(pool->device);
    if (!guard.ok) return cuda_fail(cudaErrorInvalidDevice);
    return apply_common(pool, target, x, ldx, y_base, ldyb, y, ldy, nullptr, T, meta, tile_m,
                        workspace, workspace_bytes, (cudaStream_t)stream, true);
}

lora_status_t lora_apply_host(lora_pool_t *pool, int32_t target, int32_t kind, const void *x_host,
                              const void *y_base_host, void *y_host, const int32_t *slot_idx_host,
                              int32_t T, int32_t tile_m, int32_t long_min,
                              const lora_step_buffers_t *dev, void *stream) {
    if (!pool || !dev) return LORA_ERR_INVALID_ARG;
    if (target < 0 || target >= pool->num_targets) return LORA_ERR_SLOT_RANGE;
    if (T < 0) return LORA_ERR_SHAPE;
    if (kind != 0 && kind != 1) return LORA_ERR_INVALID_ARG;
    if (T == 0) return LORA_OK;
    if (!x_host || !y_base_host || !y_host || !slot_idx_host || !dev->x_dev || !dev->y_base_dev ||
        !dev->y_dev || !dev->slot_idx_dev || !dev->meta_dev)
        return LORA_ERR_INVALID_ARG;
    const lora_target_t &tg = pool->targets[target];
    cudaStream_t st = (cudaStream_t)stream;
    DeviceGuard guard(pool->device);
    if (!guard.ok) return cuda_fail(cudaErrorInvalidDevice);
    LORA_CUDA_TRY(cudaMemcpyAsync(dev->slot_idx_dev, slot_idx_host, sizeof(int32_t) * (size_t)T,
                                  cudaMemcpyHostToDevice, st));
    LORA_CUDA_TRY(cudaMemcpyAsync(dev->x_dev, x_host, (size_t)T * tg.d_in * 2,
                                  cudaMemcpyHostToDevice, st));
    LORA_CUDA_TRY(cudaMemcpyAsync(dev->y_base_dev, y_base_host, (size_t)T * tg.d_out * 2,
                                  cudaMemcpyHostToDevice, st));
    lora_status_t s = lora_build_segments(pool, dev->slot_idx_dev, T, tile_m, long_min,
                                          dev->meta_dev, dev->meta_bytes, stream);
    if (s != LORA_OK) return s;
    if (kind == 0)
        s = lora_bgmv_apply(pool, target, dev->x_dev, tg.d_in, dev->y_base_dev, tg.d_out, dev->y_dev,
                            tg.d_out, dev->slot_idx_dev, T, dev->meta_dev, dev->workspace,
                            dev->workspace_bytes, stream);
    else
        s = lora_sgmv_apply(pool, target, dev->x_dev, tg.d_in, dev->y_base_dev, tg.d_out, dev->y_dev,
                            tg.d_out, dev->meta_dev, T, dev->workspace, dev->workspace_bytes, stream);
    if (s != LORA_OK) return s;
    LORA_CUDA_TRY(cudaMemcpyAsync(y_host, dev->y_dev, (size_t)T * tg.d_out * 2,
                                  cudaMemcpyDeviceToHost, st));
    return LORA_OK;
}

}  // extern "C"
