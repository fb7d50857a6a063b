// Pieces shared by the apply kernels: launch parameters, the unit (tile or token) a block works
// on, bf16 packing helpers and the warp reduction used by the shrink phase.
#pragma once

#include "common.cuh"

namespace lora {

constexpr int AP_THREADS = 256;
constexpr int ROWS_CAP = 128;   // largest tile_m

struct ApplyParams {
    PoolView pool;
    TargetView tv;
    const __nv_bfloat16 *x;
    const __nv_bfloat16 *yb;
    __nv_bfloat16 *y;
    int64_t ldx, ldyb, ldy;
    const int32_t *slot_idx;   // per-token mode
    const int32_t *meta;       // grouped mode (nullptr = per-token mode)
    float *ws;                 // two-phase path: [KS][T][RS] fp32 partial v
    int32_t T, RS, KS, JS;
    int32_t units;             // capacity of the unit list (tiles, 16-row pieces or tokens)
    int32_t tile_m, meta_slots;
    int32_t in_place;
    // fused path: shared-memory carve-up (bytes from the start of dynamic shared memory)
    int32_t off_part, off_vpart, off_vh, off_vl;   // warp partials, block partial, v as bf16 high / low parts
    int32_t off_stage, stage_bytes, n_stages;      // ring of job buffers
    int32_t moff_perm, moff_udesc, moff_uperm;     // word offsets: perm, unit records, unit row ids
    int32_t push;              // fused path: block partials are pushed to all blocks of the cluster (small units)
    int32_t early;             // the unit records and the pool may be read before the preceding kernel has finished
    int32_t path_filter;       // 0 = every unit; else skip runs of at least this many consecutive tokens
    int32_t no_pdl;            // 1 = plain launch (the kernel does not follow a kernel of its own stream)
};

struct Tile {
    int32_t slot, rank, row0, rows;
    float scale;
    bool valid;
};

__device__ __forceinline__ uint4 ldg16(const __nv_bfloat16 *p) {
    return __ldg(reinterpret_cast<const uint4 *>(p));
}
__device__ __forceinline__ void unpack8(const uint4 &w, float (&f)[8]) {
    f[0] = __uint_as_float(w.x << 16); f[1] = __uint_as_float(w.x & 0xffff0000u);
    f[2] = __uint_as_float(w.y << 16); f[3] = __uint_as_float(w.y & 0xffff0000u);
    f[4] = __uint_as_float(w.z << 16); f[5] = __uint_as_float(w.z & 0xffff0000u);
    f[6] = __uint_as_float(w.w << 16); f[7] = __uint_as_float(w.w & 0xffff0000u);
}
__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
    __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&h);
}
// y = bf16(y_base + s * acc), eight columns
__device__ __forceinline__ uint4 finish8(const float (&acc)[8], const uint4 &ybv, float s) {
    float yf[8];
    unpack8(ybv, yf);
    uint4 o;
    o.x = pack2(fmaf(s, acc[0], yf[0]), fmaf(s, acc[1], yf[1]));
    o.y = pack2(fmaf(s, acc[2], yf[2]), fmaf(s, acc[3], yf[3]));
    o.z = pack2(fmaf(s, acc[4], yf[4]), fmaf(s, acc[5], yf[5]));
    o.w = pack2(fmaf(s, acc[6], yf[6]), fmaf(s, acc[7], yf[7]));
    return o;
}

// Sum of v[0..31] across the warp: lane l returns the total of element l.  Each step halves
// the element count by exchanging one half with the partner lane; the summation tree over lanes
// is the same for every element.
template <int N>
__device__ __forceinline__ void fold(float (&v)[32], int lane) {
    const bool up = (lane & N) != 0;
#pragma unroll
    for (int i = 0; i < N; ++i) {
        const float send = up ? v[i] : v[i + N];
        const float keep = up ? v[i + N] : v[i];
        v[i] = keep + __shfl_xor_sync(0xffffffffu, send, N);
    }
}
__device__ __forceinline__ float warp_reduce32(float (&v)[32], int lane) {
    fold<16>(v, lane);
    fold<8>(v, lane);
    fold<4>(v, lane);
    fold<2>(v, lane);
    fold<1>(v, lane);
    return v[0];
}

__device__ __forceinline__ Tile resolve_unit(const ApplyParams &P, const MetaLayout &L, int32_t u) {
    Tile t;
    t.valid = false;
    t.slot = -1; t.rank = 0; t.row0 = 0; t.rows = 0; t.scale = 0.0f;
    if (P.meta) {
        const int4 d = *reinterpret_cast<const int4 *>(P.meta + L.tile_desc + 4 * (int64_t)u);
        if (d.x < 0) return t;   // unused entry
        t.slot = d.x;
        t.row0 = d.y;
        t.rows = d.z & 0x7fff;
        t.rank = d.z >> 16;
        t.scale = __int_as_float(d.w);
        t.valid = true;
    } else {
        if (u >= P.T) return t;
        const int32_t s = P.slot_idx[u];
        t.row0 = u;
        t.rows = 1;
        if (s >= 0 && s < P.pool.num_slots) {
            const SlotEntry e = P.pool.table[s];
            if (e.loaded) {
                t.slot = s; t.rank = e.rank; t.scale = e.scale; t.valid = true;
            }
        }
    }
    return t;
}

// y_base -> y for rows that take no adapter (out-of-place calls only); the columns are split
// over `parts` blocks, this block being number `part`.
__device__ __forceinline__ void copy_rows(const ApplyParams &P, const int32_t *rowidx, int32_t rows,
                                          int32_t part, int32_t parts, int32_t nthreads = 0) {
    if (nthreads == 0) nthreads = (int32_t)blockDim.x;   // threads that take part (the first ones of the block)
    const int32_t vecs = P.tv.d_out / 8;
    for (int32_t m = 0; m < rows; ++m) {
        const __nv_bfloat16 *src = P.yb + (int64_t)rowidx[m] * P.ldyb;
        __nv_bfloat16 *dst = P.y + (int64_t)rowidx[m] * P.ldy;
        for (int32_t v = part * nthreads + threadIdx.x; v < vecs; v += parts * nthreads)
            reinterpret_cast<uint4 *>(dst)[v] = ldg16(src + (int64_t)v * 8);
    }
}

static inline int32_t next_pow2(int32_t v) {
    int32_t p = 1;
    while (p < v) p <<= 1;
    return p;
}

// launchers (each fills in the fields it owns)
lora_status_t launch_twophase(lora_pool_t *pool, ApplyParams &P, void *workspace,
                              size_t workspace_bytes, cudaStream_t stream);
lora_status_t launch_fused(lora_pool_t *pool, ApplyParams &P, cudaStream_t stream);
lora_status_t launch_fused_items(lora_pool_t *pool, const ApplyParams *items, int32_t n_items,
                                 cudaStream_t stream);
lora_status_t build_fused_maps(lora_pool_t *pool);
lora_status_t launch_tc_long_tiles(lora_pool_t *pool, const ApplyParams &AP, void *workspace,
                                   size_t workspace_bytes, cudaStream_t stream, bool *handled,
                                   bool check_only);
// Whether a batch of T tokens built with tile_m would be given to the tensor-core kernels, and the
// launch that writes their list of long tiles into the metadata (behind the build, same stream).
bool tc_path_wanted(const lora_pool_t *pool, int32_t T, int32_t tile_m);
lora_status_t launch_tc_worklist(lora_pool_t *pool, int32_t T, int32_t tile_m, void *meta_dev,
                                 cudaStream_t stream);
lora_status_t launch_build_segments(lora_pool_t *pool, const int32_t *slot_idx_dev, int32_t T,
                                    int32_t tile_m, int32_t long_min, void *meta_dev,
                                    cudaStream_t stream);

}  // namespace lora
