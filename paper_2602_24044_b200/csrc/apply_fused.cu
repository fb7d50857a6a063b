// Fused LoRA forward y = y_base + s_i * (x . A_i) . B_i (paper Section 2.2) in ONE launch for
// every rank of a batch and for up to eight independent projections that share the batch (the
// adapted projections of one transformer layer: q, k, v, o, gate, up, down).  This file holds what
// the two kernels share (launch parameters, the tensor maps, the launcher); the kernels are in
// decode_kernel.cuh (decode batches: units of at most 8 rows, ranks up to 16, whole 64-column
// blocks) and stream_kernel.cuh (everything else).
//
// Common design.  A unit is a few token rows of one adapter in one projection.  A thread-block
// cluster owns one unit at a time (units cid, cid + G, ... of the launch; the units of projection
// 0 come first, then those of projection 1, ...); block c of the cluster takes the c-th slice of
// d_in for the shrink phase and the c-th slice of d_out for the expand phase; the intermediate
// v = x . A_i never leaves the cluster (exchange through distributed shared memory, summed in
// block order, no float atomics).  A fifth warp requests jobs (one column chunk each: the rank rows
// of A_i or B_i by one tiled TMA copy, the unit's token rows by one bulk copy per row) into a ring
// of shared-memory stages, software-pipelined by one unit so that a unit's exchange runs under the
// next unit's shrink; the four consumer warps follow the job headers.  Every per-row sum is taken
// in a fixed order that does not depend on which other rows share the unit, so a row's result
// depends only on its inputs.
//
// Consecutive launches overlap (programmatic dependent launch): a kernel lets its successor
// become resident; the successor reads the unit records and the pool and requests its first
// weight tiles while this kernel is still running, and touches activations only after
// griddepcontrol.wait.
#include <cstring>

#include "apply_common.cuh"
#include "fused_ptx.cuh"

namespace lora {

constexpr int FT = 128;          // consumer threads per block (four warps)
constexpr int FT_ALL = 160;      // plus the warp that requests the jobs
constexpr int SM_HEADER = 1024;  // general kernel: barriers, job headers and unit entries come before the carved-up buffers
constexpr int MAX_STAGES = 4;
constexpr int W_BYTES = 8192;    // decode kernel: weight tile of a job, 16 rank rows x 256 columns x 2 bytes
constexpr int GEN_W_BYTES = 16384;   // general kernel: 32 rank rows x 256 columns or 64 x 128
constexpr int TOK_PITCH = 256 + 8;   // elements between token rows of a stage (+16 B against bank conflicts)
constexpr int MAPS_PER_TARGET = 16;  // tensor maps of a target: A then B, index rows / 8 - 1 for loads of 8 .. 64 rank rows
constexpr int MAX_ITEMS = 8;

#ifndef LORA_FUSED_MIN_BLOCKS
#define LORA_FUSED_MIN_BLOCKS 6   // resident blocks per SM the register budget is held to
#endif

// one projection of a launch
struct FusedItem {
    const __nv_bfloat16 *x, *yb;
    __nv_bfloat16 *y;
    int64_t ldx, ldyb, ldy;
    int32_t d_in, d_out;
    int32_t wa, wb;          // columns of d_in / d_out per block of the cluster (multiples of 64)
    int32_t map_base;        // index of the target's first tensor map
    int32_t in_place;
};

struct FusedParams {
    PoolView pool;
    const CUtensorMap *maps;   // [num_targets][MAPS_PER_TARGET], in the pool's device buffer
    const int32_t *slot_idx;   // per-token mode
    const int32_t *meta;       // grouped mode (nullptr = per-token mode)
    int32_t T, units_cap, n_items;
    int32_t early;             // the unit records and the pool may be read before the preceding kernel has finished
    int32_t push;              // block partials are pushed to all blocks of the cluster (small units)
    int32_t path_filter;       // 0 = every unit; else skip runs of at least this many consecutive tokens
    int32_t no_pdl;            // host side only: launch without the programmatic-launch attribute
    int32_t late_trigger;      // decode kernel: let the successor in only once this kernel's blocks are set up
    int32_t copy_idle;         // some projection is out of place: rows without adapter are copied
    int32_t off_part, off_vpart, vbuf_bytes, off_vh, off_vl;   // warp partials, exchange buffers (x2), v as bf16 high / low parts
    int32_t off_w, off_tok, tok_bytes, n_stages;               // ring of job buffers: weight tiles, token rows
    int32_t w_bytes;                                           // general kernel: bytes of a stage's weight tile
    int32_t moff_perm, moff_udesc, moff_uperm;                 // word offsets: perm, unit records, unit row ids
    FusedItem item[MAX_ITEMS];
};

}  // namespace lora

#include "decode_kernel.cuh"
#include "stream_kernel.cuh"

namespace lora {

// ---------------------------------------------------------------------------------------------
// host side: tensor maps (built once per pool, kept in the pool's device buffer) and launch
// ---------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

static EncodeTiledFn tiled_encoder() {
    void *p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
        return (EncodeTiledFn)p;
    cudaGetLastError();
    return nullptr;
}

// One target's matrix family in the pool, [slot][r_max rows][d columns], viewed as a 4-D tensor
// (column inside a 64-column block, rank row, column block, slot); box = 64 x rows x blocks x 1.
// The last column block of a row may reach into the next row (or, in the last row of the last
// slot, into the pool's slack bytes); such columns are never used.
static bool weight_map(EncodeTiledFn fn, CUtensorMap *m, const void *base, int64_t d, int64_t r_max,
                       int64_t slots, int64_t slot_stride, int rows, int blocks) {
    cuuint64_t dims[4] = {64, (cuuint64_t)r_max, (cuuint64_t)((d + 63) / 64), (cuuint64_t)slots};
    cuuint64_t strides[3] = {(cuuint64_t)d * 2, 128, (cuuint64_t)slot_stride * 2};
    cuuint32_t box[4] = {64, (cuuint32_t)rows, (cuuint32_t)blocks, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Called by lora_pool_create: the tensor maps of every target, written into the pool's buffer.
lora_status_t build_fused_maps(lora_pool_t *pool) {
    static_assert(sizeof(CUtensorMap) == 128, "tensor map size");
    EncodeTiledFn fn = tiled_encoder();
    if (!fn) return cuda_fail(cudaErrorNotSupported);
    std::vector<CUtensorMap> maps((size_t)pool->num_targets * MAPS_PER_TARGET);
    memset(maps.data(), 0, maps.size() * sizeof(CUtensorMap));
    const __nv_bfloat16 *w = pool->weights_dev;
    for (int32_t t = 0; t < pool->num_targets; ++t) {
        const TargetView &tv = pool->target_views[t];
        for (int i = 0; i < 8; ++i) {
            const int rows = 8 * (i + 1);
            if (rows > ((pool->r_max + 7) & ~7)) break;   // no slot holds that many rank rows
            const int blocks = rows <= 32 ? 4 : 2;   // chunk width 256 columns up to 32 rank rows, 128 above
            if (!weight_map(fn, &maps[(size_t)t * MAPS_PER_TARGET + i], w + tv.off_a, tv.d_in, pool->r_max,
                            pool->num_slots, pool->slot_stride, rows, blocks) ||
                !weight_map(fn, &maps[(size_t)t * MAPS_PER_TARGET + 8 + i], w + tv.off_b, tv.d_out, pool->r_max,
                            pool->num_slots, pool->slot_stride, rows, blocks))
                return cuda_fail(cudaErrorInvalidValue);
        }
    }
    LORA_CUDA_TRY(cudaMemcpy(pool->maps_dev, maps.data(), maps.size() * sizeof(CUtensorMap),
                             cudaMemcpyHostToDevice));
    return LORA_OK;
}

// Shared-memory carve-up and launch.  The buffers are sized for the largest rank bucket that has
// ever been loaded into the pool.  H = 0: the decode kernel (its own fixed carve-up).
template <int H>
static lora_status_t launch_h(lora_pool_t *pool, FusedParams &P, int32_t C, const void *meta_key,
                              cudaStream_t stream) {
    void (*kern)(const FusedParams) = nullptr;
    if (H == 0) kern = decode_kernel;
    else if (H == 1) kern = stream_kernel<1>;
    else kern = stream_kernel<2>;
    const int32_t mrows = H == 2 ? 16 : 8;
    const int32_t RPmax = (pool->bucket_mask & 8u) ? 64 : (pool->bucket_mask & 4u) ? 32 : 16;
    int32_t S = pool->tuning[5];
    if (S < 2 || S > MAX_STAGES) S = 2;   // two stages and more resident blocks beat deeper rings
    int32_t o = SM_HEADER;
    const int32_t nwc = H == 2 ? 8 : 4;   // consumer warps of the kernel
    P.off_part = o;   o += mrows * 16 * nwc * 4;
    // general kernel: a block's partial stays in its own shared memory, two sets (the decode kernel
    // pushes partials into every block; its carve-up is fixed)
    P.push = 0;
    P.vbuf_bytes = mrows * RPmax * 4;
    P.off_vpart = o;  o += 2 * P.vbuf_bytes;
    P.off_vh = o;     o += mrows * gen::PV * 2;
    P.off_vl = o;     o += mrows * gen::PV * 2;
    o = (o + 1023) & ~1023;
    // a pool that has never held a rank above 16 needs only 8 KB tiles (16 rank rows x 256 columns)
    P.w_bytes = RPmax <= 16 ? W_BYTES : GEN_W_BYTES;
    P.off_w = o;      o += S * P.w_bytes;
    P.tok_bytes = mrows * TOK_PITCH * 2;
    P.off_tok = o;    o += S * P.tok_bytes;
    P.n_stages = S;
    const int32_t smem = H == 0 ? dec::smem_bytes(S) : o;
    // A launch of many projections runs for several waves of units; letting its successor's blocks
    // in early only takes resources from its own later units (measured: -10 % on a seven-projection
    // launch), while a short launch gains from the overlap.  Tuning key 11: 1 = never early, 2 = always.
    P.late_trigger = pool->tuning[11] == 1 ? 1 : pool->tuning[11] == 2 ? 0 : P.n_items >= 4 ? 1 : 0;
    P.copy_idle = 0;
    for (int32_t i = 0; i < P.n_items; ++i) P.copy_idle |= P.item[i].in_place ? 0 : 1;

    lora_pool::FusedLaunchCache &lc = pool->fused_cache[H];
    if (smem > lc.attr_smem) {
        LORA_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        lc.attr_smem = smem;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3((unsigned)(32 * (nwc + 1)), 1, 1);
    cfg.dynamicSmemBytes = (size_t)smem;
    cfg.stream = stream;
    cudaLaunchAttribute at[2];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = (unsigned)C;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    // Programmatic dependent launch (tuning key 2: 0 = when allowed, 2 = never).  Reading the table
    // and the pool ahead of the preceding kernel's end is allowed for grouped batches whose table
    // has already been read by an earlier apply: that apply was fully ordered behind the build, so
    // the table is complete before this kernel can start.
    const bool fresh = meta_key ? pool->take_fresh(meta_key) : true;
    P.early = (meta_key && !fresh && pool->tuning[2] != 2 && !P.no_pdl) ? 1 : 0;
    // Without `early` the attribute still lets the blocks become resident and set up their shared
    // memory while the kernel before them drains; they read nothing until it has completed.
    const unsigned n_attrs = (pool->tuning[2] != 2 && !P.no_pdl) ? 2 : 1;

    // Grid: no more clusters than can be resident at once (each loops over its units), so no
    // cluster of an over-sized grid waits for a slot only to find that its unit does not exist.
    if (lc.occ_smem != smem || lc.occ_c != C) {
        cfg.gridDim = dim3((unsigned)(C * pool->sm_count), 1, 1);
        cfg.numAttrs = 1;
        int n = 0;
        cudaError_t e = cudaOccupancyMaxActiveClusters(&n, kern, &cfg);
        if (e != cudaSuccess || n < 1) {
            cudaGetLastError();
            n = 0;
        }
        lc.occ_smem = smem; lc.occ_c = C; lc.occ_clusters = n;
    }
    cfg.numAttrs = n_attrs;
    int32_t want = P.units_cap * P.n_items;   // units, or 16-row copy steps if there are more of those
    bool copies = false;
    for (int32_t i = 0; i < P.n_items; ++i) copies = copies || !P.item[i].in_place;
    if (P.meta && copies && (P.T + 15) / 16 * P.n_items > want) want = (P.T + 15) / 16 * P.n_items;
    int32_t G = lc.occ_clusters > 0 && lc.occ_clusters < want ? lc.occ_clusters : want;
    // tuning key 3: upper bound on the clusters; key 9: share of the resident clusters a launch
    // takes, in percent (a launch that leaves room lets its successor become resident beside it)
    if (pool->tuning[9] > 0 && pool->tuning[9] < 100 && lc.occ_clusters > 0) {
        const int32_t part = (lc.occ_clusters * pool->tuning[9] + 99) / 100;
        if (part >= 1 && part < G) G = part;
    }
    if (pool->tuning[3] > 0 && pool->tuning[3] < G) G = pool->tuning[3];
    if (G < 1) G = 1;
    cfg.gridDim = dim3((unsigned)(G * C), 1, 1);
    LORA_CUDA_TRY(cudaLaunchKernelEx(&cfg, kern, P));
    return count_launch();
}

// items: the projections of the launch (n_items of ApplyParams with one batch, one table); the
// units of item 0 are walked first, so the caller lists the widest projections first.
lora_status_t launch_fused_items(lora_pool_t *pool, const ApplyParams *items, int32_t n_items,
                                 cudaStream_t stream) {
    if (n_items < 1 || n_items > MAX_ITEMS) return LORA_ERR_INVALID_ARG;
    const ApplyParams &A0 = items[0];
    FusedParams P;
    memset(&P, 0, sizeof(P));
    P.pool = A0.pool;
    P.maps = pool->maps_dev;
    P.slot_idx = A0.slot_idx;
    P.meta = A0.meta;
    P.T = A0.T;
    P.n_items = n_items;
    P.path_filter = A0.path_filter;
    P.no_pdl = A0.no_pdl;
    const int32_t tile_m = A0.meta ? A0.tile_m : 1;
    P.units_cap = A0.T;
    if (A0.meta) {
        const MetaLayout L = meta_layout(A0.T, A0.meta_slots, A0.tile_m);
        if (L.words > 0x7fffffff) return LORA_ERR_SHAPE;
        P.moff_perm = (int32_t)L.perm;
        P.moff_udesc = (int32_t)L.unit_desc;
        P.moff_uperm = (int32_t)L.unit_perm;
        P.units_cap = L.cap_unit;
    }
    if (P.units_cap < 1) P.units_cap = 1;
    // cluster size: as wide a split as the narrowest projection of the launch supports
    int32_t C = pool->tuning[1];
    if (C != 1 && C != 2 && C != 4 && C != 8) {
        // Eight blocks per unit shorten a unit's chain, four leave twice as many clusters for a
        // batch with several units per cluster: a long prefill-type batch that keeps all its tiles
        // here has hundreds of 16-row units (mixed chunked prefill: 84 us with 4, 91 us with 8);
        // what the tensor-core kernels leave over is a handful of units (prefill: 322 us with 8, 347 with 4).
        C = (tile_m > 8 && A0.T >= 1024 && P.path_filter == 0) ? 4 : 8;
        for (int32_t i = 0; i < n_items; ++i)
            while (C > 1 && (items[i].tv.d_in / C < 256 || items[i].tv.d_out / C < 128)) C >>= 1;
    }
    for (int32_t i = 0; i < n_items; ++i) {
        const ApplyParams &A = items[i];
        FusedItem &it = P.item[i];
        it.x = A.x; it.yb = A.yb; it.y = A.y;
        it.ldx = A.ldx; it.ldyb = A.ldyb; it.ldy = A.ldy;
        it.d_in = A.tv.d_in; it.d_out = A.tv.d_out;
        const int32_t cs64 = C * 64;
        it.wa = (A.tv.d_in + cs64 - 1) / cs64 * 64;
        it.wb = (A.tv.d_out + cs64 - 1) / cs64 * 64;
        int32_t target = -1;
        for (int32_t t = 0; t < pool->num_targets; ++t)
            if (pool->target_views[t].off_a == A.tv.off_a) target = t;
        if (target < 0) return LORA_ERR_INVALID_ARG;
        it.map_base = target * MAPS_PER_TARGET;
        it.in_place = A.in_place;
    }
    // Decode batches take the decode kernel: grouped metadata with units of at most 8 rows, no
    // adapter above rank 16 in the pool, widths in whole 64-column blocks and no block of the
    // cluster without columns (tuning key 10 = 1: always the general kernel).
    bool decode = A0.meta && tile_m <= 8 && (pool->bucket_mask & 12u) == 0 && P.path_filter == 0 &&
                  pool->tuning[10] != 1;
    for (int32_t i = 0; i < n_items && decode; ++i) {
        const FusedItem &it = P.item[i];
        decode = it.d_in % 64 == 0 && it.d_out % 64 == 0 && (C - 1) * it.wa < it.d_in &&
                 (C - 1) * it.wb < it.d_out;
    }
    if (decode) return launch_h<0>(pool, P, C, A0.meta, stream);
    return tile_m <= 8 ? launch_h<1>(pool, P, C, A0.meta, stream) : launch_h<2>(pool, P, C, A0.meta, stream);
}

lora_status_t launch_fused(lora_pool_t *pool, ApplyParams &P, cudaStream_t stream) {
    return launch_fused_items(pool, &P, 1, stream);
}

}  // namespace lora
