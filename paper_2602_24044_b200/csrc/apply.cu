// The LoRA forward y = y_base + s_i * (x . A_i) . B_i on CUDA cores (paper Section 2.2: the
// adapter's two low-rank matrices produce activations that are added to the backbone layer's
// output; several adapters are served inside one batch).
//
// Two phases per call:
//   shrink  v[t, 0:r] = x[t, :] . A_i      split over d_in across blocks (split-K), fp32
//   expand  y[t, :]   = bf16( y_base[t, :] + s_i * (v[t, :] . B_i) )
// Work units are row tiles of one adapter (from the segment metadata) or single tokens.
// Every per-row sum is taken in a fixed order that does not depend on which other rows share
// the tile, so a row's result depends only on its own inputs.
#include "common.cuh"

namespace lora {

constexpr int AP_THREADS = 256;
constexpr int ROWS_CAP = 128;            // largest tile_m
constexpr int AP_SMEM_BYTES = 32 * 1024 + ROWS_CAP * 4;

struct ApplyParams {
    PoolView pool;
    TargetView tv;
    const __nv_bfloat16 *x;
    const __nv_bfloat16 *yb;
    __nv_bfloat16 *y;
    int64_t ldx, ldyb, ldy;
    const int32_t *slot_idx;   // per-token mode
    const int32_t *meta;       // grouped mode (nullptr = per-token mode)
    float *ws;                 // [KS][T][RS] fp32 partial v
    int32_t T, RS, KS, JS;
    int32_t units;             // blocks in x that map to tiles / tokens
    int32_t tile_m, meta_slots;
    int32_t in_place;
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

// Sum of v[0..31] across the warp: lane l returns the total of element l.
// Each step halves the element count by exchanging one half with the partner lane.
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
        if (u >= P.meta[H_NTILE]) return t;
        const int32_t seg = P.meta[L.tile_seg + u];
        t.slot = P.meta[L.seg_slot + seg];
        t.rank = P.meta[L.seg_rank + seg];
        t.row0 = P.meta[L.tile_row0 + u];
        t.rows = P.meta[L.tile_rows + u];
        t.scale = P.pool.table[t.slot].scale;
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

// ---------------------------------------------------------------------------------------------
// shrink: each thread owns one 8-wide column vector of the chunk and KPT ranks; A stays in
// registers for the whole tile, rows of x stream through; 32 partial sums at a time are folded
// across the warp.
// ---------------------------------------------------------------------------------------------
template <int RP, int KPT>
__device__ __forceinline__ void shrink_tile(const ApplyParams &P, const Tile &tl, const int32_t *rowidx,
                                            float *part) {
    constexpr int KG = RP / KPT, CV = AP_THREADS / KG, DC = CV * 8, WPK = CV / 32, MG = 32 / KPT;
    const int tid = threadIdx.x, lane = tid & 31;
    const int kg = tid / CV, cv = tid % CV, wk = cv >> 5;
    const int ks = blockIdx.y;
    const int32_t d_in = P.tv.d_in, rows = tl.rows;
    const __nv_bfloat16 *A = P.pool.weights + (int64_t)tl.slot * P.pool.slot_stride + P.tv.off_a;

    for (int i = tid; i < WPK * rows * RP; i += AP_THREADS) part[i] = 0.0f;
    __syncthreads();

    const int32_t nchunks = (d_in + DC - 1) / DC;
    for (int32_t c = ks; c < nchunks; c += P.KS) {
        const int32_t d0 = c * DC + cv * 8;
        const bool dvalid = d0 < d_in;
        float a[KPT][8];
#pragma unroll
        for (int kk = 0; kk < KPT; ++kk) {
            const int k = kg * KPT + kk;
            uint4 w = make_uint4(0, 0, 0, 0);
            if (dvalid && k < tl.rank) w = ldg16(A + (int64_t)k * d_in + d0);
            unpack8(w, a[kk]);
        }
        for (int32_t m0 = 0; m0 < rows; m0 += MG) {
            uint4 xv[MG];
#pragma unroll
            for (int mi = 0; mi < MG; ++mi) {
                xv[mi] = make_uint4(0, 0, 0, 0);
                if (dvalid && m0 + mi < rows)
                    xv[mi] = ldg16(P.x + (int64_t)rowidx[m0 + mi] * P.ldx + d0);
            }
            float acc[32];
#pragma unroll
            for (int mi = 0; mi < MG; ++mi) {
                float xf[8];
                unpack8(xv[mi], xf);
#pragma unroll
                for (int kk = 0; kk < KPT; ++kk) {
                    float s = 0.0f;
#pragma unroll
                    for (int e = 0; e < 8; ++e) s = fmaf(xf[e], a[kk][e], s);
                    acc[mi * KPT + kk] = s;
                }
            }
            const float tot = warp_reduce32(acc, lane);
            const int mi = lane / KPT, kk = lane % KPT;
            if (m0 + mi < rows) part[(wk * rows + m0 + mi) * RP + kg * KPT + kk] += tot;
        }
    }
    __syncthreads();
    for (int i = tid; i < rows * RP; i += AP_THREADS) {
        const int m = i / RP, k = i % RP;
        float v = 0.0f;
#pragma unroll
        for (int w = 0; w < WPK; ++w) v += part[(w * rows + m) * RP + k];
        if (k < P.RS) P.ws[((int64_t)ks * P.T + tl.row0 + m) * P.RS + k] = v;
    }
}

__global__ void __launch_bounds__(AP_THREADS)
shrink_kernel(const ApplyParams P) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float *part = reinterpret_cast<float *>(smem_raw);
    int32_t *rowidx = reinterpret_cast<int32_t *>(smem_raw + 32 * 1024);
    MetaLayout L;
    if (P.meta) L = meta_layout(P.T, P.meta_slots, P.tile_m);
    const Tile tl = resolve_unit(P, L, blockIdx.x);
    if (!tl.valid) return;
    for (int i = threadIdx.x; i < tl.rows; i += AP_THREADS)
        rowidx[i] = P.meta ? P.meta[L.perm + tl.row0 + i] : tl.row0 + i;
    __syncthreads();
    switch (rank_bucket(tl.rank)) {
        case 8: shrink_tile<8, 4>(P, tl, rowidx, part); break;
        case 16: shrink_tile<16, 4>(P, tl, rowidx, part); break;
        case 32: shrink_tile<32, 4>(P, tl, rowidx, part); break;
        default: shrink_tile<64, 8>(P, tl, rowidx, part); break;
    }
}

// number of split-K partials that carry data for a tile of this rank bucket
__device__ __forceinline__ int32_t valid_partials(const ApplyParams &P, int32_t rank) {
    const int32_t b = rank_bucket(rank);
    const int32_t dc = b == 8 ? 1024 : b == 16 ? 512 : 256;
    const int32_t nchunks = (P.tv.d_in + dc - 1) / dc;
    return nchunks < P.KS ? nchunks : P.KS;
}

// ---------------------------------------------------------------------------------------------
// expand: each thread owns one 8-wide output column vector and up to four rows; v is read from
// shared memory (broadcast), B streams through once per group of rows.
// ---------------------------------------------------------------------------------------------
template <int NMG>
__device__ __forceinline__ void expand_rows(const ApplyParams &P, const Tile &tl,
                                            const int32_t *rowidx, const float *vsT) {
    constexpr int CVE = AP_THREADS / NMG, DCE = CVE * 8;
    const int tid = threadIdx.x;
    const int mg = tid / CVE, jv = tid % CVE;
    const int32_t d_out = P.tv.d_out, rows = tl.rows;
    const __nv_bfloat16 *B = P.pool.weights + (int64_t)tl.slot * P.pool.slot_stride + P.tv.off_b;
    const float s = tl.scale;

    for (int32_t j0 = (int32_t)blockIdx.y * DCE + jv * 8; j0 < d_out; j0 += P.JS * DCE) {
        for (int32_t m0 = 0; m0 < rows; m0 += NMG * 4) {
            const int32_t mb = m0 + mg * 4;
            if (mb >= rows) continue;
            uint4 ybv[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                ybv[i] = make_uint4(0, 0, 0, 0);
                if (mb + i < rows) ybv[i] = ldg16(P.yb + (int64_t)rowidx[mb + i] * P.ldyb + j0);
            }
            float acc[4][8];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int e = 0; e < 8; ++e) acc[i][e] = 0.0f;
#pragma unroll 4
            for (int32_t k = 0; k < tl.rank; ++k) {
                float bf[8];
                unpack8(ldg16(B + (int64_t)k * d_out + j0), bf);
                const float4 v4 = *reinterpret_cast<const float4 *>(vsT + k * ROWS_CAP + mb);
                const float vv[4] = {v4.x, v4.y, v4.z, v4.w};
#pragma unroll
                for (int i = 0; i < 4; ++i)
#pragma unroll
                    for (int e = 0; e < 8; ++e) acc[i][e] = fmaf(vv[i], bf[e], acc[i][e]);
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                if (mb + i >= rows) continue;
                float yf[8];
                unpack8(ybv[i], yf);
                uint4 o;
                o.x = pack2(fmaf(s, acc[i][0], yf[0]), fmaf(s, acc[i][1], yf[1]));
                o.y = pack2(fmaf(s, acc[i][2], yf[2]), fmaf(s, acc[i][3], yf[3]));
                o.z = pack2(fmaf(s, acc[i][4], yf[4]), fmaf(s, acc[i][5], yf[5]));
                o.w = pack2(fmaf(s, acc[i][6], yf[6]), fmaf(s, acc[i][7], yf[7]));
                *reinterpret_cast<uint4 *>(P.y + (int64_t)rowidx[mb + i] * P.ldy + j0) = o;
            }
        }
    }
}

// y_base -> y for rows that take no adapter (out-of-place calls only)
__device__ __forceinline__ void copy_rows(const ApplyParams &P, const int32_t *rowidx, int32_t rows) {
    const int32_t vecs = P.tv.d_out / 8;
    for (int32_t m = 0; m < rows; ++m) {
        const __nv_bfloat16 *src = P.yb + (int64_t)rowidx[m] * P.ldyb;
        __nv_bfloat16 *dst = P.y + (int64_t)rowidx[m] * P.ldy;
        for (int32_t v = blockIdx.y * AP_THREADS + threadIdx.x; v < vecs; v += P.JS * AP_THREADS)
            reinterpret_cast<uint4 *>(dst)[v] = ldg16(src + (int64_t)v * 8);
    }
}

__global__ void __launch_bounds__(AP_THREADS)
expand_kernel(const ApplyParams P) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float *vsT = reinterpret_cast<float *>(smem_raw);          // [rank][ROWS_CAP]
    int32_t *rowidx = reinterpret_cast<int32_t *>(smem_raw + 32 * 1024);
    MetaLayout L;
    if (P.meta) L = meta_layout(P.T, P.meta_slots, P.tile_m);
    const int tid = threadIdx.x;

    if ((int32_t)blockIdx.x >= P.units) {
        // copy blocks: 16 inactive rows each (grouped mode, out of place)
        const int32_t n_active = P.meta[H_NACTIVE];
        const int32_t first = ((int32_t)blockIdx.x - P.units) * 16;
        const int32_t rows = min(16, P.T - n_active - first);
        if (rows <= 0) return;
        if (tid < rows) rowidx[tid] = P.meta[L.perm + n_active + first + tid];
        __syncthreads();
        copy_rows(P, rowidx, rows);
        return;
    }
    const Tile tl = resolve_unit(P, L, blockIdx.x);
    if (!tl.valid) {
        if (!P.meta && (int32_t)blockIdx.x < P.T) {   // per-token mode: this token has no adapter
            if (blockIdx.y == 0 && tid == 0 && P.slot_idx[blockIdx.x] != -1)
                atomicAdd(&P.pool.status[STATUS_INVALID_TOKENS], 1);
            if (!P.in_place) {
                if (tid == 0) rowidx[0] = blockIdx.x;
                __syncthreads();
                copy_rows(P, rowidx, 1);
            }
        }
        return;
    }
    for (int i = tid; i < tl.rows; i += AP_THREADS)
        rowidx[i] = P.meta ? P.meta[L.perm + tl.row0 + i] : tl.row0 + i;
    // v = sum of the split-K partials, in order; rows past the tile's end read as zero
    const int32_t nval = valid_partials(P, tl.rank);
    const int32_t rows4 = (tl.rows + 3) & ~3;
    for (int i = tid; i < rows4 * tl.rank; i += AP_THREADS) {
        const int m = i / tl.rank, k = i % tl.rank;
        float v = 0.0f;
        if (m < tl.rows)
            for (int32_t q = 0; q < nval; ++q)
                v += P.ws[((int64_t)q * P.T + tl.row0 + m) * P.RS + k];
        vsT[k * ROWS_CAP + m] = v;
    }
    __syncthreads();
    if (tl.rows <= 4) expand_rows<1>(P, tl, rowidx, vsT);
    else if (tl.rows <= 8) expand_rows<2>(P, tl, rowidx, vsT);
    else expand_rows<4>(P, tl, rowidx, vsT);
}

// ---------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------
static inline int32_t next_pow2(int32_t v) {
    int32_t p = 1;
    while (p < v) p <<= 1;
    return p;
}

static bool ranges_overlap(const void *a, size_t na, const void *b, size_t nb) {
    const char *pa = (const char *)a, *pb = (const char *)b;
    return pa < pb + nb && pb < pa + na;
}

}  // namespace lora

using namespace lora;

namespace lora {
lora_status_t launch_build_segments(lora_pool_t *pool, const int32_t *slot_idx_dev, int32_t T,
                                    int32_t tile_m, int32_t long_min, void *meta_dev,
                                    cudaStream_t stream);

static lora_status_t check_apply_args(lora_pool_t *pool, int32_t target, const void *x, int64_t ldx,
                                      const void *yb, int64_t ldyb, void *y, int64_t ldy,
                                      int32_t T) {
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

static lora_status_t apply_common(lora_pool_t *pool, int32_t target, const void *x, int64_t ldx,
                                  const void *yb, int64_t ldyb, void *y, int64_t ldy,
                                  const int32_t *slot_idx_dev, int32_t T, const void *meta,
                                  int32_t tile_m, void *workspace, size_t workspace_bytes,
                                  cudaStream_t stream) {
    ApplyParams P;
    P.pool = pool->view();
    P.tv = pool->target_views[target];
    P.x = (const __nv_bfloat16 *)x;
    P.yb = (const __nv_bfloat16 *)yb;
    P.y = (__nv_bfloat16 *)y;
    P.ldx = ldx; P.ldyb = ldyb; P.ldy = ldy;
    P.slot_idx = slot_idx_dev;
    P.meta = (const int32_t *)meta;
    P.ws = (float *)workspace;
    P.T = T;
    P.RS = rank_bucket(pool->r_max);
    P.tile_m = tile_m;
    P.meta_slots = pool->num_slots;
    P.in_place = (y == yb);
    if (meta) {
        P.units = meta_layout(T, pool->num_slots, tile_m).cap_tile;
    } else {
        P.units = T;
    }
    if (P.units < 1) P.units = 1;
    const int32_t want = next_pow2((4 * pool->sm_count + P.units - 1) / P.units);
    int32_t KS = want < 8 ? want : 8;
    const size_t per_split = (size_t)T * P.RS * sizeof(float);
    while (KS > 1 && per_split * KS > workspace_bytes) KS >>= 1;
    if (per_split * KS > workspace_bytes || !workspace) return LORA_ERR_BUFFER_TOO_SMALL;
    if ((uintptr_t)workspace & 15) return LORA_ERR_INVALID_ARG;
    const int32_t max_ks = (P.tv.d_in + 255) / 256;
    while (KS > 1 && KS > max_ks) KS >>= 1;
    int32_t JS = want < 16 ? want : 16;
    const int32_t max_js = (P.tv.d_out + 511) / 512;
    while (JS > 1 && JS > max_js) JS >>= 1;
    P.KS = KS;
    P.JS = JS;

    static bool attr_done = false;
    if (!attr_done) {
        LORA_CUDA_TRY(cudaFuncSetAttribute(shrink_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           AP_SMEM_BYTES));
        LORA_CUDA_TRY(cudaFuncSetAttribute(expand_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           AP_SMEM_BYTES));
        attr_done = true;
    }
    shrink_kernel<<<dim3(P.units, KS), AP_THREADS, AP_SMEM_BYTES, stream>>>(P);
    lora_status_t s = count_launch();
    if (s != LORA_OK) return s;
    int32_t copy_blocks = 0;
    if (meta && !P.in_place) copy_blocks = (T + 15) / 16;
    expand_kernel<<<dim3(P.units + copy_blocks, JS), AP_THREADS, AP_SMEM_BYTES, stream>>>(P);
    return count_launch();
}
}  // namespace lora

extern "C" {

lora_status_t lora_workspace_bytes(const lora_pool_t *pool, int32_t T_max, size_t *bytes) {
    if (!pool || !bytes) return LORA_ERR_INVALID_ARG;
    if (T_max < 0) return LORA_ERR_SHAPE;
    *bytes = (size_t)8 * (size_t)(T_max > 0 ? T_max : 1) * rank_bucket(pool->r_max) * sizeof(float);
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
                        workspace, workspace_bytes, (cudaStream_t)stream);
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
                        workspace, workspace_bytes, (cudaStream_t)stream);
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
