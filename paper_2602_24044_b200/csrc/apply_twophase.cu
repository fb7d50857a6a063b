// Two-phase LoRA forward on CUDA cores with a global fp32 workspace between the phases:
//   shrink  v[t, 0:r] = x[t, :] . A_i      split over d_in across blocks (split-K), fp32
//   expand  y[t, :]   = bf16( y_base[t, :] + s_i * (v[t, :] . B_i) )
// (paper Section 2.2: the adapter's two low-rank matrices produce activations that are added to
// the backbone layer's output).  Two launches; operands are read straight from global memory.
// Selected with tuning key 0 = 1; the default path is the fused kernel in apply_fused.cu.
#include "apply_common.cuh"

namespace lora {

constexpr int TP_SMEM_BYTES = 32 * 1024 + ROWS_CAP * 4;

// shrink: each thread owns one 8-wide column vector of the chunk and KPT ranks; A stays in
// registers for the whole tile, rows of x stream through; 32 partial sums at a time are folded
// across the warp.
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

// expand: each thread owns one 8-wide output column vector and up to four rows; v is read from
// shared memory (broadcast), B streams through once per group of rows.
template <int NMG>
__device__ __forceinline__ void expand_rows(const ApplyParams &P, const Tile &tl,
                                            const int32_t *rowidx, const float *vsT) {
    constexpr int CVE = AP_THREADS / NMG, DCE = CVE * 8;
    const int tid = threadIdx.x;
    const int mg = tid / CVE, jv = tid % CVE;
    const int32_t d_out = P.tv.d_out, rows = tl.rows;
    const __nv_bfloat16 *B = P.pool.weights + (int64_t)tl.slot * P.pool.slot_stride + P.tv.off_b;

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
                *reinterpret_cast<uint4 *>(P.y + (int64_t)rowidx[mb + i] * P.ldy + j0) =
                    finish8(acc[i], ybv[i], tl.scale);
            }
        }
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
        copy_rows(P, rowidx, rows, blockIdx.y, P.JS);
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
                copy_rows(P, rowidx, 1, blockIdx.y, P.JS);
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

lora_status_t launch_twophase(lora_pool_t *pool, ApplyParams &P, void *workspace,
                              size_t workspace_bytes, cudaStream_t stream) {
    const int32_t T = P.T;
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
    P.ws = (float *)workspace;

    bool &attr_done = pool->twophase_attr_done;
    if (!attr_done) {
        LORA_CUDA_TRY(cudaFuncSetAttribute(shrink_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           TP_SMEM_BYTES));
        LORA_CUDA_TRY(cudaFuncSetAttribute(expand_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           TP_SMEM_BYTES));
        attr_done = true;
    }
    shrink_kernel<<<dim3(P.units, KS), AP_THREADS, TP_SMEM_BYTES, stream>>>(P);
    lora_status_t s = count_launch();
    if (s != LORA_OK) return s;
    int32_t copy_blocks = 0;
    if (P.meta && !P.in_place) copy_blocks = (T + 15) / 16;
    expand_kernel<<<dim3(P.units + copy_blocks, JS), AP_THREADS, TP_SMEM_BYTES, stream>>>(P);
    return count_launch();
}

}  // namespace lora
