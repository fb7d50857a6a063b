// Fused LoRA forward y = y_base + s_i * (x . A_i) . B_i (paper Section 2.2) in ONE launch.
//
// A thread-block cluster owns one unit (a row tile of one adapter, or one token).  Block c of
// the cluster takes the c-th slice of d_in for the shrink phase and the c-th slice of d_out for
// the expand phase:
//   1. the weight slices of both phases (A_i, B_i) are requested up front with bulk asynchronous
//      copies into shared memory, each signalled by an mbarrier; the y_base rows are prefetched
//      into L2; none of this depends on the shrink result, so its latency hides behind it;
//   2. shrink: fp32 partial v over the block's d_in slice (split-K, warp-shuffle reduction),
//      x rows read straight from global memory with 128-bit loads;
//   3. the partials are exchanged through distributed shared memory and summed in block order,
//      identically in every block (no global workspace, no float atomics);
//   4. expand over the block's d_out slice with the scale and the residual add fused, bf16 store.
// Blocks are kept small (128 threads, only the weight slices staged) so that many are resident
// per SM: a decode batch fits on the GPU in one wave and the hardware overlaps their latencies.
// Every per-row sum is taken in a fixed order that does not depend on which other rows share the
// tile, so a row's result depends only on its own inputs.
#include "apply_common.cuh"

namespace lora {

constexpr int FT = 128;   // threads per block of the fused kernel
#ifndef LORA_FUSED_MIN_BLOCKS
#define LORA_FUSED_MIN_BLOCKS 5   // resident blocks per SM the register budget is held to
#endif

// ---------------------------------------------------------------------------------------------
// PTX wrappers
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_mbar_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)),
                 "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// bounded wait: gives up after a fixed number of polls instead of spinning for ever
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity) {
    for (uint32_t i = 0; i < (1u << 20); ++i)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
// global -> this block's shared memory, completion counted in bytes on the mbarrier
__device__ __forceinline__ void bulk_g2s(void *dst, const void *src, uint32_t bytes, uint64_t *bar) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
            smem_u32(dst)),
        "l"(src), "r"(bytes), "r"(smem_u32(bar))
        : "memory");
}
__device__ __forceinline__ void prefetch_l2(const void *p) {
    asm volatile("prefetch.global.L2 [%0];" ::"l"(p));
}
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t cluster_nctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_arrive() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
}
__device__ __forceinline__ void cluster_wait() {
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// read a float at the same shared-memory offset in block `rank` of the cluster
__device__ __forceinline__ float ld_peer_f32(uint32_t local_addr, uint32_t rank) {
    uint32_t remote;
    float v;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_addr), "r"(rank));
    asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(remote) : "memory");
    return v;
}

enum { BAR_A = 0, BAR_B = 1, BAR_X = 2 };
constexpr int XROWS = 16;                // x rows staged at a time
constexpr int FUSED_HEAD_BYTES = 1024;   // mbarriers (64 B) + row indices (ROWS_CAP * 4 B)

// One warp requests `nrows` rows of `ncols` bf16 each; row r comes from src + r * src_pitch and
// lands at stage + r * pitch.
__device__ __forceinline__ void issue_rows(uint64_t *bar, __nv_bfloat16 *stage, int pitch, int nrows,
                                           int ncols, int lane, const __nv_bfloat16 *src,
                                           int64_t src_pitch) {
    if (lane == 0) mbar_expect_tx(bar, (uint32_t)nrows * (uint32_t)ncols * 2u);
    __syncwarp();
    for (int r = lane; r < nrows; r += 32)
        bulk_g2s(stage + r * pitch, src + (int64_t)r * src_pitch, (uint32_t)ncols * 2u, bar);
}
// the same for rows picked by an index list (token rows of a tile)
__device__ __forceinline__ void issue_gather(uint64_t *bar, __nv_bfloat16 *stage, int pitch, int nrows,
                                             int ncols, int lane, const __nv_bfloat16 *src,
                                             int64_t src_pitch, const int32_t *idx) {
    if (lane == 0) mbar_expect_tx(bar, (uint32_t)nrows * (uint32_t)ncols * 2u);
    __syncwarp();
    for (int r = lane; r < nrows; r += 32)
        bulk_g2s(stage + r * pitch, src + (int64_t)idx[r] * src_pitch, (uint32_t)ncols * 2u, bar);
}

// RP: rank bucket; DCA / DCB: columns of A / B staged at a time.
template <int RP, int DCA, int DCB>
__device__ __forceinline__ void fused_body(const ApplyParams &P, const Tile &tl, unsigned char *smem,
                                           uint32_t crank, uint32_t csize) {
    constexpr int CV = DCA / 8, KG = FT / CV, KPT = RP / KG, MG = 32 / KPT, WPK = CV / 32;
    constexpr int CVE = DCB / 8, NMG = FT / CVE, RPT = 4, EG = NMG * RPT;   // EG rows per expand pass
    constexpr int A_BYTES = RP * DCA * 2;
    static_assert(KPT * MG == 32 && WPK >= 1 && KG * KPT == RP, "shrink mapping");

    uint64_t *bars = reinterpret_cast<uint64_t *>(smem);
    const int32_t *rowidx = reinterpret_cast<const int32_t *>(smem + 64);
    float *part = reinterpret_cast<float *>(smem + P.off_part);
    float *vsT = reinterpret_cast<float *>(smem + P.off_vst);
    __nv_bfloat16 *As = reinterpret_cast<__nv_bfloat16 *>(smem + P.off_stage);
    __nv_bfloat16 *Bs = reinterpret_cast<__nv_bfloat16 *>(smem + P.off_stage + A_BYTES);
    __nv_bfloat16 *Xs = reinterpret_cast<__nv_bfloat16 *>(smem + P.off_x);   // [XROWS][DCA]

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int32_t d_in = P.tv.d_in, d_out = P.tv.d_out, rows = tl.rows, rank = tl.rank;
    const int32_t VSP = P.rows_cap;
    const __nv_bfloat16 *A = P.pool.weights + (int64_t)tl.slot * P.pool.slot_stride + P.tv.off_a;
    const __nv_bfloat16 *B = P.pool.weights + (int64_t)tl.slot * P.pool.slot_stride + P.tv.off_b;

    // this block's column slices (multiples of 8 columns)
    const int32_t Wa = (d_in + (int32_t)csize * 8 - 1) / ((int32_t)csize * 8) * 8;
    const int32_t a_lo = min((int32_t)crank * Wa, d_in), a_hi = min(a_lo + Wa, d_in);
    const int32_t na = (a_hi - a_lo + DCA - 1) / DCA;
    const int32_t Wb = (d_out + (int32_t)csize * 8 - 1) / ((int32_t)csize * 8) * 8;
    const int32_t b_lo = min((int32_t)crank * Wb, d_out), b_hi = min(b_lo + Wb, d_out);
    const int32_t nb = (b_hi - b_lo + DCB - 1) / DCB;

    // weight slices of both phases go out before any arithmetic
    if (warp == 0 && na > 0)
        issue_rows(&bars[BAR_A], As, DCA, rank, min(DCA, a_hi - a_lo), lane, A + a_lo, d_in);
    if (warp == 1 && nb > 0)
        issue_rows(&bars[BAR_B], Bs, DCB, rank, min(DCB, b_hi - b_lo), lane, B + b_lo, d_out);
    if (warp == 2 && na > 0)
        issue_gather(&bars[BAR_X], Xs, DCA, min(XROWS, rows), min(DCA, a_hi - a_lo), lane,
                     P.x + a_lo, P.ldx, rowidx);
    // pull this block's y_base columns towards L2 (128-byte lines); they are needed last
    if (b_hi > b_lo) {
        const int32_t lines = ((b_hi - b_lo) * 2 + 127) >> 7;
        for (int i = tid; i < rows * lines; i += FT) {
            const int m = i / lines, l = i - m * lines;
            prefetch_l2(reinterpret_cast<const char *>(P.yb + (int64_t)rowidx[m] * P.ldyb + b_lo) +
                        (l << 7));
        }
    }
    for (int i = tid; i < WPK * rows * RP; i += FT) part[i] = 0.0f;
    __syncthreads();

    uint32_t ph_a = 0, ph_b = 0, ph_x = 0;
    bool ok = true;

    // ---- shrink: thread = (column vector cv, rank group kg); KPT ranks x MG rows per reduction -
    {
        const int kg = tid / CV, cv = tid % CV, wk = cv >> 5;
        for (int32_t c = 0; c < na; ++c) {
            const int32_t col0 = a_lo + c * DCA, ncols = min(DCA, a_hi - col0);
            const bool cvalid = cv * 8 < ncols;
            if (c > 0 && warp == 0)
                issue_rows(&bars[BAR_A], As, DCA, rank, ncols, lane, A + col0, d_in);
            ok = mbar_wait(&bars[BAR_A], ph_a) && ok;
            ph_a ^= 1;
            for (int32_t m0 = 0; m0 < rows; m0 += MG) {
                if ((m0 % XROWS) == 0) {
                    // next XROWS rows of x: requested here unless it is the very first group,
                    // whose request went out at the start
                    if (c > 0 || m0 > 0) {
                        __syncthreads();   // everyone is done with the previous rows
                        if (warp == 2)
                            issue_gather(&bars[BAR_X], Xs, DCA, min(XROWS, rows - m0), ncols, lane,
                                         P.x + col0, P.ldx, rowidx + m0);
                    }
                    ok = mbar_wait(&bars[BAR_X], ph_x) && ok;
                    ph_x ^= 1;
                }
                float xf[MG][8];
#pragma unroll
                for (int mi = 0; mi < MG; ++mi) {
                    uint4 xv = make_uint4(0, 0, 0, 0);
                    if (cvalid && m0 + mi < rows)
                        xv = *reinterpret_cast<const uint4 *>(Xs + ((m0 % XROWS) + mi) * DCA + cv * 8);
                    unpack8(xv, xf[mi]);
                }
                float acc[32];
#pragma unroll
                for (int kk = 0; kk < KPT; ++kk) {
                    const int k = kg * KPT + kk;
                    uint4 w = make_uint4(0, 0, 0, 0);
                    if (cvalid && k < rank) w = *reinterpret_cast<const uint4 *>(As + k * DCA + cv * 8);
                    float af[8];
                    unpack8(w, af);
#pragma unroll
                    for (int mi = 0; mi < MG; ++mi) {
                        float s = 0.0f;
#pragma unroll
                        for (int e = 0; e < 8; ++e) s = fmaf(xf[mi][e], af[e], s);
                        acc[mi * KPT + kk] = s;
                    }
                }
                const float tot = warp_reduce32(acc, lane);
                const int mi = lane / KPT, kk = lane % KPT;
                if (m0 + mi < rows) part[(wk * rows + m0 + mi) * RP + kg * KPT + kk] += tot;
            }
            __syncthreads();   // the A stage is free
        }
    }
    if (WPK > 1) {
        for (int i = tid; i < rows * RP; i += FT) {
            float v = part[i];
#pragma unroll
            for (int w = 1; w < WPK; ++w) v += part[w * rows * RP + i];
            part[i] = v;
        }
    }
    // ---- exchange: every block sums all blocks' partials in block order -------------------------
    cluster_arrive();
    cluster_wait();
    {
        const uint32_t part_addr = smem_u32(part);
        const int32_t rows_pad = (rows + EG - 1) / EG * EG;
        for (int i = tid; i < rows_pad * rank; i += FT) {
            const int m = i / rank, k = i - m * rank;
            float v = 0.0f;
            if (m < rows)
                for (uint32_t q = 0; q < csize; ++q)
                    v += ld_peer_f32(part_addr + (uint32_t)(m * RP + k) * 4u, q);
            vsT[k * VSP + m] = v;
        }
    }
    cluster_arrive();   // done reading the peers; the matching wait is at the end
    __syncthreads();

    // ---- expand: thread = (output column vector jv, row group mg), RPT rows at a time ----------
    {
        const int mg = tid / CVE, jv = tid % CVE;
        const float s = tl.scale;
        for (int32_t c = 0; c < nb; ++c) {
            const int32_t col0 = b_lo + c * DCB, ncols = min(DCB, b_hi - col0);
            const bool cvalid = jv * 8 < ncols;
            if (c > 0 && warp == 1)
                issue_rows(&bars[BAR_B], Bs, DCB, rank, ncols, lane, B + col0, d_out);
            ok = mbar_wait(&bars[BAR_B], ph_b) && ok;
            ph_b ^= 1;
            for (int32_t m0 = 0; m0 < rows; m0 += EG) {
                const int32_t mb = m0 + mg * RPT;
                if (cvalid && mb < rows) {
                    uint4 ybv[RPT];
#pragma unroll
                    for (int i = 0; i < RPT; ++i) {
                        ybv[i] = make_uint4(0, 0, 0, 0);
                        if (mb + i < rows)
                            ybv[i] = ldg16(P.yb + (int64_t)rowidx[mb + i] * P.ldyb + col0 + jv * 8);
                    }
                    float acc[RPT][8];
#pragma unroll
                    for (int i = 0; i < RPT; ++i)
#pragma unroll
                        for (int e = 0; e < 8; ++e) acc[i][e] = 0.0f;
#pragma unroll 4
                    for (int32_t k = 0; k < rank; ++k) {
                        float bf[8];
                        unpack8(*reinterpret_cast<const uint4 *>(Bs + k * DCB + jv * 8), bf);
                        const float4 v4 = *reinterpret_cast<const float4 *>(vsT + k * VSP + mb);
                        const float vv[4] = {v4.x, v4.y, v4.z, v4.w};
#pragma unroll
                        for (int i = 0; i < RPT; ++i)
#pragma unroll
                            for (int e = 0; e < 8; ++e) acc[i][e] = fmaf(vv[i], bf[e], acc[i][e]);
                    }
                    if (ok) {
#pragma unroll
                        for (int i = 0; i < RPT; ++i)
                            if (mb + i < rows)
                                *reinterpret_cast<uint4 *>(P.y + (int64_t)rowidx[mb + i] * P.ldy + col0 +
                                                           jv * 8) = finish8(acc[i], ybv[i], s);
                    }
                }
            }
            __syncthreads();   // the B stage is free
        }
    }
    if (!ok && tid == 0) atomicAdd(&P.pool.status[STATUS_TIMEOUTS], 1);
    cluster_wait();   // no block leaves while a peer may still read its partials
}

__global__ void __launch_bounds__(FT, LORA_FUSED_MIN_BLOCKS)
fused_kernel(const ApplyParams P) {
    extern __shared__ __align__(128) unsigned char smem[];
    const uint32_t csize = cluster_nctarank(), crank = cluster_ctarank();
    const int32_t unit = (int32_t)(blockIdx.x / csize);
    const int tid = threadIdx.x;
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem);
    int32_t *rowidx = reinterpret_cast<int32_t *>(smem + 64);
    MetaLayout L;
    if (P.meta) L = meta_layout(P.T, P.meta_slots, P.tile_m);

    if (unit >= P.units) {
        // copy clusters: 16 rows without an adapter each (grouped mode, out of place)
        const int32_t n_active = P.meta[H_NACTIVE];
        const int32_t first = (unit - P.units) * 16;
        const int32_t rows = min(16, P.T - n_active - first);
        if (rows <= 0) return;
        if (tid < rows) rowidx[tid] = P.meta[L.perm + n_active + first + tid];
        __syncthreads();
        copy_rows(P, rowidx, rows, (int32_t)crank, (int32_t)csize);
        return;
    }
    // the tile record and the tile's row ids are fetched side by side (no dependent load)
    if (P.meta) {
        if (tid < P.tile_m) rowidx[tid] = P.meta[L.tile_perm + (int64_t)unit * P.tile_m + tid];
    } else if (tid == 0) {
        rowidx[0] = unit;
    }
    // the tile count sits in one word that every block reads (L2-hot): unused units leave on it
    const int32_t n_tile = P.meta ? __ldg(P.meta + H_NTILE) : P.T;
    const Tile tl = resolve_unit(P, L, unit);
    if (unit >= n_tile) return;
    if (!tl.valid) {
        if (!P.meta && unit < P.T) {   // per-token mode: this token has no adapter
            if (crank == 0 && tid == 0 && P.slot_idx[unit] != -1)
                atomicAdd(&P.pool.status[STATUS_INVALID_TOKENS], 1);
            if (!P.in_place) {
                __syncthreads();
                copy_rows(P, rowidx, 1, (int32_t)crank, (int32_t)csize);
            }
        }
        return;
    }
    if (tid == 0) {
        mbar_init(&bars[BAR_A], 1);
        mbar_init(&bars[BAR_B], 1);
        mbar_init(&bars[BAR_X], 1);
        fence_mbar_init();
    }
    __syncthreads();
    const int32_t b = rank_bucket(tl.rank);
    if (b <= 16) fused_body<16, 512, 512>(P, tl, smem, crank, csize);
    else if (b == 32) fused_body<32, 256, 256>(P, tl, smem, crank, csize);
    else fused_body<64, 256, 256>(P, tl, smem, crank, csize);
}

// shared memory for the two weight stages, for pools whose largest rank bucket is RS
static int32_t stage_bytes_for(int32_t RS) {
    const int32_t b16 = 2 * 16 * 512 * 2, b32 = 2 * 32 * 256 * 2, b64 = 2 * 64 * 256 * 2;
    return RS <= 16 ? b16 : RS == 32 ? (b16 > b32 ? b16 : b32) : b64;
}

lora_status_t launch_fused(lora_pool_t *pool, ApplyParams &P, cudaStream_t stream) {
    const int32_t RS = P.RS < 16 ? 16 : P.RS;
    int32_t rows_cap = P.meta ? P.tile_m : 1;
    rows_cap = (rows_cap + 15) & ~15;
    P.rows_cap = rows_cap;
    // partial v: WPK copies of [rows][RP]; WPK * RP is 32 for the <=16 bucket, RP above
    const int32_t part_floats_per_row = RS == 16 ? 32 : RS;
    P.off_part = FUSED_HEAD_BYTES;
    P.off_vst = P.off_part + rows_cap * part_floats_per_row * 4;
    P.off_stage = (P.off_vst + RS * rows_cap * 4 + 127) & ~127;
    P.off_x = P.off_stage + stage_bytes_for(RS);
    int32_t x_rows = ((P.meta ? P.tile_m : 1) + 7) & ~7;
    if (x_rows > XROWS) x_rows = XROWS;
    const int32_t smem = P.off_x + x_rows * 512 * 2;   // x stage: up to XROWS rows of 512 columns

    // cluster size: as wide a split as the projection supports, narrower when there are many units
    int32_t C = pool->tuning[1];
    if (C != 1 && C != 2 && C != 4 && C != 8) {
        C = 8;
        while (C > 1 && (P.tv.d_in / C < 256 || P.tv.d_out / C < 128)) C >>= 1;
        while (C > 1 && (int64_t)P.units * C > (int64_t)16 * pool->sm_count) C >>= 1;
    }
    int32_t copy_units = 0;
    if (P.meta && !P.in_place) copy_units = (P.T + 15) / 16;

    static int32_t attr_smem = 0;
    if (smem > attr_smem) {
        LORA_CUDA_TRY(cudaFuncSetAttribute(fused_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           smem));
        attr_smem = smem;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)((P.units + copy_units) * C), 1, 1);
    cfg.blockDim = dim3(FT, 1, 1);
    cfg.dynamicSmemBytes = (size_t)smem;
    cfg.stream = stream;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = (unsigned)C;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    LORA_CUDA_TRY(cudaLaunchKernelEx(&cfg, fused_kernel, P));
    return count_launch();
}

}  // namespace lora
