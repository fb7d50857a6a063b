// Fused LoRA forward y = y_base + s_i * (x . A_i) . B_i (paper Section 2.2) in ONE launch.
//
// A thread-block cluster owns one unit (a row tile of one adapter, or one token).  Block c of
// the cluster takes the c-th slice of d_in for the shrink phase and the c-th slice of d_out for
// the expand phase:
//   1. all operands of both phases (A_i slice, x rows, B_i slice, y_base rows) are requested up
//      front with bulk asynchronous copies into shared memory, each group signalled by an mbarrier;
//      the expand operands do not depend on the shrink result, so their latency hides behind it;
//   2. shrink: fp32 partial v over the block's d_in slice (split-K, warp-shuffle reduction);
//   3. the partials are exchanged through distributed shared memory and summed in block order,
//      identically in every block (no global workspace, no float atomics);
//   4. expand over the block's d_out slice with the scale and the residual add fused, bf16 store.
// Every per-row sum is taken in a fixed order that does not depend on which other rows share the
// tile, so a row's result depends only on its own inputs.
#include "apply_common.cuh"

namespace lora {

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

enum { BAR_A = 0, BAR_X = 1, BAR_B = 2, BAR_Y = 3 };
constexpr int FUSED_HEAD_BYTES = 1024;   // mbarriers (64 B) + row indices (ROWS_CAP * 4 B)

// One warp requests `nrows` rows of `ncols` bf16 each; row r comes from src(r) and lands at
// stage + r * pitch.
template <typename SrcFn>
__device__ __forceinline__ void issue_rows(uint64_t *bar, __nv_bfloat16 *stage, int pitch, int nrows,
                                           int ncols, int lane, SrcFn src) {
    if (lane == 0) mbar_expect_tx(bar, (uint32_t)nrows * (uint32_t)ncols * 2u);
    __syncwarp();
    for (int r = lane; r < nrows; r += 32) bulk_g2s(stage + r * pitch, src(r), (uint32_t)ncols * 2u, bar);
}

template <int RP, int KPT, int CVE>
__device__ __forceinline__ void fused_body(const ApplyParams &P, const Tile &tl, unsigned char *smem,
                                           uint32_t crank, uint32_t csize) {
    constexpr int KG = RP / KPT, CV = AP_THREADS / KG, DCA = CV * 8, WPK = CV / 32, MG = 32 / KPT;
    constexpr int NMG = AP_THREADS / CVE, RPT = 16 / NMG, DCB = CVE * 8;
    constexpr int A_BYTES = RP * DCA * 2, X_BYTES = 16 * DCA * 2, B_BYTES = RP * DCB * 2;
    static_assert(MG <= 16 && RPT >= 1, "mapping");

    uint64_t *bars = reinterpret_cast<uint64_t *>(smem);
    const int32_t *rowidx = reinterpret_cast<const int32_t *>(smem + 64);
    float *part = reinterpret_cast<float *>(smem + P.off_part);
    float *vsT = reinterpret_cast<float *>(smem + P.off_vst);
    __nv_bfloat16 *As = reinterpret_cast<__nv_bfloat16 *>(smem + P.off_stage);
    __nv_bfloat16 *Xs = reinterpret_cast<__nv_bfloat16 *>(smem + P.off_stage + A_BYTES);
    __nv_bfloat16 *Bs = reinterpret_cast<__nv_bfloat16 *>(smem + P.off_stage + A_BYTES + X_BYTES);
    __nv_bfloat16 *Ys =
        reinterpret_cast<__nv_bfloat16 *>(smem + P.off_stage + A_BYTES + X_BYTES + B_BYTES);

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
    const int32_t nsub = (rows + 15) >> 4;

    auto issue_A = [&](int32_t c) {
        const int32_t col0 = a_lo + c * DCA, ncols = min(DCA, a_hi - col0);
        issue_rows(&bars[BAR_A], As, DCA, rank, ncols, lane,
                   [&](int r) { return A + (int64_t)r * d_in + col0; });
    };
    auto issue_X = [&](int32_t sub, int32_t c) {
        const int32_t col0 = a_lo + c * DCA, ncols = min(DCA, a_hi - col0);
        const int32_t m0 = sub * 16, nrows = min(16, rows - m0);
        issue_rows(&bars[BAR_X], Xs, DCA, nrows, ncols, lane,
                   [&](int r) { return P.x + (int64_t)rowidx[m0 + r] * P.ldx + col0; });
    };
    auto issue_B = [&](int32_t c) {
        const int32_t col0 = b_lo + c * DCB, ncols = min(DCB, b_hi - col0);
        issue_rows(&bars[BAR_B], Bs, DCB, rank, ncols, lane,
                   [&](int r) { return B + (int64_t)r * d_out + col0; });
    };
    auto issue_Y = [&](int32_t sub, int32_t c) {
        const int32_t col0 = b_lo + c * DCB, ncols = min(DCB, b_hi - col0);
        const int32_t m0 = sub * 16, nrows = min(16, rows - m0);
        issue_rows(&bars[BAR_Y], Ys, DCB, nrows, ncols, lane,
                   [&](int r) { return P.yb + (int64_t)rowidx[m0 + r] * P.ldyb + col0; });
    };

    // first requests of both phases go out before any arithmetic
    if (warp == 0 && na > 0) { issue_A(0); issue_X(0, 0); }
    if (warp == 1 && nb > 0) { issue_B(0); issue_Y(0, 0); }
    for (int i = tid; i < WPK * rows * RP; i += AP_THREADS) part[i] = 0.0f;
    __syncthreads();

    uint32_t ph_a = 0, ph_x = 0, ph_b = 0, ph_y = 0;
    bool ok = true;

    // ---- shrink -------------------------------------------------------------------------------
    {
        const int kg = tid / CV, cv = tid % CV, wk = cv >> 5;
        for (int32_t c = 0; c < na; ++c) {
            const int32_t ncols = min(DCA, a_hi - (a_lo + c * DCA));
            const bool cvalid = cv * 8 < ncols;
            if (c > 0 && warp == 0) issue_A(c);
            ok = mbar_wait(&bars[BAR_A], ph_a) && ok;
            ph_a ^= 1;
            float a[KPT][8];
#pragma unroll
            for (int kk = 0; kk < KPT; ++kk) {
                const int k = kg * KPT + kk;
                uint4 w = make_uint4(0, 0, 0, 0);
                if (cvalid && k < rank) w = *reinterpret_cast<const uint4 *>(As + k * DCA + cv * 8);
                unpack8(w, a[kk]);
            }
            for (int32_t sub = 0; sub < nsub; ++sub) {
                if ((c > 0 || sub > 0) && warp == 0) issue_X(sub, c);
                ok = mbar_wait(&bars[BAR_X], ph_x) && ok;
                ph_x ^= 1;
                const int32_t m0 = sub * 16, nrows = min(16, rows - m0);
#pragma unroll
                for (int g = 0; g < 16; g += MG) {
                    if (g < nrows) {
                        float acc[32];
#pragma unroll
                        for (int mi = 0; mi < MG; ++mi) {
                            uint4 xv = make_uint4(0, 0, 0, 0);
                            if (cvalid && g + mi < nrows)
                                xv = *reinterpret_cast<const uint4 *>(Xs + (g + mi) * DCA + cv * 8);
                            float xf[8];
                            unpack8(xv, xf);
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
                        if (g + mi < nrows)
                            part[(wk * rows + m0 + g + mi) * RP + kg * KPT + kk] += tot;
                    }
                }
                __syncthreads();   // the x stage (and after the last sub-tile the A stage) is free
            }
        }
    }
    if (WPK > 1) {
        for (int i = tid; i < rows * RP; i += AP_THREADS) {
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
        const int32_t rows16 = (rows + 15) & ~15;
        for (int i = tid; i < rows16 * rank; i += AP_THREADS) {
            const int m = i / rank, k = i % rank;
            float v = 0.0f;
            if (m < rows)
                for (uint32_t q = 0; q < csize; ++q)
                    v += ld_peer_f32(part_addr + (uint32_t)(m * RP + k) * 4u, q);
            vsT[k * VSP + m] = v;
        }
    }
    cluster_arrive();   // done reading the peers; the matching wait is at the end
    __syncthreads();

    // ---- expand -------------------------------------------------------------------------------
    {
        const int mg = tid / CVE, jv = tid % CVE;
        const float s = tl.scale;
        for (int32_t c = 0; c < nb; ++c) {
            const int32_t col0 = b_lo + c * DCB, ncols = min(DCB, b_hi - col0);
            const bool cvalid = jv * 8 < ncols;
            if (c > 0 && warp == 1) issue_B(c);
            ok = mbar_wait(&bars[BAR_B], ph_b) && ok;
            ph_b ^= 1;
            for (int32_t sub = 0; sub < nsub; ++sub) {
                if ((c > 0 || sub > 0) && warp == 1) issue_Y(sub, c);
                ok = mbar_wait(&bars[BAR_Y], ph_y) && ok;
                ph_y ^= 1;
                const int32_t m0 = sub * 16, nrows = min(16, rows - m0);
                const int32_t ml = mg * RPT;   // first local row of this thread
                if (cvalid && ml < nrows) {
                    float acc[RPT][8];
#pragma unroll
                    for (int i = 0; i < RPT; ++i)
#pragma unroll
                        for (int e = 0; e < 8; ++e) acc[i][e] = 0.0f;
#pragma unroll 4
                    for (int32_t k = 0; k < rank; ++k) {
                        float bf[8];
                        unpack8(*reinterpret_cast<const uint4 *>(Bs + k * DCB + jv * 8), bf);
                        float vv[RPT];
                        if (RPT == 4) {
                            const float4 v4 =
                                *reinterpret_cast<const float4 *>(vsT + k * VSP + m0 + ml);
                            vv[0] = v4.x; vv[1] = v4.y; vv[2 % RPT] = v4.z; vv[3 % RPT] = v4.w;
                        } else {
                            const float2 v2 =
                                *reinterpret_cast<const float2 *>(vsT + k * VSP + m0 + ml);
                            vv[0] = v2.x; vv[1 % RPT] = v2.y;
                        }
#pragma unroll
                        for (int i = 0; i < RPT; ++i)
#pragma unroll
                            for (int e = 0; e < 8; ++e) acc[i][e] = fmaf(vv[i], bf[e], acc[i][e]);
                    }
                    if (ok) {
#pragma unroll
                        for (int i = 0; i < RPT; ++i) {
                            if (ml + i < nrows) {
                                const uint4 ybv =
                                    *reinterpret_cast<const uint4 *>(Ys + (ml + i) * DCB + jv * 8);
                                *reinterpret_cast<uint4 *>(P.y + (int64_t)rowidx[m0 + ml + i] * P.ldy +
                                                           col0 + jv * 8) = finish8(acc[i], ybv, s);
                            }
                        }
                    }
                }
                __syncthreads();   // the y_base stage (and after the last sub-tile the B stage) is free
            }
        }
    }
    if (!ok && tid == 0) atomicAdd(&P.pool.status[STATUS_TIMEOUTS], 1);
    cluster_wait();   // no block leaves while a peer may still read its partials
}

__global__ void __launch_bounds__(AP_THREADS, 2)
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
    const Tile tl = resolve_unit(P, L, unit);
    if (!tl.valid) {
        if (!P.meta && unit < P.T) {   // per-token mode: this token has no adapter
            if (crank == 0 && tid == 0 && P.slot_idx[unit] != -1)
                atomicAdd(&P.pool.status[STATUS_INVALID_TOKENS], 1);
            if (!P.in_place) {
                if (tid == 0) rowidx[0] = unit;
                __syncthreads();
                copy_rows(P, rowidx, 1, (int32_t)crank, (int32_t)csize);
            }
        }
        return;
    }
    if (tid == 0) {
#pragma unroll
        for (int i = 0; i < 4; ++i) mbar_init(&bars[i], 1);
        fence_mbar_init();
    }
    for (int i = tid; i < tl.rows; i += AP_THREADS)
        rowidx[i] = P.meta ? P.meta[L.perm + tl.row0 + i] : tl.row0 + i;
    __syncthreads();
    switch (rank_bucket(tl.rank)) {
        case 8: fused_body<8, 2, 64>(P, tl, smem, crank, csize); break;
        case 16: fused_body<16, 4, 64>(P, tl, smem, crank, csize); break;
        case 32: fused_body<32, 4, 64>(P, tl, smem, crank, csize); break;
        default: fused_body<64, 8, 32>(P, tl, smem, crank, csize); break;
    }
}

// shared memory the kernel needs for pools whose largest rank bucket is RS
static int32_t stage_bytes_for(int32_t RS) {
    // per bucket: A + X + B + YB stages (see fused_body)
    const int32_t b8 = 8 * 512 * 2 + 16 * 512 * 2 + 8 * 512 * 2 + 16 * 512 * 2;
    const int32_t b16 = 16 * 512 * 2 + 16 * 512 * 2 + 16 * 512 * 2 + 16 * 512 * 2;
    const int32_t b32 = 32 * 256 * 2 + 16 * 256 * 2 + 32 * 512 * 2 + 16 * 512 * 2;
    const int32_t b64 = 64 * 256 * 2 + 16 * 256 * 2 + 64 * 256 * 2 + 16 * 256 * 2;
    int32_t m = b8;
    if (RS >= 16 && b16 > m) m = b16;
    if (RS >= 32 && b32 > m) m = b32;
    if (RS >= 64 && b64 > m) m = b64;
    return m;
}

lora_status_t launch_fused(lora_pool_t *pool, ApplyParams &P, cudaStream_t stream) {
    const int32_t RS = P.RS;
    int32_t rows_cap = P.meta ? P.tile_m : 1;
    rows_cap = (rows_cap + 15) & ~15;
    P.rows_cap = rows_cap;
    const int32_t part_floats_per_row = RS == 8 ? 16 : RS == 16 ? 32 : RS;   // WPK * RP, worst bucket
    P.off_part = FUSED_HEAD_BYTES;
    P.off_vst = P.off_part + rows_cap * part_floats_per_row * 4;
    P.off_stage = (P.off_vst + RS * rows_cap * 4 + 127) & ~127;
    const int32_t smem = P.off_stage + stage_bytes_for(RS);

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
    cfg.blockDim = dim3(AP_THREADS, 1, 1);
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
