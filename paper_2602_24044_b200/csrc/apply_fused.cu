// Fused LoRA forward y = y_base + s_i * (x . A_i) . B_i (paper Section 2.2) in ONE launch.
//
// A thread-block cluster owns one unit (a row tile of one adapter, or one token).  Block c of
// the cluster takes the c-th slice of d_in for the shrink phase and the c-th slice of d_out for
// the expand phase:
//   1. everything the block will read is requested before any arithmetic: the A_i and B_i slices
//      and the tile's x rows by bulk asynchronous copies into shared memory (mbarrier-signalled),
//      the y_base rows by loads into registers; none of the expand operands depends on the shrink
//      result, so their latency hides behind it;
//   2. shrink: partial v over the block's d_in slice, split-K over the four warps, bf16 tensor-core
//      MMA with fp32 accumulation;
//   3. the partials are exchanged through distributed shared memory and summed in block order,
//      identically in every block (no global workspace, no float atomics);
//   4. expand over the block's d_out slice on the tensor cores, v carried as the sum of two bf16
//      numbers (high and low part) so that it keeps ~16 mantissa bits; scale and residual add fused,
//      one rounding to bf16 at the store.
// Blocks are small (128 threads, ~44 KB of shared memory for decode tiles) so that many are
// resident per SM: a decode batch fits on the GPU in one wave and the hardware overlaps their
// latencies.  Every per-row sum is taken in a fixed order that does not depend on which other
// rows share the tile (MMA rows are independent), so a row's result depends only on its inputs.
#include <cstdio>
#include <cstdlib>

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
// D += A(16x16, row) . B(16x8, col), bf16 inputs, fp32 accumulate
__device__ __forceinline__ void mma16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0,
                                         uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// four 8x8 b16 matrices, transposed on the way in (rows of shared memory become MMA columns)
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
// programmatic dependent launch: let the next kernel of the stream be scheduled / wait until all
// work queued before this kernel is complete and visible (a no-op without the launch attribute)
__device__ __forceinline__ void griddep_launch_dependents() {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
__device__ __forceinline__ void griddep_wait() {
    asm volatile("griddepcontrol.wait;" ::: "memory");
}
__device__ __forceinline__ uint32_t lds32(const __nv_bfloat16 *p) {
    return *reinterpret_cast<const uint32_t *>(p);
}

enum { BAR_A = 0, BAR_B = 1, BAR_X0 = 2, BAR_X1 = 3 };

// One warp requests `nrows` rows of `ncols` bf16 each; row r comes from src + r * src_pitch (or
// src + idx[r] * src_pitch) and lands at stage + r * pitch.
__device__ __forceinline__ void issue_rows(uint64_t *bar, __nv_bfloat16 *stage, int pitch, int nrows,
                                           int ncols, int lane, const __nv_bfloat16 *src,
                                           int64_t src_pitch, const int32_t *idx) {
    if (lane == 0) mbar_expect_tx(bar, (uint32_t)nrows * (uint32_t)ncols * 2u);
    __syncwarp();
    for (int r = lane; r < nrows; r += 32)
        bulk_g2s(stage + r * pitch, src + (int64_t)(idx ? idx[r] : r) * src_pitch,
                 (uint32_t)ncols * 2u, bar);
}

// RP: rank bucket (16, 32, 64); DCA / DCB: columns of A / B staged at a time.
// H: 1 when a row tile holds at most 8 rows (decode tiles), 2 when rows 8..15 can be occupied.
template <int RP, int DCA, int DCB, int H>
__device__ __forceinline__ void fused_body(const ApplyParams &P, const Tile &tl, unsigned char *smem,
                                           uint32_t crank, uint32_t csize, uint32_t (&ph)[4]) {
    constexpr int PA = DCA + 8, PB = DCB + 8;   // shared-memory row pitches: +16 B against bank conflicts
    constexpr int PV = RP + 8;                  // pitch of the bf16 copies of v
    constexpr int NT_S = RP / 8;                // rank tiles of 8 in the shrink MMA
    constexpr int KW = DCA / 4, NW = DCB / 4;   // columns per warp: shrink (split-K), expand
    constexpr int NPASS = NW / 64;              // expand passes of 64 columns per warp
    constexpr int A_BYTES = RP * PA * 2;
    static_assert(NPASS >= 1 && KW % 16 == 0, "mapping");

    uint64_t *bars = reinterpret_cast<uint64_t *>(smem);
    const int32_t *rowidx = reinterpret_cast<const int32_t *>(smem + 64);
    float *part = reinterpret_cast<float *>(smem + P.off_part);     // [4 warps][mrows][RP]
    float *vpart = reinterpret_cast<float *>(smem + P.off_vpart);   // [rows][RP], read by the peers
    __nv_bfloat16 *Vh = reinterpret_cast<__nv_bfloat16 *>(smem + P.off_vh);   // [rows][PV]
    __nv_bfloat16 *Vl = reinterpret_cast<__nv_bfloat16 *>(smem + P.off_vl);
    __nv_bfloat16 *As = reinterpret_cast<__nv_bfloat16 *>(smem + P.off_stage);            // [RP][PA]
    __nv_bfloat16 *Bs = reinterpret_cast<__nv_bfloat16 *>(smem + P.off_stage + A_BYTES);  // [RP][PB]
    __nv_bfloat16 *Xs = reinterpret_cast<__nv_bfloat16 *>(smem + P.off_x);   // [xbufs][mrows][520]
    constexpr int PX = 520;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, t = lane & 3;
    const int32_t d_in = P.tv.d_in, d_out = P.tv.d_out, rows = tl.rows, rank = tl.rank;
    const int32_t rank16 = (rank + 15) & ~15;
    constexpr int32_t mrows = 8 * H;
    constexpr bool hi_rows = H == 2;   // rows 8..15 of a row tile can be occupied
    const int32_t n_mt = (rows + 15) >> 4;
    const __nv_bfloat16 *A = P.pool.weights + (int64_t)tl.slot * P.pool.slot_stride + P.tv.off_a;
    const __nv_bfloat16 *B = P.pool.weights + (int64_t)tl.slot * P.pool.slot_stride + P.tv.off_b;

    // this block's column slices (multiples of 8 columns)
    const int32_t Wa = (d_in + (int32_t)csize * 8 - 1) / ((int32_t)csize * 8) * 8;
    const int32_t a_lo = min((int32_t)crank * Wa, d_in), a_hi = min(a_lo + Wa, d_in);
    const int32_t na = (a_hi - a_lo + DCA - 1) / DCA;
    const int32_t Wb = (d_out + (int32_t)csize * 8 - 1) / ((int32_t)csize * 8) * 8;
    const int32_t b_lo = min((int32_t)crank * Wb, d_out), b_hi = min(b_lo + Wb, d_out);
    const int32_t nb = (b_hi - b_lo + DCB - 1) / DCB;
    const int32_t n_items = na * n_mt;   // (column chunk, row tile) pairs of the shrink phase

    auto issue_x = [&](int32_t it, int buf) {
        const int32_t c = it / n_mt, mt = it - c * n_mt;
        const int32_t col0 = a_lo + c * DCA;
        issue_rows(&bars[BAR_X0 + buf], Xs + buf * mrows * PX, PX, min(mrows, rows - mt * 16),
                   min(DCA, a_hi - col0), lane, P.x + col0, P.ldx, rowidx + mt * 16);
    };
    // y_base of one (chunk, row tile, pass) in the MMA accumulator layout: [column tile of 8][row
    // g / g+8], two adjacent columns (2t, 2t+1) per word
    auto load_yb = [&](uint32_t (&ybw)[8][H], int32_t c, int32_t mt, int p) {
        const int32_t col0 = b_lo + c * DCB, ncols = min(DCB, b_hi - col0);
#pragma unroll
        for (int h = 0; h < H; ++h) {
            const int32_t m = mt * 16 + g + 8 * h;
            const __nv_bfloat16 *row = P.yb + (int64_t)rowidx[m < rows ? m : 0] * P.ldyb + col0 + 2 * t;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int32_t col = warp * NW + p * 64 + j * 8;
                ybw[j][h] = 0u;
                if (m < rows && col < ncols)
                    ybw[j][h] = __ldg(reinterpret_cast<const uint32_t *>(row + col));
            }
        }
    };

    // ---- everything this block reads is requested here ------------------------------------------
    if (warp == 0 && na > 0)
        issue_rows(&bars[BAR_A], As, PA, rank, min(DCA, a_hi - a_lo), lane, A + a_lo, d_in, nullptr);
    if (warp == 1 && nb > 0)
        issue_rows(&bars[BAR_B], Bs, PB, rank, min(DCB, b_hi - b_lo), lane, B + b_lo, d_out, nullptr);
    if (warp == 2 && n_items > 0) issue_x(0, 0);
    if (warp == 3) {
        // rows rank .. rank16-1 of the B stage are multiplied by zeros of v: make them finite
        const int32_t vec_per_row = PB / 8;
        for (int i = lane; i < (rank16 - rank) * vec_per_row; i += 32)
            reinterpret_cast<uint4 *>(Bs + (rank + i / vec_per_row) * PB)[i % vec_per_row] =
                make_uint4(0, 0, 0, 0);
    }
    // y_base of the first row tile is requested into registers now (it is used last); for tiles
    // with more row tiles the rest is pulled towards L2 (128-byte lines)
    uint32_t ybw[NPASS][8][H];
    if (nb > 0) load_yb(ybw[0], 0, 0, 0);
    if (rows > 16 && b_hi > b_lo) {
        const int32_t lines = ((b_hi - b_lo) * 2 + 127) >> 7;
        for (int i = tid; i < (rows - 16) * lines; i += FT) {
            const int m = 16 + i / lines, l = i % lines;
            prefetch_l2(reinterpret_cast<const char *>(P.yb + (int64_t)rowidx[m] * P.ldyb + b_lo) +
                        (l << 7));
        }
    }

    // mbarrier phase bits live across the units a block processes
    uint32_t &ph_a = ph[BAR_A], &ph_b = ph[BAR_B], &ph_x0 = ph[BAR_X0], &ph_x1 = ph[BAR_X1];
    bool ok = true;

    // ---- shrink: warp w takes columns [w*KW, (w+1)*KW) of the staged chunk (split-K) ------------
    for (int32_t it = 0; it < n_items; ++it) {
        const int32_t c = it / n_mt, mt = it - c * n_mt;
        const int32_t ncols = min(DCA, a_hi - (a_lo + c * DCA));
        if (mt == 0) {
            if (c > 0 && warp == 0)
                issue_rows(&bars[BAR_A], As, PA, rank, ncols, lane, A + a_lo + c * DCA, d_in, nullptr);
            ok = mbar_wait(&bars[BAR_A], ph_a) && ok;
            ph_a ^= 1;
        }
        int buf = 0;
        if (P.xbufs == 2) {
            buf = it & 1;
            if (it + 1 < n_items && warp == 2) issue_x(it + 1, buf ^ 1);
        } else if (it > 0 && warp == 2) {
            issue_x(it, 0);
        }
        if (buf == 0) { ok = mbar_wait(&bars[BAR_X0], ph_x0) && ok; ph_x0 ^= 1; }
        else { ok = mbar_wait(&bars[BAR_X1], ph_x1) && ok; ph_x1 ^= 1; }

        const __nv_bfloat16 *X = Xs + buf * mrows * PX;
        float acc[NT_S][4];
#pragma unroll
        for (int nt = 0; nt < NT_S; ++nt) acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.0f;
#pragma unroll
        for (int ks = 0; ks < KW; ks += 16) {
            const int kk = warp * KW + ks;
            if (kk < ncols) {
                const bool full = ncols - kk >= 16;   // else only 8 columns are left
                uint32_t a[4];
                a[0] = lds32(X + g * PX + kk + 2 * t);
                a[1] = hi_rows ? lds32(X + (g + 8) * PX + kk + 2 * t) : 0u;
                a[2] = full ? lds32(X + g * PX + kk + 8 + 2 * t) : 0u;
                a[3] = (full && hi_rows) ? lds32(X + (g + 8) * PX + kk + 8 + 2 * t) : 0u;
#pragma unroll
                for (int nt = 0; nt < NT_S; ++nt) {
                    const __nv_bfloat16 *ar = As + (nt * 8 + g) * PA + kk + 2 * t;
                    mma16816(acc[nt], a, lds32(ar), full ? lds32(ar + 8) : 0u);
                }
            }
        }
#pragma unroll
        for (int nt = 0; nt < NT_S; ++nt) {
            float *p0 = part + (warp * mrows + g) * RP + nt * 8 + 2 * t;
            *reinterpret_cast<float2 *>(p0) = make_float2(acc[nt][0], acc[nt][1]);
            if (hi_rows) *reinterpret_cast<float2 *>(p0 + 8 * RP) = make_float2(acc[nt][2], acc[nt][3]);
        }
        __syncthreads();
        // block partial: the four warps' sums in warp order, accumulated over column chunks
        for (int i = tid; i < mrows * RP; i += FT) {
            const int r = i / RP, k = i - r * RP;
            if (mt * 16 + r < rows) {
                const float s = ((part[(0 * mrows + r) * RP + k] + part[(1 * mrows + r) * RP + k]) +
                                 part[(2 * mrows + r) * RP + k]) + part[(3 * mrows + r) * RP + k];
                float *dst = vpart + (mt * 16 + r) * RP + k;
                *dst = c == 0 ? s : *dst + s;
            }
        }
        __syncthreads();   // partial buffers, the x stage and (after the last row tile) the A stage are free
    }
    if (n_items == 0) {   // this block owns no d_in columns: its partial is zero
        for (int i = tid; i < rows * RP; i += FT) vpart[i] = 0.0f;
    }
    // ---- exchange: every block sums all blocks' partials in block order -------------------------
    cluster_arrive();
    cluster_wait();
    {
        const uint32_t vp_addr = smem_u32(vpart);
        for (int i = tid; i < rows * rank16; i += FT) {
            const int m = i / rank16, k = i - m * rank16;
            float v = 0.0f;
            if (k < rank) {
                // all remote loads are issued before the first add, so their latencies overlap;
                // the sum is still taken in block order
                float pv[8];
#pragma unroll
                for (uint32_t q = 0; q < 8; ++q)
                    pv[q] = q < csize ? ld_peer_f32(vp_addr + (uint32_t)(m * RP + k) * 4u, q) : 0.0f;
#pragma unroll
                for (uint32_t q = 0; q < 8; ++q) v += pv[q];
            }
            const __nv_bfloat16 hi = __float2bfloat16_rn(v);
            Vh[m * PV + k] = hi;
            Vl[m * PV + k] = __float2bfloat16_rn(v - __bfloat162float(hi));
        }
    }
    cluster_arrive();   // done reading the peers; the matching wait is at the end
    __syncthreads();

    // ---- expand: warp w takes columns [w*NW, (w+1)*NW) of the staged chunk ----------------------
    {
        const float s = tl.scale;
        for (int32_t c = 0; c < nb; ++c) {
            const int32_t col0 = b_lo + c * DCB, ncols = min(DCB, b_hi - col0);
            if (c > 0 && warp == 1)
                issue_rows(&bars[BAR_B], Bs, PB, rank, ncols, lane, B + col0, d_out, nullptr);
            ok = mbar_wait(&bars[BAR_B], ph_b) && ok;
            ph_b ^= 1;
            for (int32_t mt = 0; mt < n_mt; ++mt) {
                const __nv_bfloat16 *vh = Vh + (mt * 16 + g) * PV + 2 * t;
                const __nv_bfloat16 *vl = Vl + (mt * 16 + g) * PV + 2 * t;
#pragma unroll
                for (int p = 0; p < NPASS; ++p) {
                    const int base = warp * NW + p * 64;
                    if (base >= ncols) continue;
                    // y_base of the next pass is requested while this pass computes
                    if (p == 0 && (c > 0 || mt > 0)) load_yb(ybw[0], c, mt, 0);
                    if (p + 1 < NPASS) load_yb(ybw[(p + 1) % NPASS], c, mt, p + 1);
                    float acc[8][4];
#pragma unroll
                    for (int j = 0; j < 8; ++j) acc[j][0] = acc[j][1] = acc[j][2] = acc[j][3] = 0.0f;
                    for (int ks = 0; ks < rank16; ks += 16) {
                        uint32_t ah[4], al[4];
                        ah[0] = lds32(vh + ks);
                        ah[1] = hi_rows ? lds32(vh + 8 * PV + ks) : 0u;
                        ah[2] = lds32(vh + ks + 8);
                        ah[3] = hi_rows ? lds32(vh + 8 * PV + ks + 8) : 0u;
                        al[0] = lds32(vl + ks);
                        al[1] = hi_rows ? lds32(vl + 8 * PV + ks) : 0u;
                        al[2] = lds32(vl + ks + 8);
                        al[3] = hi_rows ? lds32(vl + 8 * PV + ks + 8) : 0u;
#pragma unroll
                        for (int np = 0; np < 4; ++np) {
                            // matrices: (k 0..7, tile 2np), (k 8..15, tile 2np), (k 0..7, 2np+1), (k 8..15, 2np+1)
                            const int mi = lane >> 3;
                            const __nv_bfloat16 *bp = Bs + (ks + (mi & 1) * 8 + (lane & 7)) * PB + base +
                                                      (np * 2 + (mi >> 1)) * 8;
                            uint32_t b[4];
                            ldmatrix_x4_trans(b, smem_u32(bp));
                            mma16816(acc[np * 2], ah, b[0], b[1]);
                            mma16816(acc[np * 2], al, b[0], b[1]);
                            mma16816(acc[np * 2 + 1], ah, b[2], b[3]);
                            mma16816(acc[np * 2 + 1], al, b[2], b[3]);
                        }
                    }
                    // epilogue straight from the accumulator layout: each lane owns two adjacent
                    // columns of a row per column tile; a quad covers 16 contiguous bytes
#pragma unroll
                    for (int h = 0; h < H; ++h) {
                        const int32_t m = mt * 16 + g + 8 * h;
                        if (m < rows && ok) {
                            __nv_bfloat16 *yrow = P.y + (int64_t)rowidx[m] * P.ldy + col0 + base + 2 * t;
#pragma unroll
                            for (int j = 0; j < 8; ++j) {
                                if (base + j * 8 < ncols) {
                                    const uint32_t w = ybw[p][j][h];
                                    const float y0 = fmaf(s, acc[j][2 * h], __uint_as_float(w << 16));
                                    const float y1 = fmaf(s, acc[j][2 * h + 1], __uint_as_float(w & 0xffff0000u));
                                    *reinterpret_cast<uint32_t *>(yrow + j * 8) = pack2(y0, y1);
                                }
                            }
                        }
                    }
                }
            }
            __syncthreads();   // the B stage is free
        }
    }
    if (!ok && tid == 0) atomicAdd(&P.pool.status[STATUS_TIMEOUTS], 1);
    cluster_wait();   // no block leaves while a peer may still read its partials
}

// One kernel per rank bucket (RP) and row-tile occupancy (H); units of another bucket are skipped.
// P.aux != 0 marks the launch that also counts invalid tokens and copies adapter-less rows.
template <int RP, int DCA, int DCB, int H>
__global__ void __launch_bounds__(FT, LORA_FUSED_MIN_BLOCKS)
fused_kernel(const ApplyParams P) {
    extern __shared__ __align__(128) unsigned char smem[];
    const uint32_t csize = cluster_nctarank(), crank = cluster_ctarank();
    const int32_t cid = (int32_t)(blockIdx.x / csize), G = (int32_t)(gridDim.x / csize);
    const int tid = threadIdx.x;
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem);
    int32_t *rowidx = reinterpret_cast<int32_t *>(smem + 64);

    // set-up that touches no global memory; the next kernel on the stream may be scheduled from
    // here on, and this one waits for everything queued before it
    if (tid == 0) {
        mbar_init(&bars[BAR_A], 1);
        mbar_init(&bars[BAR_B], 1);
        mbar_init(&bars[BAR_X0], 1);
        mbar_init(&bars[BAR_X1], 1);
        fence_mbar_init();
    }
    griddep_launch_dependents();
    __syncthreads();
    griddep_wait();

    uint32_t ph[4] = {0u, 0u, 0u, 0u};
    int32_t n_tile = P.meta ? 0x7fffffff : P.T;
    // The grid holds as many clusters as fit on the GPU at once; each takes units cid, cid + G, ...
    // Tiles of more than 16 rows are worked on in pieces of 16 rows (P.sub pieces per tile), so
    // the shared-memory footprint of a block does not grow with tile_m.
    // Such batches are walked through the metadata's list of pieces (no empty entries); decode
    // batches (tile_m <= 16) index the tile table directly, which saves a dependent load.
    const int32_t sub = P.sub, piece_rows = sub > 1 ? 16 : P.tile_m;
    for (int32_t unit = cid; unit < P.units * sub && unit < n_tile; unit += G) {
        // the tile record, the tile's row ids and (first time) the count are fetched side by side
        Tile tl;
        if (P.meta) {
            int32_t u = unit, piece = 0;
            if (sub > 1) {
                if (unit == cid) n_tile = __ldg(P.meta + H_NPIECE);   // here: number of pieces
                if (unit >= n_tile) break;
                const int32_t e = __ldg(P.meta + P.moff_piece + unit);
                u = e >> 4;
                piece = e & 15;
            }
            if (tid < piece_rows)
                rowidx[tid] = __ldg(P.meta + P.moff_tperm + u * P.tile_m + piece * 16 + tid);
            if (sub == 1 && unit == cid) n_tile = __ldg(P.meta + H_NTILE);
            const int4 d = __ldg(reinterpret_cast<const int4 *>(P.meta + P.moff_desc) + u);
            const int32_t tile_rows = d.z & 0x7fff;
            tl.slot = d.x;
            tl.row0 = d.y + piece * 16;
            tl.rows = min(piece_rows, tile_rows - piece * 16);
            tl.rank = d.z >> 16;
            tl.scale = __int_as_float(d.w);
            tl.valid = d.x >= 0;
            if (sub == 1 && u >= n_tile) break;
            // runs of consecutive tokens belong to the tensor-core kernels when those ran
            if (tl.rows <= 0 || (P.path_filter && tile_rows >= P.path_filter && ((d.z >> 15) & 1))) {
                __syncthreads();
                continue;
            }
        } else {
            if (tid == 0) rowidx[0] = unit;
            MetaLayout L;
            tl = resolve_unit(P, L, unit);
        }
        __syncthreads();   // row ids visible
        if (!tl.valid) {
            if (!P.meta && P.aux) {   // per-token mode: this token has no adapter
                if (crank == 0 && tid == 0 && P.slot_idx[unit] != -1)
                    atomicAdd(&P.pool.status[STATUS_INVALID_TOKENS], 1);
                if (!P.in_place) copy_rows(P, rowidx, 1, (int32_t)crank, (int32_t)csize);
            }
            __syncthreads();   // before the row ids are overwritten
            continue;
        }
        const int32_t b = rank_bucket(tl.rank);
        if ((b <= 16 ? 16 : b) != RP) {   // another launch's bucket
            __syncthreads();
            continue;
        }
        fused_body<RP, DCA, DCB, H>(P, tl, smem, crank, csize, ph);
    }
    // rows that take no adapter: y_base -> y, 16 rows per cluster step (grouped mode, out of place)
    if (P.meta && !P.in_place && P.aux) {
        const int32_t n_active = __ldg(P.meta + H_NACTIVE);
        for (int32_t first = cid * 16; first < P.T - n_active; first += G * 16) {
            const int32_t rows = min(16, P.T - n_active - first);
            __syncthreads();
            if (tid < rows) rowidx[tid] = __ldg(P.meta + P.moff_perm + n_active + first + tid);
            __syncthreads();
            copy_rows(P, rowidx, rows, (int32_t)crank, (int32_t)csize);
        }
    }
}

// One launch for the tiles of one rank bucket.  The shared-memory carve-up is sized for that bucket.
template <int RP, int DCA, int DCB, int H>
static lora_status_t launch_bucket(lora_pool_t *pool, ApplyParams P, int32_t C, cudaStream_t stream) {
    auto kern = fused_kernel<RP, DCA, DCB, H>;
    const int32_t tile_m = P.meta ? P.tile_m : 1;
    const int32_t vrows = H == 1 ? 8 : P.rows_cap;      // rows of the v buffers
    int32_t o = (64 + P.rows_cap * 4 + 127) & ~127;     // mbarriers, row ids
    P.off_part = o;   o += 4 * (8 * H) * RP * 4;
    P.off_vpart = o;  o += vrows * RP * 4;
    P.off_vh = o;     o += vrows * (RP + 8) * 2;
    P.off_vl = o;     o += vrows * (RP + 8) * 2;
    o = (o + 127) & ~127;
    P.off_stage = o;  o += RP * (DCA + 8) * 2 + RP * (DCB + 8) * 2;
    P.off_x = o;      o += P.xbufs * (8 * H) * 520 * 2;
    P.off_vst = 0;
    const int32_t smem = o;
    (void)tile_m;

    static int32_t attr_smem = 0;
    if (smem > attr_smem) {
        LORA_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        attr_smem = smem;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3(FT, 1, 1);
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
    const unsigned n_attrs = pool->tuning[2] == 1 ? 2 : 1;   // tuning key 2 = 1: programmatic dependent launch

    // Grid: no more clusters than can be resident at once (each loops over its units), so no
    // cluster of an over-sized grid waits for a slot only to find that its unit does not exist.
    static int32_t occ_smem = -1, occ_c = -1, occ_clusters = 0;
    if (occ_smem != smem || occ_c != C) {
        cfg.gridDim = dim3((unsigned)(C * pool->sm_count), 1, 1);
        cfg.numAttrs = 1;
        int n = 0;
        cudaError_t e = cudaOccupancyMaxActiveClusters(&n, kern, &cfg);
        if (e != cudaSuccess || n < 1) {
            cudaGetLastError();
            n = 0;
        }
        occ_smem = smem; occ_c = C; occ_clusters = n;
        if (getenv("LORA_B200_DEBUG"))
            fprintf(stderr, "lora_b200: fused kernel rank<=%d rows<=%d: smem %d B, cluster %d, resident clusters %d\n",
                    RP, 8 * H, smem, C, n);
    }
    cfg.numAttrs = n_attrs;
    int32_t want = P.units * P.sub;   // tile pieces, or 16-row copy steps if there are more of those
    if (P.aux && P.meta && !P.in_place && (P.T + 15) / 16 > want) want = (P.T + 15) / 16;
    int32_t G = occ_clusters > 0 && occ_clusters < want ? occ_clusters : want;
    if (pool->tuning[3] > 0 && pool->tuning[3] < G) G = pool->tuning[3];
    cfg.gridDim = dim3((unsigned)(G * C), 1, 1);
    LORA_CUDA_TRY(cudaLaunchKernelEx(&cfg, kern, P));
    return count_launch();
}

lora_status_t launch_fused(lora_pool_t *pool, ApplyParams &P, cudaStream_t stream) {
    const int32_t tile_m = P.meta ? P.tile_m : 1;
    P.sub = tile_m > 16 ? (tile_m + 15) / 16 : 1;   // larger tiles are worked on in 16-row pieces
    P.rows_cap = 16;
    P.mrows = tile_m <= 8 ? 8 : 16;
    P.xbufs = 1;
    P.moff_perm = P.moff_desc = P.moff_tperm = P.moff_piece = 0;
    if (P.meta) {
        const MetaLayout L = meta_layout(P.T, P.meta_slots, P.tile_m);
        if (L.words > 0x7fffffff) return LORA_ERR_SHAPE;
        P.moff_perm = (int32_t)L.perm;
        P.moff_desc = (int32_t)L.tile_desc;
        P.moff_tperm = (int32_t)L.tile_perm;
        P.moff_piece = (int32_t)L.tile_piece;
    }
    // cluster size: as wide a split as the projection supports, narrower when there are many units
    int32_t C = pool->tuning[1];
    if (C != 1 && C != 2 && C != 4 && C != 8) {
        C = 8;
        while (C > 1 && (P.tv.d_in / C < 256 || P.tv.d_out / C < 128)) C >>= 1;
    }
    // one launch per rank bucket that has ever been loaded into the pool (ranks <= 16 share one)
    bool need[3] = {(pool->bucket_mask & 3u) != 0, (pool->bucket_mask & 4u) != 0,
                    (pool->bucket_mask & 8u) != 0};
    if (!need[0] && !need[1] && !need[2]) need[0] = true;   // empty pool: rows are still copied
    P.aux = 1;
    for (int b = 0; b < 3; ++b) {
        if (!need[b]) continue;
        lora_status_t s;
        if (P.mrows == 8) {
            s = b == 0 ? launch_bucket<16, 512, 512, 1>(pool, P, C, stream)
              : b == 1 ? launch_bucket<32, 256, 256, 1>(pool, P, C, stream)
                       : launch_bucket<64, 256, 256, 1>(pool, P, C, stream);
        } else {
            s = b == 0 ? launch_bucket<16, 512, 512, 2>(pool, P, C, stream)
              : b == 1 ? launch_bucket<32, 256, 256, 2>(pool, P, C, stream)
                       : launch_bucket<64, 256, 256, 2>(pool, P, C, stream);
        }
        if (s != LORA_OK) return s;
        P.aux = 0;
    }
    return LORA_OK;
}

}  // namespace lora
