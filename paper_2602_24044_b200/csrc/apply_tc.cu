// Tensor-core path of lora_sgmv_apply for LONG tiles: runs of 32 .. 128 consecutive tokens of one
// adapter (prefill / chunked-prefill segments), y = y_base + s_i * (x . A_i) . B_i (paper Section 2.2).
//
// Such a tile is a dense contraction, so it runs on the 5th-generation tensor cores:
//   tc_worklist_kernel  the long tiles of the batch, in tile order, as a compact list
//   tc_shrink_kernel    V[128, r] = X[128, d_in] . A_i[r, d_in]^T, computed in pieces: the (tile,
//       K-block) pairs of all tiles form one walk cut into equal spans, one per block of a grid
//       that fills the GPU once.  X and A_i tiles arrive by TMA (128-byte swizzle) through a
//       three-stage mbarrier ring; one thread requests them, one issues tcgen05.mma (M = 128,
//       N = rank bucket, K = 16) with the accumulator in tensor memory, four warps write each
//       finished piece to its fp32 slab of the workspace.
//   tc_expand_kernel    Y[128, N-slice] = Y_base + s * V . B_i[r, N-slice]
//       V = sum of the tile's pieces (in order), carried as a high and a low bf16 part (two MMAs,
//       ~16 mantissa bits); per 64-column block one TMA load of the B_i tile and of the y_base
//       tile, MMA into a ring of tensor-memory accumulators, epilogue tcgen05.ld -> fused scale +
//       residual add -> bf16 written in place into the y_base tile -> TMA store.
// Both kernels are HBM-bound streaming kernels: the tensor cores only keep the arithmetic off the
// critical path.  Every wait on an mbarrier is bounded; on expiry the block records it in the
// pool's status word, frees its tensor memory and leaves without storing.
// All other tiles (short, ragged or scattered) are handled by the fused kernel.
#include <cuda.h>

#include <cstdio>
#include <cstdlib>
#include <cstring>

#include "apply_common.cuh"

namespace lora {

// ---------------------------------------------------------------------------------------------
// PTX wrappers
// ---------------------------------------------------------------------------------------------
namespace tc {
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
    for (uint32_t i = 0; i < (1u << 18); ++i)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tma_load_2d(void *dst, const CUtensorMap *map, int c0, int c1,
                                            uint64_t *bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, "
        "%3}], [%4];" ::"r"(smem_u32(dst)),
        "l"(map), "r"(c0), "r"(c1), "r"(smem_u32(bar))
        : "memory");
}
__device__ __forceinline__ void tma_load_3d(void *dst, const CUtensorMap *map, int c0, int c1, int c2,
                                            uint64_t *bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, "
        "%3, %4}], [%5];" ::"r"(smem_u32(dst)),
        "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(smem_u32(bar))
        : "memory");
}
__device__ __forceinline__ void tma_store_2d(const CUtensorMap *map, int c0, int c1, const void *src) {
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%1, %2}], [%3];" ::"l"(map),
                 "r"(c0), "r"(c1), "r"(smem_u32(src))
                 : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read() {
    asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void fence_proxy_async() {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t *dst_smem, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst_smem)),
                 "r"(ncols)
                 : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() {
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after() {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
// D[tmem] (+)= A[smem desc] . B[smem desc], bf16 x bf16 -> fp32, issued by one thread
__device__ __forceinline__ void umma(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                     uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// the mbarrier receives one arrival when every MMA issued so far by this thread has completed
__device__ __forceinline__ void umma_commit(uint64_t *bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(
                     smem_u32(bar))
                 : "memory");
}
// 32 lanes x 16 consecutive columns of tensor memory -> 16 registers per thread (lane = thread)
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, "
        "%14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// shared-memory matrix descriptor (start address, leading / stride byte offsets in 16-byte units,
// descriptor version 1, layout type in the top three bits)
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes,
                                              uint32_t layout_type) {
    uint64_t d = (uint64_t)((addr & 0x3FFFFu) >> 4);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)layout_type << 61;
    return d;
}
constexpr uint32_t LAYOUT_NONE = 0, LAYOUT_SW128 = 2;
// instruction descriptor: fp32 accumulator, bf16 A and B, majors, N / 8, M / 16
__host__ __device__ constexpr uint32_t instr_desc(uint32_t M, uint32_t N, uint32_t a_mn_major,
                                                  uint32_t b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | (a_mn_major << 15) | (b_mn_major << 16) | ((N >> 3) << 17) |
           ((M >> 4) << 24);
}
}  // namespace tc

constexpr int XQ = 2;               // expand: epilogue warps per quarter of the rows (each takes 64 / XQ columns; 1: 561, 2: 553, 4: 557 us per prefill step)
constexpr int TCX_THREADS = 32 * (4 * XQ + 2);   // plus one warp that issues MMAs and one that issues copies
constexpr int TC_ROWS = 128;       // rows of a long tile
constexpr int SH_STAGES = 3;       // shrink: ring of (x tile, A tile) stages
constexpr int XT_BYTES = TC_ROWS * 128;   // 128 rows x 64 bf16

struct TcParams {
    PoolView pool;
    TargetView tv;
    const int32_t *meta;
    float *ws;              // [KS][T][RS] fp32 partial v: one slab per piece of a tile
    int32_t T, RS, KS;      // KS: slabs the workspace holds
    int32_t expand_grid;    // blocks of the expand launch
    int32_t shrink_grid;    // blocks of the shrink launch (fixes how the walk is cut into pieces)
    int32_t moff_perm, moff_desc;
    int32_t target_rows;    // r_max: rows of a slot's matrices
    __nv_bfloat16 *y;       // output, for tiles with fewer than 128 rows (stored row by row)
    int64_t ldy;
    int32_t *list;          // list of long tiles in the metadata: [0] = their number, then their tile numbers
    int32_t list_cap;
};

// tile record -> (valid long tile of this bucket?, slot, first token, position in perm, rank, scale)
constexpr int TC_MIN_ROWS = 32;    // shortest run of consecutive tokens given to the tensor cores
// Batches of fewer than this many 128-row tiles do not come here: a handful of long tiles cannot
// fill the GPU with 128-row blocks, and the three extra launches cost more than they save
// (mixed chunked-prefill batch with sixteen long tiles: 127 us with them, 97 us on the stream kernel alone).
constexpr int TC_MIN_TILES = 32;
struct LongTile {
    int32_t slot, t0, row0, rank, rows;
    float scale;
    bool ok;
};
// entry: position in the work list (the grid is sized by a bound on the list's length)
__device__ __forceinline__ LongTile long_tile(const TcParams &P, int32_t entry) {
    LongTile lt;
    lt.ok = false;
    if (entry >= P.list[0]) return lt;
    const int32_t unit = P.list[1 + entry];
    const int4 d = __ldg(reinterpret_cast<const int4 *>(P.meta + P.moff_desc) + unit);
    const int32_t rows = d.z & 0x7fff, contiguous = (d.z >> 15) & 1, rank = d.z >> 16;
    if (d.x < 0 || rows < TC_MIN_ROWS || !contiguous) return lt;
    lt.rows = rows;
    lt.slot = d.x;
    lt.row0 = d.y;
    lt.rank = rank;
    lt.scale = __int_as_float(d.w);
    lt.t0 = __ldg(P.meta + P.moff_perm + d.y);
    lt.ok = true;
    return lt;
}

// The tiles this path takes (runs of at least TC_MIN_ROWS consecutive tokens), in tile order, as a
// compact list in the metadata buffer, written once behind the build (every apply on that table
// reads it): the kernels below walk list entries, not the tiles of the batch (a mixed batch has
// hundreds of tiles and a handful of long ones).
__global__ void __launch_bounds__(256)
tc_worklist_kernel(const TcParams P) {
    __shared__ int32_t warp_count[8];
    __shared__ int32_t base_s;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int32_t n_tile = P.meta[H_NTILE];
    if (tid == 0) base_s = 0;
    __syncthreads();
    for (int32_t t0 = 0; t0 < n_tile; t0 += 256) {
        const int32_t idx = t0 + tid;
        bool take = false;
        if (idx < n_tile) {
            const int4 d = *(reinterpret_cast<const int4 *>(P.meta + P.moff_desc) + idx);
            take = d.x >= 0 && (d.z & 0x7fff) >= TC_MIN_ROWS && ((d.z >> 15) & 1);
        }
        const uint32_t m = __ballot_sync(0xffffffffu, take);
        if (lane == 0) warp_count[warp] = __popc(m);
        __syncthreads();
        int32_t before = base_s;
        for (int w = 0; w < warp; ++w) before += warp_count[w];
        const int32_t pos = before + __popc(m & ((1u << lane) - 1u));
        if (take && pos < P.list_cap) P.list[1 + pos] = idx;
        __syncthreads();
        if (tid == 0) {
            int32_t tot = 0;
            for (int w = 0; w < 8; ++w) tot += warp_count[w];
            base_s += tot;
        }
        __syncthreads();
    }
    if (tid == 0) P.list[0] = min(base_s, P.list_cap);
}

// ---------------------------------------------------------------------------------------------
// shrink
// ---------------------------------------------------------------------------------------------
// The shrink walks the (long tile, 64-column K-block) pairs of the batch in tile order.  The walk is
// cut into equal spans, one per block of a grid that fills the GPU exactly once, so every block
// streams the same number of bytes whatever the number of long tiles is.  A span may end inside a
// tile: the part of tile t that block b computes is the tile's "piece" b - first_block(t), and its
// fp32 partial goes to slab [piece] of the workspace; the expand adds a tile's pieces in order.
struct ShrinkSplit {
    int64_t total;     // K-blocks of all long tiles
    int32_t nkb;       // K-blocks of one tile
    int32_t span;      // K-blocks per block
};
// slabs: partial slabs the workspace holds (a tile must not be cut into more pieces than that)
__host__ __device__ inline ShrinkSplit shrink_split(int32_t n_long, int32_t d_in, int32_t slabs, int32_t grid) {
    ShrinkSplit sp;
    sp.nkb = (d_in + 63) / 64;
    sp.total = (int64_t)n_long * sp.nkb;
    int64_t span = (sp.total + grid - 1) / grid;
    if (slabs <= 1) {
        span = ((span + sp.nkb - 1) / sp.nkb) * sp.nkb;          // whole tiles only
    } else {
        const int64_t least = (sp.nkb + slabs - 2) / (slabs - 1);   // at most slabs pieces per tile
        if (span < least) span = least;
    }
    if (span < 1) span = 1;
    sp.span = (int32_t)span;
    return sp;
}
// pieces of tile entry t: blocks first .. last of the walk touch it
__host__ __device__ inline int32_t first_block_of(const ShrinkSplit &sp, int32_t t) {
    return (int32_t)(((int64_t)t * sp.nkb) / sp.span);
}
__host__ __device__ inline int32_t last_block_of(const ShrinkSplit &sp, int32_t t) {
    return (int32_t)((((int64_t)t + 1) * sp.nkb - 1) / sp.span);
}

constexpr int TCS_THREADS = 192;   // shrink: four warps that write partials, one MMA thread, one loading thread

template <int RP>
__global__ void __launch_bounds__(TCS_THREADS)
tc_shrink_kernel(const TcParams P, const __grid_constant__ CUtensorMap map_x,
                 const __grid_constant__ CUtensorMap map_a) {
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    // the swizzled tiles want 1024-byte aligned bases
    unsigned char *smem = reinterpret_cast<unsigned char *>(
        ((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    constexpr int AT_BYTES = RP * 128;               // RP rank rows x 64 bf16
    constexpr int STAGE = XT_BYTES + ((AT_BYTES + 1023) & ~1023);
    constexpr uint32_t ACC = RP < 32 ? 32 : RP;      // columns of one accumulator
    constexpr uint32_t TMEM_COLS = 2 * ACC;          // two accumulators: a piece is written out while the next one runs
    uint64_t *full = reinterpret_cast<uint64_t *>(smem + SH_STAGES * STAGE);
    uint64_t *empty = full + SH_STAGES;
    uint64_t *done = empty + SH_STAGES;              // [2] all MMAs of a piece have completed
    uint64_t *acc_free = done + 2;                   // [2] the accumulator has been read out
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(acc_free + 2);
    volatile int32_t *failed = reinterpret_cast<volatile int32_t *>(tmem_slot + 1);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int32_t n_long = P.list[0];
    if (n_long <= 0) return;
    const ShrinkSplit sp = shrink_split(n_long, P.tv.d_in, P.KS, (int32_t)gridDim.x);
    const int64_t g0 = (int64_t)blockIdx.x * sp.span;
    const int64_t g1 = min(g0 + (int64_t)sp.span, sp.total);
    if (g0 >= g1) return;

    if (tid == 0) {
        for (int s = 0; s < SH_STAGES; ++s) { tc::mbar_init(&full[s], 1); tc::mbar_init(&empty[s], 1); }
        for (int s = 0; s < 2; ++s) { tc::mbar_init(&done[s], 1); tc::mbar_init(&acc_free[s], 128); }
        *failed = 0;
        tc::fence_mbar_init();
    }
    if (warp == 4) {
        tc::tmem_alloc(tmem_slot, TMEM_COLS);
        tc::tmem_relinquish();
    }
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp == 5) {
        // ---- loading thread: requests the (x tile, A tile) pairs of the whole span in order; it
        // alone waits for a stage to be read out before refilling it ----------------------------
        if (lane == 0) {
            int32_t issued = 0;
            bool ok = true;
            int32_t t = (int32_t)(g0 / sp.nkb), kb = (int32_t)(g0 % sp.nkb);
            LongTile lt = long_tile(P, t);
            for (int64_t g = g0; g < g1 && ok; ++g) {
                const int s = issued % SH_STAGES;
                if (issued >= SH_STAGES) ok = tc::mbar_wait(&empty[s], (uint32_t)(issued / SH_STAGES - 1) & 1u);
                if (!ok || *failed || !lt.ok) { ok = false; break; }
                unsigned char *st = smem + s * STAGE;
                tc::mbar_expect_tx(&full[s], XT_BYTES + AT_BYTES);
                tc::tma_load_2d(st, &map_x, kb * 64, lt.t0, &full[s]);
                tc::tma_load_3d(st + XT_BYTES, &map_a, kb * 64, 0, lt.slot, &full[s]);
                ++issued;
                if (++kb == sp.nkb && g + 1 < g1) {
                    kb = 0;
                    lt = long_tile(P, ++t);
                }
            }
            if (!ok) {
                *failed = 1;
                // copies still on their way into this block's shared memory must land before it
                // leaves: the most recent request of every stage is waited for (bounded)
                for (int32_t q = max(issued - SH_STAGES, 0); q < issued; ++q)
                    tc::mbar_wait(&full[q % SH_STAGES], (uint32_t)(q / SH_STAGES) & 1u);
            }
        }
        __syncwarp();
    } else if (warp == 4) {
        // ---- MMA thread: it only ever waits for data (and, from the third piece on, for the
        // accumulator it reuses) -----------------------------------------------------------------
        if (lane == 0) {
            constexpr uint32_t IDESC = tc::instr_desc(128, RP, 0, 0);
            int32_t i = 0, piece = 0;
            bool ok = true;
            for (int64_t g = g0; g < g1 && ok; ++piece) {
                const int32_t kb = (int32_t)(g % sp.nkb);
                const int32_t len = (int32_t)min((int64_t)(sp.nkb - kb), g1 - g);
                const uint32_t acc = tmem + (uint32_t)(piece & 1) * ACC;
                if (piece >= 2) ok = tc::mbar_wait(&acc_free[piece & 1], (uint32_t)(piece / 2 - 1) & 1u);
                tc::tc_fence_after();
                for (int32_t k = 0; k < len && ok; ++k, ++i) {
                    const int s = i % SH_STAGES;
                    ok = !*failed && tc::mbar_wait(&full[s], (uint32_t)(i / SH_STAGES) & 1u);
                    if (!ok) break;
                    tc::tc_fence_after();
                    const uint32_t xa = tc::smem_u32(smem + s * STAGE), aa = xa + XT_BYTES;
#pragma unroll
                    for (int k4 = 0; k4 < 4; ++k4) {   // four K = 16 steps inside the 128-byte swizzle atom
                        const uint64_t ad = tc::smem_desc(xa + k4 * 32, 16, 1024, tc::LAYOUT_SW128);
                        const uint64_t bd = tc::smem_desc(aa + k4 * 32, 16, 1024, tc::LAYOUT_SW128);
                        tc::umma(acc, ad, bd, IDESC, (k > 0 || k4 > 0) ? 1u : 0u);
                    }
                    tc::umma_commit(&empty[s]);   // the stage may be refilled once these MMAs have read it
                }
                if (ok) tc::umma_commit(&done[piece & 1]);
                g += len;
            }
            if (!ok) *failed = 1;
        }
        __syncwarp();
    } else {
        // ---- four warps move each finished piece from tensor memory to its slab (thread = row) --
        const int32_t m = warp * 32 + lane;
        int32_t piece = 0;
        for (int64_t g = g0; g < g1; ++piece) {
            const int32_t t = (int32_t)(g / sp.nkb), kb = (int32_t)(g % sp.nkb);
            const int32_t len = (int32_t)min((int64_t)(sp.nkb - kb), g1 - g);
            const LongTile lt = long_tile(P, t);
            const int32_t slab = (int32_t)blockIdx.x - first_block_of(sp, t);
            const uint32_t bad =
                (*failed != 0 || !lt.ok || !tc::mbar_wait(&done[piece & 1], (uint32_t)(piece / 2) & 1u)) ? 1u : 0u;
            uint32_t any_bad;
            asm volatile(
                "{\n\t.reg .pred p, q;\n\t"
                "setp.ne.u32 p, %1, 0;\n\t"
                "bar.red.or.pred q, 1, 128, p;\n\t"
                "selp.u32 %0, 1, 0, q;\n\t}"
                : "=r"(any_bad)
                : "r"(bad)
                : "memory");
            if (any_bad) { *failed = 1; break; }
            tc::tc_fence_after();
            float *dst = P.ws + ((int64_t)slab * P.T + lt.row0 + m) * P.RS;
#pragma unroll
            for (int c = 0; c < RP; c += 16) {
                uint32_t r[16];
                tc::tmem_ld16(tmem + ((uint32_t)(warp * 32) << 16) + (uint32_t)(piece & 1) * ACC + c, r);
                tc::tmem_ld_wait();
                if (m < lt.rows) {  // rows past a short tile's end belong to other tiles
#pragma unroll
                    for (int i = 0; i < 16; i += 4)
                        *reinterpret_cast<uint4 *>(dst + c + i) = make_uint4(r[i], r[i + 1], r[i + 2], r[i + 3]);
                }
            }
            tc::tc_fence_before();
            tc::mbar_arrive(&acc_free[piece & 1]);
            g += len;
        }
    }
    tc::tc_fence_before();
    __syncthreads();
    if (tid == 0 && *failed) atomicAdd(&P.pool.status[STATUS_TIMEOUTS], 1);
    if (warp == 4) tc::tmem_dealloc(tmem, TMEM_COLS);
}

// ---------------------------------------------------------------------------------------------
// expand
// ---------------------------------------------------------------------------------------------
template <int RP>
struct ExpandCfg {
#ifdef LORA_TC_EXPAND_STAGES
    static constexpr int STAGES = LORA_TC_EXPAND_STAGES;
#else
    static constexpr int STAGES = 3;   // three stages leave room for a block of the fused kernel beside two of these
#endif
    static constexpr int BT_BYTES = RP * 128;                       // RP rank rows x 64 columns
    static constexpr int STAGE = XT_BYTES + ((BT_BYTES + 1023) & ~1023);   // y_base/out tile + B tile
    static constexpr int V_BYTES = TC_ROWS * RP * 2;                // one bf16 copy of v
    static constexpr int SMEM = 2 * V_BYTES + STAGES * STAGE + 256 + 1024;
    static constexpr uint32_t TMEM_COLS = STAGES <= 2 ? 128 : STAGES <= 4 ? 256 : 512;  // ring of 64-column accumulators
};

// The expand walks the (long tile, 64-column block of d_out) pairs in tile order, cut into equal
// spans like the shrink's walk, one span per block; the grid is several waves of blocks.  A block
// whose span crosses into the next tile builds that tile's v when it gets there.
template <int RP>
__global__ void __launch_bounds__(TCX_THREADS)
tc_expand_kernel(const TcParams P, const __grid_constant__ CUtensorMap map_b,
                 const __grid_constant__ CUtensorMap map_yb, const __grid_constant__ CUtensorMap map_y) {
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    using C = ExpandCfg<RP>;
    constexpr int S = C::STAGES;
    // the swizzled tiles want 1024-byte aligned bases
    unsigned char *smem = reinterpret_cast<unsigned char *>(
        ((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    unsigned char *stages = smem;                                   // [S][y_base tile | B tile]
    unsigned char *Vh = smem + S * C::STAGE;                        // core-matrix layout, see below
    unsigned char *Vl = Vh + C::V_BYTES;
    uint64_t *full = reinterpret_cast<uint64_t *>(Vl + C::V_BYTES);
    uint64_t *mma_done = full + S;
    uint64_t *epi_done = mma_done + S;  // every epilogue thread has finished its row of the stage
    uint64_t *v_ready = epi_done + S;   // the tile's v (both bf16 parts) is in shared memory
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(v_ready + 1);
    volatile int32_t *failed = reinterpret_cast<volatile int32_t *>(tmem_slot + 1);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int32_t n_long = P.list[0];
    if (n_long <= 0) return;
    const int32_t nblk = (P.tv.d_out + 63) / 64;            // column blocks of one tile
    const int64_t total = (int64_t)n_long * nblk;
    // at least 16 column blocks per block: every span starts by building its tile's v
    const int64_t span = max((total + gridDim.x - 1) / gridDim.x, (int64_t)16);
    const int64_t g0 = (int64_t)blockIdx.x * span, g1 = min(g0 + span, total);
    if (g0 >= g1) return;
    const ShrinkSplit sp = shrink_split(n_long, P.tv.d_in, P.KS, P.shrink_grid);

    if (tid == 0) {
        for (int s = 0; s < S; ++s) {
            tc::mbar_init(&full[s], 1);
            tc::mbar_init(&mma_done[s], 1);
            tc::mbar_init(&epi_done[s], XQ * TC_ROWS);
        }
        tc::mbar_init(v_ready, XQ * TC_ROWS);
        *failed = 0;
        tc::fence_mbar_init();
    }
    if (warp == 4 * XQ) {
        tc::tmem_alloc(tmem_slot, C::TMEM_COLS);
        tc::tmem_relinquish();
    }
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    constexpr uint32_t IDESC = tc::instr_desc(128, 64, 0, 1);   // A = v (K-major), B = B_i tile (N-major)

    if (warp == 4 * XQ) {
        // ---- one thread issues each block's MMAs as soon as its tiles have landed; it only ever
        // waits for data (and, at the first column block of a tile, for the tile's v) -------------
        if (lane == 0) {
            int32_t i = 0, piece = 0;
            bool ok = true;
            for (int64_t g = g0; g < g1 && ok; ++piece) {
                const int32_t t = (int32_t)(g / nblk), j0 = (int32_t)(g % nblk);
                const int32_t len = (int32_t)min((int64_t)(nblk - j0), g1 - g);
                const LongTile lt = long_tile(P, t);
                ok = lt.ok && tc::mbar_wait(v_ready, (uint32_t)piece & 1u);
                tc::tc_fence_after();
                const int32_t ksteps = (lt.rank + 15) >> 4;
                const uint32_t vh = tc::smem_u32(Vh), vl = tc::smem_u32(Vl);
                for (int32_t j = 0; j < len && ok; ++j, ++i) {
                    const int s = i % S;
                    ok = !*failed && tc::mbar_wait(&full[s], (uint32_t)(i / S) & 1u);
                    if (!ok) break;
                    tc::tc_fence_after();
                    const uint32_t ba = tc::smem_u32(stages + s * C::STAGE + XT_BYTES);
                    for (int32_t k = 0; k < ksteps; ++k) {
                        // v: two rank groups per step, 2048 bytes apart; B tile: 16 rank rows = 2048 bytes per step
                        const uint64_t bd = tc::smem_desc(ba + k * 2048, 16, 1024, tc::LAYOUT_SW128);
                        tc::umma(tmem + s * 64, tc::smem_desc(vh + k * 4096, 2048, 128, tc::LAYOUT_NONE), bd, IDESC,
                                 k > 0 ? 1u : 0u);
                        tc::umma(tmem + s * 64, tc::smem_desc(vl + k * 4096, 2048, 128, tc::LAYOUT_NONE), bd, IDESC, 1u);
                    }
                    tc::umma_commit(&mma_done[s]);
                }
                g += len;
            }
            if (!ok) *failed = 1;
        }
        __syncwarp();
    } else if (warp == 4 * XQ + 1) {
        // ---- one thread owns the stages' life cycle: it requests the first S blocks, and whenever
        // the epilogue has finished a block it sends the tile out (TMA store), waits until the
        // store has read the stage and requests the block that reuses it.  Every stage that is not
        // being finished or stored therefore has a load in flight. ---------------------------------
        if (lane == 0) {
            const int32_t n = (int32_t)(g1 - g0);
            int32_t issued = 0;
            bool ok = true;
            // cursor of the requests (runs S blocks ahead of the cursor of the stores)
            int32_t lt_t = (int32_t)(g0 / nblk), lj = (int32_t)(g0 % nblk);
            LongTile llt = long_tile(P, lt_t);
            auto issue_load = [&]() {
                const int s = issued % S;
                unsigned char *st = stages + s * C::STAGE;
                tc::mbar_expect_tx(&full[s], XT_BYTES + C::BT_BYTES);
                tc::tma_load_2d(st, &map_yb, lj * 64, llt.t0, &full[s]);
                tc::tma_load_3d(st + XT_BYTES, &map_b, lj * 64, 0, llt.slot, &full[s]);
                ++issued;
                if (++lj == nblk && issued < n) {
                    lj = 0;
                    llt = long_tile(P, ++lt_t);
                }
            };
            ok = llt.ok;
            while (ok && issued < n && issued < S) {
                issue_load();
                ok = llt.ok;
            }
            int32_t st_t = (int32_t)(g0 / nblk), sj = (int32_t)(g0 % nblk);
            LongTile slt = long_tile(P, st_t);
            for (int32_t j = 0; j < n && ok; ++j) {
                const int s = j % S;
                if (!tc::mbar_wait(&epi_done[s], (uint32_t)(j / S) & 1u) || *failed) { ok = false; break; }
                if (slt.rows == TC_ROWS) {
                    tc::tma_store_2d(&map_y, sj * 64, slt.t0, stages + s * C::STAGE);
                    tc::bulk_commit();
                    tc::bulk_wait_read<0>();
                }
                if (issued < n) {
                    issue_load();
                    ok = llt.ok;
                }
                if (++sj == nblk && j + 1 < n) {
                    sj = 0;
                    slt = long_tile(P, ++st_t);
                }
            }
            tc::bulk_wait_read<0>();
            if (!ok) {
                *failed = 1;
                // copies still on their way into this block's shared memory must land before it
                // leaves: the most recent request of every stage is waited for (bounded)
                for (int32_t q = max(issued - S, 0); q < issued; ++q)
                    tc::mbar_wait(&full[q % S], (uint32_t)(q / S) & 1u);
            }
        }
        __syncwarp();
    } else {
        // ---- epilogue warps: thread = row.  At the first column block of a tile they build v; per
        // column block the y_base tile (128-byte swizzle) is updated in place -----------------------
        const int quarter = warp & 3, part = warp >> 2;
        const int m = quarter * 32 + lane;
        int32_t i = 0, piece = 0;
        bool ok = true;
        for (int64_t g = g0; g < g1 && ok; ++piece) {
            const int32_t t = (int32_t)(g / nblk), j0 = (int32_t)(g % nblk);
            const int32_t len = (int32_t)min((int64_t)(nblk - j0), g1 - g);
            const LongTile lt = long_tile(P, t);
            // v = sum of the tile's pieces (in order).  Stored as bf16 high and low parts in the
            // no-swizzle K-major layout: 8 x 8 core matrices of 128 bytes, the core matrix of row
            // group mg and rank group kg at (kg * 16 + mg) * 128 bytes.  The MMAs of the tile
            // before have completed: this thread has waited for the last of them.
            if (part == 0) {
                const int32_t n_pieces = last_block_of(sp, t) - first_block_of(sp, t) + 1;
                const float *src = P.ws + ((int64_t)lt.row0 + m) * P.RS;
                const int64_t ks_stride = (int64_t)P.T * P.RS;
#pragma unroll
                for (int kg = 0; kg < RP / 8; ++kg) {
                    float v[8];
#pragma unroll
                    for (int e = 0; e < 8; ++e) v[e] = 0.0f;
                    for (int32_t q = 0; q < n_pieces && lt.ok && m < lt.rows; ++q) {   // rows past a short tile's end stay zero
                        const float4 a = *reinterpret_cast<const float4 *>(src + q * ks_stride + kg * 8);
                        const float4 b = *reinterpret_cast<const float4 *>(src + q * ks_stride + kg * 8 + 4);
                        v[0] += a.x; v[1] += a.y; v[2] += a.z; v[3] += a.w;
                        v[4] += b.x; v[5] += b.y; v[6] += b.z; v[7] += b.w;
                    }
                    uint32_t hi[4], lo[4];
#pragma unroll
                    for (int e = 0; e < 8; e += 2) {
                        const float v0 = kg * 8 + e < lt.rank ? v[e] : 0.0f;
                        const float v1 = kg * 8 + e + 1 < lt.rank ? v[e + 1] : 0.0f;
                        const __nv_bfloat16 h0 = __float2bfloat16_rn(v0), h1 = __float2bfloat16_rn(v1);
                        hi[e / 2] = pack2(__bfloat162float(h0), __bfloat162float(h1));
                        lo[e / 2] = pack2(v0 - __bfloat162float(h0), v1 - __bfloat162float(h1));
                    }
                    const int off = (kg * 16 + (m >> 3)) * 128 + (m & 7) * 16;
                    *reinterpret_cast<uint4 *>(Vh + off) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
                    *reinterpret_cast<uint4 *>(Vl + off) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
                }
                tc::fence_proxy_async();     // v was written with ordinary stores and is read by the MMA unit
            }
            tc::mbar_arrive(v_ready);
            for (int32_t j = 0; j < len; ++j, ++i) {
                const int s = i % S;
                // all four warps take the same decision (a thread that left alone would strand the
                // others at the named barrier)
                const uint32_t bad =
                    (*failed != 0 || !lt.ok || !tc::mbar_wait(&mma_done[s], (uint32_t)(i / S) & 1u)) ? 1u : 0u;
                uint32_t any_bad;
                asm volatile(
                    "{\n\t.reg .pred p, q;\n\t"
                    "setp.ne.u32 p, %1, 0;\n\t"
                    "bar.red.or.pred q, 1, %2, p;\n\t"
                    "selp.u32 %0, 1, 0, q;\n\t}"
                    : "=r"(any_bad)
                    : "r"(bad), "n"(XQ * TC_ROWS)
                    : "memory");
                if (any_bad) { ok = false; *failed = 1; break; }
                tc::tc_fence_after();
                unsigned char *tile = stages + s * C::STAGE;
#pragma unroll
                for (int cc = 0; cc < 64 / XQ; cc += 16) {
                    const int c = part * (64 / XQ) + cc;
                    uint32_t r[16];
                    tc::tmem_ld16(tmem + ((uint32_t)(quarter * 32) << 16) + s * 64 + c, r);
                    tc::tmem_ld_wait();
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        const int chunk = (c >> 3) + h;
                        uint4 *p = reinterpret_cast<uint4 *>(tile + m * 128 + ((chunk ^ (m & 7)) << 4));
                        float acc[8];
#pragma unroll
                        for (int e = 0; e < 8; ++e) acc[e] = __uint_as_float(r[h * 8 + e]);
                        *p = finish8(acc, *p, lt.scale);
                    }
                }
                tc::tc_fence_before();
                if (lt.rows < TC_ROWS) {
                    // short tile: the rows after it belong to other tokens, so each thread stores its own row
                    const int32_t colb = (j0 + j) * 64;
                    if (m < lt.rows) {
                        __nv_bfloat16 *yrow = P.y + (int64_t)(lt.t0 + m) * P.ldy + colb;
#pragma unroll
                        for (int chunk = part * (8 / XQ); chunk < (part + 1) * (8 / XQ); ++chunk)
                            if (colb + chunk * 8 < P.tv.d_out)
                                *reinterpret_cast<uint4 *>(yrow + chunk * 8) =
                                    *reinterpret_cast<const uint4 *>(tile + m * 128 + ((chunk ^ (m & 7)) << 4));
                    }
                } else {
                    tc::fence_proxy_async();    // the tile is read by the TMA store
                }
                tc::mbar_arrive(&epi_done[s]);  // 128 arrivals: every row of the stage is finished
            }
            g += len;
        }
    }
    tc::tc_fence_before();
    __syncthreads();
    if (tid == 0 && *failed) atomicAdd(&P.pool.status[STATUS_TIMEOUTS], 1);
    if (warp == 4 * XQ) tc::tmem_dealloc(tmem, C::TMEM_COLS);
}

// ---------------------------------------------------------------------------------------------
// host side: tensor maps and launches
// ---------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
    // looked up once per process; a function-local static is initialised under the language's own lock
    static const EncodeTiledFn fn = [] {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            return (EncodeTiledFn)p;
        cudaGetLastError();
        return (EncodeTiledFn) nullptr;
    }();
    return fn;
}

// 2-D bf16 tensor [rows, cols] with a row pitch in elements; box = 64 columns x 128 rows
static bool make_map_2d(CUtensorMap *m, const void *base, int64_t rows, int64_t cols, int64_t ld) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
    cuuint32_t box[2] = {64, (cuuint32_t)TC_ROWS};
    cuuint32_t estr[2] = {1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
// 3-D view of one target's matrices in the pool: [slot][r_max rows][d columns]; box = 64 x box_rows x 1
static bool make_map_3d(CUtensorMap *m, const void *base, int64_t d, int64_t r_max, int64_t slots,
                        int64_t slot_stride, int box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[3] = {(cuuint64_t)d, (cuuint64_t)r_max, (cuuint64_t)slots};
    cuuint64_t strides[2] = {(cuuint64_t)d * 2, (cuuint64_t)slot_stride * 2};
    cuuint32_t box[3] = {64, (cuuint32_t)box_rows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int RP>
static lora_status_t launch_tc_bucket(lora_pool_t *pool, const TcParams &P, const ApplyParams &AP,
                                      cudaStream_t stream) {
    CUtensorMap mx, myb, my, ma, mb;
    const __nv_bfloat16 *w = pool->weights_dev;
    if (!make_map_2d(&mx, AP.x, AP.T, AP.tv.d_in, AP.ldx) || !make_map_2d(&myb, AP.yb, AP.T, AP.tv.d_out, AP.ldyb) ||
        !make_map_2d(&my, AP.y, AP.T, AP.tv.d_out, AP.ldy) ||
        !make_map_3d(&ma, w + AP.tv.off_a, AP.tv.d_in, pool->r_max, pool->num_slots, pool->slot_stride, RP) ||
        !make_map_3d(&mb, w + AP.tv.off_b, AP.tv.d_out, pool->r_max, pool->num_slots, pool->slot_stride, RP))
        return LORA_ERR_INVALID_ARG;

    constexpr int SH_SMEM = SH_STAGES * (XT_BYTES + ((RP * 128 + 1023) & ~1023)) + 256 + 1024;
    bool &attr_done = pool->tc_attr_done[RP == 16 ? 0 : RP == 32 ? 1 : 2];
    if (!attr_done) {
        LORA_CUDA_TRY(cudaFuncSetAttribute(tc_shrink_kernel<RP>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           SH_SMEM));
        LORA_CUDA_TRY(cudaFuncSetAttribute(tc_expand_kernel<RP>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           ExpandCfg<RP>::SMEM));
        attr_done = true;
    }
    tc_shrink_kernel<RP><<<P.shrink_grid, TCS_THREADS, SH_SMEM, stream>>>(P, mx, ma);
    lora_status_t s = count_launch();
    if (s != LORA_OK) return s;
    tc_expand_kernel<RP><<<P.expand_grid, TCX_THREADS, ExpandCfg<RP>::SMEM, stream>>>(P, mb, myb, my);
    return count_launch();
}

bool tc_path_wanted(const lora_pool_t *pool, int32_t T, int32_t tile_m) {
    if (tile_m != TC_ROWS || T < TC_ROWS || pool->tuning[4] == 1 || pool->tuning[0] == 1) return false;
    // Short batches stay on the stream kernel alone (tuning key 4 = 2: these kernels whenever they apply).
    return T / TC_ROWS >= TC_MIN_TILES || pool->tuning[4] == 2;
}

lora_status_t launch_tc_worklist(lora_pool_t *pool, int32_t T, int32_t tile_m, void *meta_dev,
                                 cudaStream_t stream) {
    const MetaLayout L = meta_layout(T, pool->num_slots, tile_m);
    if (L.words > 0x7fffffff) return LORA_ERR_SHAPE;
    TcParams P;
    memset(&P, 0, sizeof(P));
    P.meta = (const int32_t *)meta_dev;
    P.T = T;
    P.moff_perm = (int32_t)L.perm;
    P.moff_desc = (int32_t)L.tile_desc;
    P.list = (int32_t *)meta_dev + L.long_list;
    P.list_cap = L.cap_tile;
    tc_worklist_kernel<<<1, 256, 0, stream>>>(P);
    return count_launch();
}

// Runs the long tiles of a batch.  Returns LORA_OK with *handled = false when the path does not
// apply (no tensor-map support, misaligned operands); the caller then gives every tile to the
// fused kernel.  check_only: decide, launch nothing.
lora_status_t launch_tc_long_tiles(lora_pool_t *pool, const ApplyParams &AP, void *workspace,
                                   size_t workspace_bytes, cudaStream_t stream, bool *handled,
                                   bool check_only) {
    *handled = false;
    if (!AP.meta || AP.tile_m != TC_ROWS || AP.T < TC_ROWS) return LORA_OK;
    if (!tc_path_wanted(pool, AP.T, AP.tile_m)) return LORA_OK;
    if (!encode_fn()) return LORA_OK;
    // TMA wants 16-byte aligned bases and row pitches
    if ((((uintptr_t)AP.x | (uintptr_t)AP.yb | (uintptr_t)AP.y) & 15) || (AP.ldx % 8) || (AP.ldyb % 8) ||
        (AP.ldy % 8))
        return LORA_OK;
    const int32_t RS = rank_bucket(pool->r_max) < 16 ? 16 : rank_bucket(pool->r_max);
    if (!pool->meta_has_list(AP.meta)) return LORA_OK;   // built before the batch qualified (tuning changed)
    const size_t per_split = (size_t)AP.T * RS * sizeof(float);
    if (!workspace || workspace_bytes < per_split || ((uintptr_t)workspace & 15)) return LORA_OK;
    int32_t KS = (int32_t)(workspace_bytes / per_split < 8 ? workspace_bytes / per_split : 8);   // slabs of partials

    TcParams P;
    P.pool = AP.pool;
    P.tv = AP.tv;
    P.meta = AP.meta;
    P.ws = (float *)workspace;
    P.T = AP.T;
    P.RS = RS;
    P.KS = KS;
    const MetaLayout L = meta_layout(AP.T, AP.meta_slots, AP.tile_m);
    if (L.words > 0x7fffffff) return LORA_OK;
    P.moff_perm = (int32_t)L.perm;
    P.moff_desc = (int32_t)L.tile_desc;
    P.target_rows = pool->r_max;
    P.list = const_cast<int32_t *>(AP.meta) + L.long_list;
    P.list_cap = L.cap_tile;
    P.shrink_grid = 2 * pool->sm_count;   // two blocks fit on an SM: the grid fills the GPU exactly once
    // The expand's walk is cut finer: four waves of blocks (two per SM at a time), so that blocks that
    // start late or share their SM with the fused kernel do not leave the others waiting at the end
    // (blocks per SM in the grid 2 / 4 / 8 / 12 / 16: prefill step 577 / 545 / 540 / 553 / 566 us).
    // Tuning key 8 overrides the number of blocks per SM.
    P.expand_grid = (pool->tuning[8] > 0 ? pool->tuning[8] : 8) * pool->sm_count;
    if (check_only) {   // nothing has been launched: the caller only asks whether the path applies
        *handled = true;
        return LORA_OK;
    }

    P.y = AP.y;
    P.ldy = AP.ldy;
    // one pair of launches for every rank: the kernels are sized for the pool's largest rank
    // bucket, and the rows above a slot's rank are zero
    lora_status_t s = RS <= 16   ? launch_tc_bucket<16>(pool, P, AP, stream)
                      : RS == 32 ? launch_tc_bucket<32>(pool, P, AP, stream)
                                 : launch_tc_bucket<64>(pool, P, AP, stream);
    if (s == LORA_OK) *handled = true;
    return s;
}

}  // namespace lora
