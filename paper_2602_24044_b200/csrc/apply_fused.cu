// Fused LoRA forward y = y_base + s_i * (x . A_i) . B_i (paper Section 2.2) in ONE launch for
// every rank of a batch.
//
// A unit is at most 16 token rows of one adapter.  A thread-block cluster owns one unit at a time
// (units cid, cid + G, ... of the batch); block c of the cluster takes the c-th slice of d_in for
// the shrink phase and the c-th slice of d_out for the expand phase.  Inside a block the work of
// all its units is ONE stream of jobs
//     unit 0: shrink chunk 0 .. na-1, expand chunk 0 .. nb-1, unit 1: shrink chunk 0 ...
// and a job is one column chunk: the rank rows of A_i (or B_i), fetched by ONE tiled bulk copy
// (TMA, 128-byte swizzle, the matrix viewed as blocks of 64 columns), plus the unit's rows of x (or
// y_base), one bulk copy per row, into one stage of a small ring of shared-memory buffers
// (mbarrier-signalled).  Few large copies matter: every bulk copy costs the issuing thread and the
// copy engine a fixed time, and a copy per weight row made that time the bottleneck.  A fifth
// warp does nothing but request jobs: it reads the unit records itself, one unit ahead, and refills
// a stage as soon as the four consumer warps have left it (per-stage mbarriers), so issuing copies
// (0.4-0.7 us per job when a consumer warp did it) is off the consumers' critical path, and the
// next job of the stream may belong to the next unit, so the memory latency of
// a unit hides behind the arithmetic of the one before.  The chunk width shrinks as the rank
// grows (256 / 128 / 64 columns for ranks <= 16 / 32 / 64), so a stage is the same size for
// every rank and one launch serves all of them.
//
//   shrink  partial v over the block's d_in slice, the four warps splitting rank tiles and columns,
//           bf16 tensor-core MMA (m16n8k16) with fp32 accumulation carried across chunks in registers;
//   exchange the block partials are summed through distributed shared memory in block order,
//           identically in every block (no global workspace, no float atomics): small units push
//           their partial into every block of the cluster and sum locally, larger ones fetch the
//           partials from the blocks that hold them; the blocks signal each other through
//           mbarriers in each other's shared memory (bounded waits), not the hardware cluster barrier;
//   expand  over the block's d_out slice on the tensor cores, v carried as the sum of two bf16
//           numbers (high and low part, ~16 mantissa bits); scale and residual add fused, y_base
//           read from the job's stage, one rounding to bf16 at the store.
// Every per-row sum is taken in a fixed order that does not depend on which other rows share the
// unit (MMA rows are independent), so a row's result depends only on its inputs.
#include <cstdio>
#include <cstdlib>

#include "apply_common.cuh"

namespace lora {

constexpr int FT = 128;          // consumer threads per block (four warps)
constexpr int FT_ALL = 160;      // plus the warp that requests the jobs
constexpr int UNIT_RING = 4;     // unit records held in shared memory: previous, current, next, next but one
constexpr int RING_ENTRY = 80;   // one record: 16 bytes + 16 row ids
constexpr int SM_RING = 64;      // byte offset of the record ring (mbarriers come first)
constexpr int SM_XBAR = 384;     // mbarrier: every block of the cluster has published its partial
constexpr int SM_YBAR = 392;     // mbarrier: every block of the cluster has read the partials
constexpr int SM_HEADER = 448;   // bytes before the first carved-up buffer
constexpr int MAX_STAGES = 4;
constexpr int W_BYTES = 8192;    // weight tile of a job: rank bucket x chunk width x 2 bytes, for every bucket

// tensor maps of one target: index rows / 8 - 1 for loads of `rows` rank rows (8, 16, .. 64)
struct FusedMaps {
    CUtensorMap a[8], b[8];
};
#ifndef LORA_FUSED_MIN_BLOCKS
#define LORA_FUSED_MIN_BLOCKS 6   // resident blocks per SM the register budget is held to
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
__device__ __forceinline__ void fence_proxy_async() {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)),
                 "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// barrier among the four consumer warps (the requesting warp runs on its own)
__device__ __forceinline__ void consumer_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }
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
// one tile of a 4-D tensor (column in block, rank row, column block, slot) -> shared memory
__device__ __forceinline__ void tma_load_4d(void *dst, const CUtensorMap *map, int c0, int c1, int c2,
                                            int c3, uint64_t *bar) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, "
        "%3, %4, %5}], [%6];" ::"r"(smem_u32(dst)),
        "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(smem_u32(bar))
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
// one arrival on the mbarrier at the same shared-memory offset in block `rank` of the cluster; the
// arriving thread's earlier writes and reads are ordered before it (release at cluster scope)
__device__ __forceinline__ void mbar_arrive_peer(uint64_t *local_bar, uint32_t rank) {
    uint32_t remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(smem_u32(local_bar)), "r"(rank));
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(remote) : "memory");
}
// bounded wait on this block's mbarrier for arrivals from the whole cluster (acquire at cluster scope)
__device__ __forceinline__ bool mbar_wait_cluster(uint64_t *bar, uint32_t parity) {
    for (uint32_t i = 0; i < (1u << 20); ++i) {
        uint32_t ok;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(ok)
            : "r"(smem_u32(bar)), "r"(parity)
            : "memory");
        if (ok) return true;
    }
    return false;
}
// read a float at the same shared-memory offset in block `rank` of the cluster
__device__ __forceinline__ float ld_peer_f32(uint32_t local_addr, uint32_t rank) {
    uint32_t remote;
    float v;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_addr), "r"(rank));
    asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(remote) : "memory");
    return v;
}
// write a float at the same shared-memory offset in block `rank` of the cluster
__device__ __forceinline__ void st_peer_f32(uint32_t local_addr, uint32_t rank, float v) {
    uint32_t remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_addr), "r"(rank));
    asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(remote), "f"(v) : "memory");
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
// work queued before this kernel is complete and visible (no-ops without the launch attribute)
__device__ __forceinline__ void griddep_launch_dependents() {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
__device__ __forceinline__ void griddep_wait() {
    asm volatile("griddepcontrol.wait;" ::: "memory");
}
__device__ __forceinline__ uint32_t lds32(const __nv_bfloat16 *p) {
    return *reinterpret_cast<const uint32_t *>(p);
}
__device__ __forceinline__ uint32_t lds32b(const unsigned char *p) {
    return *reinterpret_cast<const uint32_t *>(p);
}
__device__ __forceinline__ int4 ldg_int4(const int32_t *p) {
    int4 v;
    asm volatile("ld.global.nc.v4.s32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}
__device__ __forceinline__ int32_t ldg_int(const int32_t *p) {
    int32_t v;
    asm volatile("ld.global.nc.s32 %0, [%1];" : "=r"(v) : "l"(p));
    return v;
}

// ---------------------------------------------------------------------------------------------
// units and the record ring
// ---------------------------------------------------------------------------------------------
struct Unit {
    int32_t slot, rank, rows;
    int32_t RP, CW;      // rank bucket (16, 32, 64) and its chunk width (256, 128, 64 columns)
    int32_t rb;          // rank rows a tile load fetches: the rank rounded up to 8
    int32_t na, nb;      // shrink / expand jobs of this block
    float scale;
    bool run;            // the unit has jobs in this launch
};

// record: {slot (-1: token without adapter, -2: past the end), position, rows | tile rows << 8 |
// consecutive ids << 16 | rank << 17, scale bits}
__device__ __forceinline__ Unit decode_unit(const ApplyParams &P, const int4 rec, int32_t a_w,
                                            int32_t b_w) {
    Unit u;
    u.slot = rec.x;
    u.rows = rec.z & 0xff;
    const int32_t tile_rows = (rec.z >> 8) & 0xff, contiguous = (rec.z >> 16) & 1;
    u.rank = (rec.z >> 17) & 0x7f;
    u.scale = __int_as_float(rec.w);
    // runs of consecutive tokens belong to the tensor-core kernels when those ran
    u.run = rec.x >= 0 && u.rows > 0 && u.rank > 0 &&
            !(P.path_filter && contiguous && tile_rows >= P.path_filter);
    const int32_t sh = u.rank <= 16 ? 0 : u.rank <= 32 ? 1 : 2;
    u.rb = (u.rank + 7) & ~7;
    u.RP = 16 << sh;
    u.CW = 256 >> sh;
    u.na = (a_w + u.CW - 1) >> (8 - sh);
    u.nb = (b_w + u.CW - 1) >> (8 - sh);
    return u;
}

struct UnitRegs {   // a record on its way from global memory to the ring (lane 16: record, lanes 0-15: row ids)
    int4 rec;
    int32_t rowid;
};

// Requests the record of unit u.  `cap` bounds the addresses that may be read; whether u is a real
// unit is decided when the record is stored.
__device__ __forceinline__ UnitRegs fetch_unit(const ApplyParams &P, int32_t u, int32_t cap, int lane) {
    UnitRegs m;
    m.rec = make_int4(-2, 0, 0, 0);
    m.rowid = 0;
    if (u >= cap) return m;
    if (P.meta) {
        if (lane == 16) m.rec = ldg_int4(P.meta + P.moff_udesc + 4 * (int64_t)u);
        else if (lane < 16) m.rowid = ldg_int(P.meta + P.moff_uperm + 16 * (int64_t)u + lane);
    } else {
        m.rowid = u;
        if (lane == 16) {
            const int32_t s = ldg_int(P.slot_idx + u);
            m.rec = make_int4(-1, s != -1 ? 1 : 0, 0, 0);   // y = 1: not an adapter-less token either
            if (s >= 0 && s < P.pool.num_slots) {
                const SlotEntry e = P.pool.table[s];
                if (e.loaded)
                    m.rec = make_int4(s, u, 1 | (1 << 8) | (1 << 16) | (e.rank << 17),
                                      __float_as_int(e.scale));
            }
        }
    }
    return m;
}
__device__ __forceinline__ void store_unit(unsigned char *smem, int32_t iter, const UnitRegs &m,
                                           bool real, int lane) {
    unsigned char *e = smem + SM_RING + (iter % UNIT_RING) * RING_ENTRY;
    if (lane == 16) *reinterpret_cast<int4 *>(e) = real ? m.rec : make_int4(-2, 0, 0, 0);
    else if (lane < 16) reinterpret_cast<int32_t *>(e + 16)[lane] = m.rowid;
}

// What every part of a block needs to know about its place and progress.
struct Ctx {
    unsigned char *smem;
    uint64_t *full;            // [n_stages] a job's data has landed
    uint64_t *empty;           // [n_stages] the four consumer warps are done with the stage
    int32_t cid, G, n_units;   // cluster index, clusters in the grid, units in the batch
    uint32_t crank, csize;
    int32_t a_lo, a_hi, b_lo, b_hi;   // this block's column slices of d_in and d_out
    int32_t ci;                // unit iteration the consumers work on
    int32_t cq;                // jobs consumed so far
    int32_t k_run;             // units this block has exchanged partials for (phase of the two mbarriers)
    bool ok;                   // no wait has expired
};

// Requesting warp: one job into stage `st`.  mode 0: whole job; 1: only the weight tile (and the
// byte count of the whole job); 2: only the token rows of a job whose tile was requested in mode 1.
// Lane l < 16 holds the id of the unit's row l in `rowid`.
__device__ __forceinline__ void request_job(const ApplyParams &P, const FusedMaps &M, const Ctx &cx,
                                            const Unit &un, int32_t j, int st, int32_t rowid, int lane,
                                            int mode) {
    unsigned char *ws = cx.smem + P.off_stage + st * P.stage_bytes;
    const bool shrink = j < un.na;
    const int32_t c = shrink ? j : j - un.na;
    const int32_t col0 = (shrink ? cx.a_lo : cx.b_lo) + c * un.CW;   // a multiple of 64
    const int32_t ncols = min(un.CW, (shrink ? cx.a_hi : cx.b_hi) - col0);
    const int32_t pitch = un.CW + 8;
    const CUtensorMap *map = shrink ? &M.a[(un.rb >> 3) - 1] : &M.b[(un.rb >> 3) - 1];
    const __nv_bfloat16 *tok = (shrink ? P.x : P.yb) + col0;
    const int64_t tld = shrink ? P.ldx : P.ldyb;
    __nv_bfloat16 *ts = reinterpret_cast<__nv_bfloat16 *>(ws + W_BYTES);
    if (lane == 0 && mode != 2) {
        // the tile load always delivers its whole box: rb rows of CW columns
        mbar_expect_tx(&cx.full[st], (uint32_t)un.rb * (uint32_t)un.CW * 2u +
                                         (uint32_t)un.rows * (uint32_t)ncols * 2u);
        tma_load_4d(ws, map, 0, 0, col0 >> 6, un.slot, &cx.full[st]);
    }
    __syncwarp();
    if (lane < un.rows && mode != 1)
        bulk_g2s(ts + lane * pitch, tok + (int64_t)rowid * tld, (uint32_t)ncols * 2u, &cx.full[st]);
}

// The requesting warp: walks the same units as the consumers (it reads the records itself, one
// unit ahead, into registers), and keeps the ring full: a job is requested as soon as the four
// consumer warps have left its stage, whatever they are doing meanwhile, so the time it takes to
// issue copies is off their critical path.
__device__ __forceinline__ void producer_warp(const ApplyParams &P, const FusedMaps &M, Ctx &cx, int lane) {
    const int32_t S = P.n_stages;
    int32_t n_units = P.meta ? ldg_int(P.meta + H_NPIECE) : P.T;
    UnitRegs cur = fetch_unit(P, cx.cid, P.units, lane);
    if (n_units > P.units) n_units = P.units;
    int32_t q = 0, skip = 0;
    bool ok = true;
    for (int32_t i = 0;; ++i) {
        const int32_t u = cx.cid + i * cx.G;
        if (u >= n_units) {
            if (i == 0 && P.early) griddep_wait();
            break;
        }
        const UnitRegs nxt = fetch_unit(P, u + cx.G, n_units, lane);   // the next unit's record, meanwhile
        int4 rec;
        rec.x = __shfl_sync(0xffffffffu, cur.rec.x, 16);
        rec.y = __shfl_sync(0xffffffffu, cur.rec.y, 16);
        rec.z = __shfl_sync(0xffffffffu, cur.rec.z, 16);
        rec.w = __shfl_sync(0xffffffffu, cur.rec.w, 16);
        const Unit un = decode_unit(P, rec, cx.a_hi - cx.a_lo, cx.b_hi - cx.b_lo);
        const int32_t njobs = un.run ? un.na + un.nb : 0;
        if (i == 0 && P.early) {
            // The kernel before this one may still be running: the pool may be read (the host
            // vouches for it), the activations not yet.  Weight tiles of the first jobs now, their
            // token rows after the wait.
            skip = njobs < S ? njobs : S;
            for (int32_t j = 0; j < skip; ++j) request_job(P, M, cx, un, j, j, cur.rowid, lane, 1);
            griddep_wait();
            for (int32_t j = 0; j < skip; ++j) request_job(P, M, cx, un, j, j, cur.rowid, lane, 2);
        }
        for (int32_t j = 0; j < njobs; ++j, ++q) {
            if (i == 0 && j < skip) continue;
            const int st = q % S;
            if (q >= S) ok = mbar_wait(&cx.empty[st], (uint32_t)(q / S - 1) & 1u) && ok;
            request_job(P, M, cx, un, j, st, cur.rowid, lane, 0);
        }
        cur = nxt;
    }
    if (!ok && lane == 0) atomicAdd(&P.pool.status[STATUS_TIMEOUTS], 1);
}

// Consumers: wait for the data of the next job; returns its stage.
__device__ __forceinline__ const unsigned char *acquire_job(const ApplyParams &P, Ctx &cx) {
    const int st = cx.cq % P.n_stages;
    cx.ok = mbar_wait(&cx.full[st], (uint32_t)(cx.cq / P.n_stages) & 1u) && cx.ok;
    return cx.smem + P.off_stage + st * P.stage_bytes;
}
// Consumers: this warp is done with the job's stage.
__device__ __forceinline__ void release_job(const ApplyParams &P, Ctx &cx, int lane) {
    __syncwarp();
    if (lane == 0) mbar_arrive(&cx.empty[cx.cq % P.n_stages]);
    ++cx.cq;
}

// RP: rank bucket of the unit; H: 1 when a unit holds at most 8 rows, 2 when rows 8..15 can be occupied.
template <int RP, int H>
__device__ __forceinline__ void unit_body(const ApplyParams &P, const Unit &un, const int32_t *rowidx,
                                          Ctx &cx) {
    constexpr int CW = 4096 / RP;      // columns per job
    constexpr int PW = CW + 8;         // row pitch of the token rows: +16 B against bank conflicts
    constexpr int PV = RP + 8;         // pitch of the bf16 copies of v
    // shrink: the four warps split the rank tiles WN ways and the chunk's columns WK ways, so that
    // every warp owns two rank tiles of 8 and 64 columns of every job, whatever the bucket
    constexpr int WN = RP / 16, WK = 4 / WN;
    constexpr int KW = CW / WK;        // = 64 columns per warp and job
    constexpr int NW = CW / 4;         // expand: columns per warp and job
    constexpr int NT_E = NW / 8;       // expand: column tiles of 8 per warp
    constexpr int mrows = 8 * H;
    constexpr bool hi_rows = H == 2;

    unsigned char *smem = cx.smem;
    float *part = reinterpret_cast<float *>(smem + P.off_part);     // [WK][mrows][RP] = mrows x 64 floats
    float *vpart = reinterpret_cast<float *>(smem + P.off_vpart);   // [mrows][RP], read by the peers
    float *vall = vpart;   // push mode: [cluster size][mrows][RP], written by the peers
    __nv_bfloat16 *Vh = reinterpret_cast<__nv_bfloat16 *>(smem + P.off_vh);   // [mrows][PV]
    __nv_bfloat16 *Vl = reinterpret_cast<__nv_bfloat16 *>(smem + P.off_vl);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, t = lane & 3;
    const int32_t rows = un.rows, rank = un.rank;
    const int32_t rank16 = (rank + 15) & ~15;
    // A weight tile is stored as blocks of 64 columns, rb rows of 128 bytes each, the 16-byte
    // chunks of a row exchanged by the row number's low three bits (128-byte swizzle).
    const uint32_t blk_bytes = (uint32_t)un.rb * 128u;

    // ---- shrink: warp (wk, wn) takes columns [wk*KW, (wk+1)*KW) of every chunk and rank tiles 2wn, 2wn+1
    const int wk = warp % WK, wn = warp / WK;
    float acc[2][4];
#pragma unroll
    for (int i = 0; i < 2; ++i) acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0.0f;
    for (int32_t c = 0; c < un.na; ++c) {
        const unsigned char *As = acquire_job(P, cx);   // tile of A_i, then [mrows][PW] rows of x
        const __nv_bfloat16 *X = reinterpret_cast<const __nv_bfloat16 *>(As + W_BYTES);
        const int32_t ncols = min(CW, cx.a_hi - (cx.a_lo + c * CW));
#pragma unroll
        for (int ks = 0; ks < KW; ks += 16) {
            const int kk = wk * KW + ks;
            if (kk < ncols) {
                const bool full = ncols - kk >= 16;   // else only 8 columns are left
                uint32_t a[4];
                a[0] = lds32(X + g * PW + kk + 2 * t);
                a[1] = hi_rows ? lds32(X + (g + 8) * PW + kk + 2 * t) : 0u;
                a[2] = full ? lds32(X + g * PW + kk + 8 + 2 * t) : 0u;
                a[3] = (full && hi_rows) ? lds32(X + (g + 8) * PW + kk + 8 + 2 * t) : 0u;
                const unsigned char *ab = As + (uint32_t)(kk >> 6) * blk_bytes + g * 128 + 4 * t;
                const uint32_t ch = (uint32_t)(kk & 63) >> 3;   // even
#pragma unroll
                for (int i = 0; i < 2; ++i) {
                    const int nt = wn * 2 + i;
                    mma16816(acc[i], a, lds32b(ab + nt * 1024 + ((ch ^ (uint32_t)g) << 4)),
                             full ? lds32b(ab + nt * 1024 + (((ch + 1) ^ (uint32_t)g) << 4)) : 0u);
                }
            }
        }
        release_job(P, cx, lane);
    }
    // The exchange is signalled with two mbarriers per block instead of the cluster-wide hardware
    // barrier (0.8 us a round even without skew): every block of the cluster arrives on every block's
    // barrier, once when its partial is published, once when it has read the partials.
    uint64_t *xbar = reinterpret_cast<uint64_t *>(smem + SM_XBAR);
    uint64_t *ybar = reinterpret_cast<uint64_t *>(smem + SM_YBAR);
    // the peers have finished reading the previous unit's partials before they are overwritten
    if (cx.k_run > 0) cx.ok = mbar_wait_cluster(ybar, (uint32_t)(cx.k_run - 1) & 1u) && cx.ok;
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        float *p0 = part + (wk * mrows + g) * RP + (wn * 2 + i) * 8 + 2 * t;
        *reinterpret_cast<float2 *>(p0) = make_float2(acc[i][0], acc[i][1]);
        if (hi_rows) *reinterpret_cast<float2 *>(p0 + 8 * RP) = make_float2(acc[i][2], acc[i][3]);
    }
    consumer_sync();
    // block partial: the column splits' sums in order
    for (int i = tid; i < mrows * RP; i += FT) {
        const int r = i / RP;
        if (r < rows) {
            float v = part[i];
#pragma unroll
            for (int w = 1; w < WK; ++w) v += part[w * mrows * RP + i];
            if (P.push) {
                // small units: every block hands its partial to all blocks (remote stores need no
                // answer), so that after the barrier the sum is taken from local shared memory
                const uint32_t dst = smem_u32(vall + ((int)cx.crank * mrows * RP + i));
                for (uint32_t q = 0; q < cx.csize; ++q) st_peer_f32(dst, q, v);
            } else {
                vpart[i] = v;
            }
        }
    }
    // ---- exchange: every block sums all blocks' partials in block order -------------------------
    // one arrival per block and peer: thread q tells block q, after the block's threads have met
    // (its release then covers all their writes)
    consumer_sync();
    if (tid < (int)cx.csize) mbar_arrive_peer(xbar, (uint32_t)tid);
    cx.ok = mbar_wait_cluster(xbar, (uint32_t)cx.k_run & 1u) && cx.ok;
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
                    pv[q] = q >= cx.csize ? 0.0f
                            : P.push     ? vall[(int)q * mrows * RP + m * RP + k]
                                         : ld_peer_f32(vp_addr + (uint32_t)(m * RP + k) * 4u, q);
#pragma unroll
                for (uint32_t q = 0; q < 8; ++q) v += pv[q];
            }
            const __nv_bfloat16 hi = __float2bfloat16_rn(v);
            Vh[m * PV + k] = hi;
            Vl[m * PV + k] = __float2bfloat16_rn(v - __bfloat162float(hi));
        }
    }
    ++cx.k_run;
    consumer_sync();
    // done reading the partials; the matching wait comes before the next overwrite (or the exit)
    if (tid < (int)cx.csize) mbar_arrive_peer(ybar, (uint32_t)tid);

    // ---- expand: warp w takes columns [w*NW, (w+1)*NW) of every chunk ---------------------------
    const float s = un.scale;
    for (int32_t c = 0; c < un.nb; ++c) {
        const unsigned char *Bs = acquire_job(P, cx);   // tile of B_i, then [mrows][PW] rows of y_base
        const __nv_bfloat16 *Ys = reinterpret_cast<const __nv_bfloat16 *>(Bs + W_BYTES);
        const int32_t col0 = cx.b_lo + c * CW, ncols = min(CW, cx.b_hi - col0);
        const int base = warp * NW;
        // column tiles in groups of at most four: 16 accumulator registers at a time
        constexpr int NG = NT_E < 4 ? NT_E : 4;
#pragma unroll
        for (int j0 = 0; j0 < NT_E; j0 += NG) {
            const int gbase = base + j0 * 8;
            if (gbase >= ncols) break;
            float ex[NG][4];
#pragma unroll
            for (int j = 0; j < NG; ++j) ex[j][0] = ex[j][1] = ex[j][2] = ex[j][3] = 0.0f;
            const __nv_bfloat16 *vh = Vh + g * PV + 2 * t;
            const __nv_bfloat16 *vl = Vl + g * PV + 2 * t;
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
                for (int np = 0; np < NG / 2; ++np) {
                    // matrices: (k 0..7, tile 2np), (k 8..15, tile 2np), (k 0..7, 2np+1), (k 8..15, 2np+1)
                    const int mi = lane >> 3;
                    const int col = gbase + (np * 2 + (mi >> 1)) * 8;
                    const unsigned char *bp = Bs + (uint32_t)(col >> 6) * blk_bytes +
                                              (ks + (mi & 1) * 8 + (lane & 7)) * 128 +
                                              ((((uint32_t)(col & 63) >> 3) ^ (uint32_t)(lane & 7)) << 4);
                    uint32_t b[4];
                    ldmatrix_x4_trans(b, smem_u32(bp));
                    mma16816(ex[np * 2], ah, b[0], b[1]);
                    mma16816(ex[np * 2], al, b[0], b[1]);
                    mma16816(ex[np * 2 + 1], ah, b[2], b[3]);
                    mma16816(ex[np * 2 + 1], al, b[2], b[3]);
                }
            }
            // epilogue straight from the accumulator layout: each lane owns two adjacent columns of
            // a row per column tile; a quad covers 16 contiguous bytes
#pragma unroll
            for (int h = 0; h < H; ++h) {
                const int32_t m = g + 8 * h;
                if (m < rows && cx.ok) {
                    __nv_bfloat16 *yrow = P.y + (int64_t)rowidx[m] * P.ldy + col0 + gbase + 2 * t;
                    const __nv_bfloat16 *ybrow = Ys + m * PW + gbase + 2 * t;
#pragma unroll
                    for (int j = 0; j < NG; ++j) {
                        if (gbase + j * 8 < ncols) {
                            const uint32_t w = lds32(ybrow + j * 8);
                            const float y0 = fmaf(s, ex[j][2 * h], __uint_as_float(w << 16));
                            const float y1 = fmaf(s, ex[j][2 * h + 1], __uint_as_float(w & 0xffff0000u));
                            *reinterpret_cast<uint32_t *>(yrow + j * 8) = pack2(y0, y1);
                        }
                    }
                }
            }
        }
        release_job(P, cx, lane);
    }
}

// H: 1 when a unit holds at most 8 rows (decode tiles, single tokens), 2 otherwise.
template <int H>
__global__ void __launch_bounds__(FT_ALL, LORA_FUSED_MIN_BLOCKS)
fused_kernel(const ApplyParams P, const __grid_constant__ FusedMaps M) {
    extern __shared__ __align__(1024) unsigned char smem[];
    Ctx cx;
    cx.smem = smem;
    cx.full = reinterpret_cast<uint64_t *>(smem);
    cx.csize = cluster_nctarank();
    cx.crank = cluster_ctarank();
    cx.cid = (int32_t)(blockIdx.x / cx.csize);
    cx.G = (int32_t)(gridDim.x / cx.csize);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // the swizzled tiles want 1024-byte aligned stages; the carve-up assumes an aligned base
    if (smem_u32(smem) & 1023u) {
        if (tid == 0 && blockIdx.x == 0) atomicAdd(&P.pool.status[STATUS_TIMEOUTS], 1);
        return;
    }

    // barriers; the next lines touch no memory another kernel writes
    cx.empty = cx.full + MAX_STAGES;
    if (tid == 0) {
        for (int s = 0; s < P.n_stages; ++s) {
            mbar_init(&cx.full[s], 1);
            mbar_init(&cx.empty[s], 4);
        }
        mbar_init(reinterpret_cast<uint64_t *>(smem + SM_XBAR), cx.csize);
        mbar_init(reinterpret_cast<uint64_t *>(smem + SM_YBAR), cx.csize);
        fence_mbar_init();
    }
    // the only cluster-wide hardware barrier: no block signals a peer whose barriers are not set up
    cluster_arrive();
    // this block's column slices (multiples of 64 columns: tile loads address whole column blocks)
    {
        const int32_t cs64 = (int32_t)cx.csize * 64;
        const int32_t Wa = (P.tv.d_in + cs64 - 1) / cs64 * 64, Wb = (P.tv.d_out + cs64 - 1) / cs64 * 64;
        cx.a_lo = min((int32_t)cx.crank * Wa, P.tv.d_in);
        cx.a_hi = min(cx.a_lo + Wa, P.tv.d_in);
        cx.b_lo = min((int32_t)cx.crank * Wb, P.tv.d_out);
        cx.b_hi = min(cx.b_lo + Wb, P.tv.d_out);
    }
    // zeros in every stage (rows above a unit's rank are never copied, and what they hold is
    // multiplied by zeros of v, so it has to be finite)
    for (int i = tid; i < P.n_stages * P.stage_bytes / 16; i += FT_ALL)
        reinterpret_cast<uint4 *>(smem + P.off_stage)[i] = make_uint4(0, 0, 0, 0);
    fence_proxy_async();   // the stages are written by bulk copies from here on
    // Under programmatic dependent launch this kernel may start while the one before it on the
    // stream is still running.  Activations are only touched after griddep_wait().  The unit
    // records and the pool were complete before that kernel started when P.early is set (the host
    // sets it only then), so they are read, and the first weight tiles requested, ahead of the wait.
    if (!P.early) griddep_wait();
    __syncthreads();
    cluster_wait();
    cx.ci = 0;
    cx.cq = 0;
    cx.k_run = 0;
    cx.ok = true;
    if (warp == 4) {   // the requesting warp goes its own way from here
        producer_warp(P, M, cx, lane);
        return;
    }
    {
        // the number of units and the records of this cluster's first two units, side by side
        UnitRegs m0, m1;
        if (warp == 3) {
            m0 = fetch_unit(P, cx.cid, P.units, lane);
            m1 = fetch_unit(P, cx.cid + cx.G, P.units, lane);
        }
        cx.n_units = P.meta ? ldg_int(P.meta + H_NPIECE) : P.T;
        if (cx.n_units > P.units) cx.n_units = P.units;
        if (warp == 3) {
            store_unit(smem, 0, m0, cx.cid < cx.n_units, lane);
            store_unit(smem, 1, m1, cx.cid + cx.G < cx.n_units, lane);
        }
    }
    consumer_sync();
    if (P.early) griddep_wait();
    // the next kernel on the stream may be scheduled from here on: everything older than this
    // kernel is complete
    griddep_launch_dependents();

    for (;; ++cx.ci) {
        const int32_t u = cx.cid + cx.ci * cx.G;
        if (u >= cx.n_units) break;
        // the record of the unit after next is requested now and stored when this unit is done
        UnitRegs mn;
        if (warp == 3) mn = fetch_unit(P, u + 2 * cx.G, cx.n_units, lane);
        const unsigned char *e = smem + SM_RING + (cx.ci % UNIT_RING) * RING_ENTRY;
        const int4 rec = *reinterpret_cast<const int4 *>(e);
        const int32_t *rowidx = reinterpret_cast<const int32_t *>(e + 16);
        const Unit un = decode_unit(P, rec, cx.a_hi - cx.a_lo, cx.b_hi - cx.b_lo);
        if (un.run) {
            if (un.RP == 16) unit_body<16, H>(P, un, rowidx, cx);
            else if (un.RP == 32) unit_body<32, H>(P, un, rowidx, cx);
            else unit_body<64, H>(P, un, rowidx, cx);
        } else if (!P.meta && rec.x == -1) {   // per-token mode: this token has no adapter
            if (cx.crank == 0 && tid == 0 && rec.y) atomicAdd(&P.pool.status[STATUS_INVALID_TOKENS], 1);
            if (!P.in_place) copy_rows(P, rowidx, 1, (int32_t)cx.crank, (int32_t)cx.csize, FT);
        }
        if (warp == 3) store_unit(smem, cx.ci + 2, mn, true, lane);
        consumer_sync();   // the new record is visible; nobody reads the current one any more
    }
    if (!cx.ok && tid == 0) atomicAdd(&P.pool.status[STATUS_TIMEOUTS], 1);

    // rows that take no adapter: y_base -> y, 16 rows per cluster step (grouped mode, out of place)
    if (P.meta && !P.in_place) {
        int32_t *rowidx = reinterpret_cast<int32_t *>(smem + SM_RING + 16);
        const int32_t n_active = __ldg(P.meta + H_NACTIVE);
        for (int32_t first = cx.cid * 16; first < P.T - n_active; first += cx.G * 16) {
            const int32_t rows = min(16, P.T - n_active - first);
            consumer_sync();
            if (tid < rows) rowidx[tid] = __ldg(P.meta + P.moff_perm + n_active + first + tid);
            consumer_sync();
            copy_rows(P, rowidx, rows, (int32_t)cx.crank, (int32_t)cx.csize, FT);
        }
    }
    // no block leaves while a peer may still read its partials or signal its barriers
    if (cx.k_run > 0 && !mbar_wait_cluster(reinterpret_cast<uint64_t *>(smem + SM_YBAR),
                                           (uint32_t)(cx.k_run - 1) & 1u) && tid == 0)
        atomicAdd(&P.pool.status[STATUS_TIMEOUTS], 1);
}

// ---------------------------------------------------------------------------------------------
// host side: tensor maps (built once per target, kept in the pool handle) and launch
// ---------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

static EncodeTiledFn tiled_encoder() {
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
        else
            cudaGetLastError();
    }
    return fn;
}

// One target's matrix family in the pool, [slot][r_max rows][d columns], viewed as a 4-D tensor
// (column inside a 64-column block, rank row, column block, slot); box = 64 x rows x blocks x 1.
// The last column block of a row may reach into the next row (or, in the last row of the last
// slot, into the pool's slack bytes); such columns are never used.
static bool weight_map(CUtensorMap *m, const void *base, int64_t d, int64_t r_max, int64_t slots,
                       int64_t slot_stride, int rows, int blocks) {
    EncodeTiledFn fn = tiled_encoder();
    if (!fn) return false;
    cuuint64_t dims[4] = {64, (cuuint64_t)r_max, (cuuint64_t)((d + 63) / 64), (cuuint64_t)slots};
    cuuint64_t strides[3] = {(cuuint64_t)d * 2, 128, (cuuint64_t)slot_stride * 2};
    cuuint32_t box[4] = {64, (cuuint32_t)rows, (cuuint32_t)blocks, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

static lora_status_t target_maps(lora_pool_t *pool, const ApplyParams &P, const FusedMaps **out) {
    static_assert(sizeof(lora_pool::TargetMaps) == sizeof(FusedMaps), "same layout");
    int32_t target = -1;
    for (int32_t t = 0; t < pool->num_targets; ++t)
        if (pool->target_views[t].off_a == P.tv.off_a) target = t;
    if (target < 0) return LORA_ERR_INVALID_ARG;
    if (pool->fused_maps.empty()) {
        pool->fused_maps.resize(pool->num_targets);
        pool->fused_maps_ready.assign(pool->num_targets, 0);
    }
    lora_pool::TargetMaps &tm = pool->fused_maps[target];
    if (!pool->fused_maps_ready[target]) {
        const __nv_bfloat16 *w = pool->weights_dev;
        for (int i = 0; i < 8; ++i) {
            const int rows = 8 * (i + 1);
            if (rows > ((pool->r_max + 7) & ~7)) break;   // no slot holds that many rank rows
            const int blocks = rows <= 16 ? 4 : rows <= 32 ? 2 : 1;   // chunk width 256 / 128 / 64
            if (!weight_map(&tm.a[i], w + P.tv.off_a, P.tv.d_in, pool->r_max, pool->num_slots,
                            pool->slot_stride, rows, blocks) ||
                !weight_map(&tm.b[i], w + P.tv.off_b, P.tv.d_out, pool->r_max, pool->num_slots,
                            pool->slot_stride, rows, blocks))
                return cuda_fail(cudaErrorNotSupported);
        }
        pool->fused_maps_ready[target] = 1;
    }
    *out = reinterpret_cast<const FusedMaps *>(&tm);
    return LORA_OK;
}

// Shared-memory carve-up and launch.  The buffers are sized for the largest rank bucket that has
// ever been loaded into the pool.
template <int H>
static lora_status_t launch_h(lora_pool_t *pool, ApplyParams P, int32_t C, const FusedMaps *maps,
                              cudaStream_t stream) {
    auto kern = fused_kernel<H>;
    const int32_t mrows = 8 * H;
    const int32_t RPmax = (pool->bucket_mask & 8u) ? 64 : (pool->bucket_mask & 4u) ? 32 : 16;
    // a stage: the weight tile, then the token rows at the widest chunk (rank bucket 16)
    const int32_t stage = (W_BYTES + mrows * (256 + 8) * 2 + 1023) & ~1023;
    int32_t S = pool->tuning[5];
    if (S < 2 || S > MAX_STAGES) S = 2;   // two stages and more resident blocks beat deeper rings
    int32_t o = SM_HEADER;
    P.off_part = o;   o += mrows * 64 * 4;
    // the partials of all blocks of the cluster fit beside each other when units are small: then
    // they are pushed to every block instead of fetched by every block
    P.push = (8 * mrows * RPmax * 4 <= 4096 && pool->tuning[6] != 1) ? 1 : 0;
    P.off_vpart = o;  o += (P.push ? 8 : 1) * mrows * RPmax * 4;
    P.off_vh = o;     o += mrows * (RPmax + 8) * 2;
    P.off_vl = o;     o += mrows * (RPmax + 8) * 2;
    o = (o + 1023) & ~1023;
    P.off_stage = o;  o += S * stage;
    P.stage_bytes = stage;
    P.n_stages = S;
    const int32_t smem = o;

    const int dv = device_index(pool->device);
    static int32_t attr_smem[DEVICE_TABLE] = {};
    if (smem > attr_smem[dv]) {
        LORA_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        attr_smem[dv] = smem;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3(FT_ALL, 1, 1);
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
    // Programmatic dependent launch (tuning key 2: 0 = when allowed, 2 = never).  Allowed for
    // grouped batches whose table has already been read by an earlier apply: that apply was fully
    // ordered behind the build, so the table is complete before this kernel can start.
    const bool fresh = P.meta ? pool->take_fresh(P.meta) : true;
    P.early = (P.meta && !fresh && pool->tuning[2] != 2) ? 1 : 0;
    // Without `early` the attribute still lets the blocks become resident and set up their shared
    // memory while the kernel before them drains; they read nothing until it has completed.
    const unsigned n_attrs = pool->tuning[2] != 2 ? 2 : 1;

    // Grid: no more clusters than can be resident at once (each loops over its units), so no
    // cluster of an over-sized grid waits for a slot only to find that its unit does not exist.
    static int32_t occ_smem_d[DEVICE_TABLE] = {}, occ_c_d[DEVICE_TABLE] = {}, occ_clusters_d[DEVICE_TABLE] = {};
    int32_t &occ_smem = occ_smem_d[dv], &occ_c = occ_c_d[dv], &occ_clusters = occ_clusters_d[dv];
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
            fprintf(stderr, "lora_b200: fused kernel rows<=%d ranks<=%d: smem %d B (%d stages of %d B), cluster %d, "
                    "resident clusters %d\n", mrows, RPmax, smem, S, stage, C, n);
    }
    cfg.numAttrs = n_attrs;
    int32_t want = P.units;   // units, or 16-row copy steps if there are more of those
    if (P.meta && !P.in_place && (P.T + 15) / 16 > want) want = (P.T + 15) / 16;
    int32_t G = occ_clusters > 0 && occ_clusters < want ? occ_clusters : want;
    if (pool->tuning[3] > 0 && pool->tuning[3] < G) G = pool->tuning[3];
    cfg.gridDim = dim3((unsigned)(G * C), 1, 1);
    LORA_CUDA_TRY(cudaLaunchKernelEx(&cfg, kern, P, *maps));
    return count_launch();
}

lora_status_t launch_fused(lora_pool_t *pool, ApplyParams &P, cudaStream_t stream) {
    const int32_t tile_m = P.meta ? P.tile_m : 1;
    P.moff_perm = P.moff_udesc = P.moff_uperm = 0;
    P.units = P.T;
    if (P.meta) {
        const MetaLayout L = meta_layout(P.T, P.meta_slots, P.tile_m);
        if (L.words > 0x7fffffff) return LORA_ERR_SHAPE;
        P.moff_perm = (int32_t)L.perm;
        P.moff_udesc = (int32_t)L.unit_desc;
        P.moff_uperm = (int32_t)L.unit_perm;
        P.units = L.cap_unit;
    }
    if (P.units < 1) P.units = 1;
    // cluster size: as wide a split as the projection supports
    int32_t C = pool->tuning[1];
    if (C != 1 && C != 2 && C != 4 && C != 8) {
        C = 8;
        while (C > 1 && (P.tv.d_in / C < 256 || P.tv.d_out / C < 128)) C >>= 1;
    }
    const FusedMaps *maps = nullptr;
    lora_status_t s = target_maps(pool, P, &maps);
    if (s != LORA_OK) return s;
    return tile_m <= 8 ? launch_h<1>(pool, P, C, maps, stream) : launch_h<2>(pool, P, C, maps, stream);
}

}  // namespace lora
