// Fused LoRA forward y = y_base + s_i * (x . A_i) . B_i (paper Section 2.2) in ONE launch for
// every rank of a batch and for up to eight independent projections that share the batch (the
// adapted projections of one transformer layer: q, k, v, o, gate, up, down).
//
// A unit is at most 16 token rows of one adapter in one projection.  A thread-block cluster owns
// one unit at a time (global units cid, cid + G, ... of the launch; the units of projection 0
// come first, then those of projection 1, ...); block c of the cluster takes the c-th slice of
// d_in for the shrink phase and the c-th slice of d_out for the expand phase.  Inside a block the
// work of all its units is ONE stream of jobs, software-pipelined by one unit:
//     shrink(u0)  shrink(u1)  expand(u0)  shrink(u2)  expand(u1)  ...
// so that the exchange of a unit's partial sums across the cluster (the one step that has to wait
// for the slowest block) runs under the next unit's shrink.  A job is one column chunk: the rank
// rows of A_i (or B_i), fetched by ONE tiled bulk copy (TMA, 128-byte swizzle, the matrix viewed as
// blocks of 64 columns), plus the unit's rows of x (or y_base), one bulk copy per row, into one
// stage of a small ring of shared-memory buffers (mbarrier-signalled).  A fifth warp does nothing
// but request jobs: it reads the unit records itself, one unit ahead, refills a stage as soon as
// the four consumer warps have left it, and asks the L2 cache for the tiles and rows of the next
// unit ahead of time.  The chunk width shrinks as the rank grows (256 / 128 / 64 columns for
// ranks <= 16 / 32 / 64), so a stage is the same size for every rank and one launch serves all.
//
//   shrink  partial v over the block's d_in slice, the four warps splitting rank tiles and columns,
//           bf16 tensor-core MMA (m16n8k16) with fp32 accumulation carried across chunks in registers;
//   exchange the block partials are summed through distributed shared memory in block order,
//           identically in every block (no global workspace, no float atomics): small units push
//           their partial into every block of the cluster and sum locally, larger ones fetch the
//           partials from the blocks that hold them; two sets of buffers and mbarriers alternate
//           between consecutive units, the blocks signal each other through mbarriers in each
//           other's shared memory (bounded waits);
//   expand  over the block's d_out slice on the tensor cores, v carried as the sum of two bf16
//           numbers (high and low part, ~16 mantissa bits); scale and residual add fused, y_base
//           read from the job's stage, one rounding to bf16 at the store.
// Every per-row sum is taken in a fixed order that does not depend on which other rows share the
// unit (MMA rows are independent), so a row's result depends only on its inputs.
//
// Consecutive launches overlap (programmatic dependent launch): a kernel lets its successor
// become resident at once; the successor reads the unit records and the pool, requests its first
// weight tiles and prefetches the rest into L2 while this kernel is still running, and touches
// activations only after griddepcontrol.wait.  A wait that runs out marks the block dead: it
// stops touching its peers, drains its own copies and goes to the closing cluster barrier.
#include <cstring>

#include "apply_common.cuh"
#include "fused_ptx.cuh"

namespace lora {

constexpr int FT = 128;          // consumer threads per block (four warps)
constexpr int FT_ALL = 160;      // plus the warp that requests the jobs
constexpr int UNIT_RING = 4;     // unit records held in shared memory: previous, current, next, next but one
constexpr int RING_ENTRY = 80;   // one record: 16 bytes + 16 row ids
constexpr int SM_RING = 64;      // byte offset of the record ring (the ring's mbarriers come first)
constexpr int SM_XBAR = 384;     // two mbarriers: every block of the cluster has published its partial
constexpr int SM_YBAR = 400;     // two mbarriers: every block of the cluster has read the partials
constexpr int SM_DEAD = 416;     // int32: a bounded wait of this block has expired
constexpr int SM_ISSUED = 420;   // int32: jobs requested so far (read when a dead block drains its copies)
constexpr int SM_HEADER = 448;   // bytes before the first carved-up buffer
constexpr int MAX_STAGES = 4;
constexpr int W_BYTES = 8192;    // weight tile of a job: rank bucket x chunk width x 2 bytes, for every bucket
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
    int32_t prefetch;          // ask L2 for the next unit's tiles and rows ahead of the ring
    int32_t late_trigger;      // decode kernel: let the successor in only once this kernel's blocks are set up
    int32_t copy_idle;         // some projection is out of place: rows without adapter are copied
    int32_t off_part, off_vpart, vbuf_bytes, off_vh, off_vl;   // warp partials, exchange buffers (x2), v as bf16 high / low parts
    int32_t off_w, off_tok, tok_bytes, n_stages;               // ring of job buffers: weight tiles, token rows
    int32_t moff_perm, moff_udesc, moff_uperm;                 // word offsets: perm, unit records, unit row ids
    FusedItem item[MAX_ITEMS];
};

// ---------------------------------------------------------------------------------------------
// units and the record ring
// ---------------------------------------------------------------------------------------------
struct Unit {
    int32_t slot, rank, rows;
    int32_t item;        // projection of the launch
    int32_t RP, CW;      // rank bucket (16, 32, 64) and its chunk width (256, 128, 64 columns)
    int32_t rb;          // rank rows a tile load fetches: the rank rounded up to 8
    int32_t na, nb;      // shrink / expand jobs of this block
    int32_t a_lo, a_hi, b_lo, b_hi;   // this block's column slices of d_in and d_out
    float scale;
    bool run;            // the unit has jobs in this launch
};

// Position in the launch's unit list: unit g is unit u of projection `item`.  A cluster walks
// g = cid, cid + G, ...; the split into (item, u) is carried along instead of divided out.
struct Walk {
    int32_t g, item, u;
    __device__ __forceinline__ void start(int32_t cid, int32_t n_units) {
        g = u = cid;
        item = 0;
        while (u >= n_units) { u -= n_units; ++item; }
    }
    __device__ __forceinline__ Walk next(int32_t G, int32_t n_units) const {
        Walk w;
        w.g = g + G; w.u = u + G; w.item = item;
        while (w.u >= n_units) { w.u -= n_units; ++w.item; }
        return w;
    }
};

// What every part of a block needs to know about its place and progress.
struct Ctx {
    unsigned char *smem;
    uint64_t *full;            // [n_stages] a job's data has landed
    uint64_t *empty;           // [n_stages] the four consumer warps are done with the stage
    int32_t cid, G;            // cluster index, clusters in the grid
    int32_t n_units, total;    // units per projection, units of the launch
    uint32_t crank, csize;
    int32_t st;                // ring stage of the next job (consumers: to consume, requesting warp: to fill)
    uint32_t ph;               // how often the ring has wrapped, low bit = the stage's phase
    int32_t kp, kr;            // units whose partials this block has published / summed
    bool ok;                   // no wait has expired
};

__device__ __forceinline__ volatile int32_t *dead_flag(unsigned char *smem) {
    return reinterpret_cast<volatile int32_t *>(smem + SM_DEAD);
}
__device__ __forceinline__ void ring_advance(const FusedParams &P, Ctx &cx) {
    if (++cx.st == P.n_stages) {
        cx.st = 0;
        ++cx.ph;
    }
}

// record: {slot (-1: token without adapter, -2: past the end), position, rows | tile rows << 8 |
// consecutive ids << 16 | rank << 17, scale bits}
__device__ __forceinline__ Unit decode_unit(const FusedParams &P, const Ctx &cx, const int4 rec, int32_t item) {
    Unit u;
    u.slot = rec.x;
    u.rows = rec.z & 0xff;
    const int32_t tile_rows = (rec.z >> 8) & 0xff, contiguous = (rec.z >> 16) & 1;
    u.rank = (rec.z >> 17) & 0x7f;
    u.scale = __int_as_float(rec.w);
    u.item = min(item, P.n_items - 1);
    const FusedItem &it = P.item[u.item];
    u.a_lo = min((int32_t)cx.crank * it.wa, it.d_in);
    u.a_hi = min(u.a_lo + it.wa, it.d_in);
    u.b_lo = min((int32_t)cx.crank * it.wb, it.d_out);
    u.b_hi = min(u.b_lo + it.wb, it.d_out);
    // runs of consecutive tokens belong to the tensor-core kernels when those ran
    u.run = rec.x >= 0 && u.rows > 0 && u.rank > 0 &&
            !(P.path_filter && contiguous && tile_rows >= P.path_filter);
    const int32_t sh = u.rank <= 16 ? 0 : u.rank <= 32 ? 1 : 2;
    u.rb = (u.rank + 7) & ~7;
    u.RP = 16 << sh;
    u.CW = 256 >> sh;
    u.na = (u.a_hi - u.a_lo + u.CW - 1) >> (8 - sh);
    u.nb = (u.b_hi - u.b_lo + u.CW - 1) >> (8 - sh);
    return u;
}

struct UnitRegs {   // a record on its way from global memory to the ring (lane 16: record, lanes 0-15: row ids)
    int4 rec;
    int32_t rowid;
};

// Requests the record of unit u of the batch (`valid`: the address may be read; whether the unit
// is a real one is decided when the record is used).
__device__ __forceinline__ UnitRegs fetch_unit(const FusedParams &P, int32_t u, bool valid, int lane) {
    UnitRegs m;
    m.rec = make_int4(-2, 0, 0, 0);
    m.rowid = 0;
    if (!valid) return m;
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
    unsigned char *e = smem + SM_RING + (iter & (UNIT_RING - 1)) * RING_ENTRY;
    if (lane == 16) *reinterpret_cast<int4 *>(e) = real ? m.rec : make_int4(-2, 0, 0, 0);
    else if (lane < 16) reinterpret_cast<int32_t *>(e + 16)[lane] = m.rowid;
}
__device__ __forceinline__ int4 bcast_rec(const UnitRegs &m) {
    int4 rec;
    rec.x = __shfl_sync(0xffffffffu, m.rec.x, 16);
    rec.y = __shfl_sync(0xffffffffu, m.rec.y, 16);
    rec.z = __shfl_sync(0xffffffffu, m.rec.z, 16);
    rec.w = __shfl_sync(0xffffffffu, m.rec.w, 16);
    return rec;
}
// The unit count of the batch as the kernel sees it, and the launch's total.
__device__ __forceinline__ void set_counts(const FusedParams &P, Ctx &cx, int32_t n_units) {
    if (n_units > P.units_cap) n_units = P.units_cap;
    cx.total = n_units * P.n_items;
    cx.n_units = n_units < 1 ? 1 : n_units;
}

// ---------------------------------------------------------------------------------------------
// the requesting warp
// ---------------------------------------------------------------------------------------------
// One job into stage `st`.  mode 0: whole job; 1: only the weight tile (and the byte count of the
// whole job); 2: only the token rows of a job whose tile was requested in mode 1.  Job j of a unit
// is shrink chunk j for j < na, else expand chunk j - na.  Lane l < 16 holds the id of the unit's
// row l in `rowid`.
__device__ __forceinline__ void request_job(const FusedParams &P, const Ctx &cx, const Unit &un, int32_t j,
                                            int st, int32_t rowid, int lane, int mode) {
    const FusedItem &it = P.item[un.item];
    unsigned char *ws = cx.smem + P.off_w + st * W_BYTES;
    __nv_bfloat16 *ts = reinterpret_cast<__nv_bfloat16 *>(cx.smem + P.off_tok + st * P.tok_bytes);
    const bool shrink = j < un.na;
    const int32_t c = shrink ? j : j - un.na;
    const int32_t col0 = (shrink ? un.a_lo : un.b_lo) + c * un.CW;   // a multiple of 64
    const int32_t ncols = min(un.CW, (shrink ? un.a_hi : un.b_hi) - col0);
    const CUtensorMap *map = P.maps + it.map_base + (shrink ? 0 : 8) + (un.rb >> 3) - 1;
    const __nv_bfloat16 *tok = (shrink ? it.x : it.yb) + col0;
    const int64_t tld = shrink ? it.ldx : it.ldyb;
    if (lane == 0 && mode != 2) {
        // the tile load always delivers its whole box: rb rows of CW columns
        mbar_expect_tx(&cx.full[st], (uint32_t)un.rb * (uint32_t)un.CW * 2u +
                                         (uint32_t)un.rows * (uint32_t)ncols * 2u);
        tma_load_4d(ws, map, 0, 0, col0 >> 6, un.slot, &cx.full[st]);
    }
    __syncwarp();
    if (lane < un.rows && mode != 1)
        bulk_g2s(ts + lane * TOK_PITCH, tok + (int64_t)rowid * tld, (uint32_t)ncols * 2u, &cx.full[st]);
}

// Hints to L2 for a whole unit: every weight tile of the block's jobs from job `first` on (one lane
// per tile) and the block's slices of the unit's x and y_base rows.  Values are not consumed, so
// this may run before the preceding kernel has finished.
__device__ __forceinline__ void prefetch_unit(const FusedParams &P, const Unit &un, int32_t first,
                                              int32_t rowid, int lane) {
    if (!un.run) return;
    const FusedItem &it = P.item[un.item];
    const CUtensorMap *ma = P.maps + it.map_base + (un.rb >> 3) - 1;
    for (int32_t j = first + lane; j < un.na + un.nb; j += 32) {
        const bool shrink = j < un.na;
        const int32_t col0 = shrink ? un.a_lo + j * un.CW : un.b_lo + (j - un.na) * un.CW;
        tma_prefetch_4d(shrink ? ma : ma + 8, 0, 0, col0 >> 6, un.slot);
    }
    if (lane < un.rows) {
        if (un.a_hi > un.a_lo)
            bulk_prefetch_l2(it.x + (int64_t)rowid * it.ldx + un.a_lo, (uint32_t)(un.a_hi - un.a_lo) * 2u);
        if (un.b_hi > un.b_lo)
            bulk_prefetch_l2(it.yb + (int64_t)rowid * it.ldyb + un.b_lo, (uint32_t)(un.b_hi - un.b_lo) * 2u);
    }
}

// Walks the same units as the consumers in the same pipelined order (it reads the records itself,
// one unit ahead, into registers) and keeps the ring full: a job is requested as soon as the four
// consumer warps have left its stage, whatever they are doing meanwhile.
__device__ __forceinline__ void producer_warp(const FusedParams &P, Ctx &cx, int lane) {
    const int32_t S = P.n_stages;
    volatile int32_t *dead = dead_flag(cx.smem);
    volatile int32_t *issued = reinterpret_cast<volatile int32_t *>(cx.smem + SM_ISSUED);
    // the unit count and (speculatively, as if the table were full) the first record, side by side
    const int32_t n_hdr = P.meta ? ldg_int(P.meta + H_NPIECE) : P.T;
    UnitRegs cur = fetch_unit(P, cx.cid, P.n_items == 1 && cx.cid < P.units_cap, lane);
    set_counts(P, cx, n_hdr);
    Walk w;
    w.start(cx.cid, cx.n_units);
    if (P.n_items > 1) cur = fetch_unit(P, w.u, w.g < cx.total, lane);
    int32_t q = 0, skip = 0;
    bool have_pend = false, waited = !P.early;
    Unit pend;
    int32_t pend_rowid = 0;

    for (int32_t i = 0;; ++i) {
        const bool real = w.g < cx.total;
        if (!real && !have_pend) break;
        const Walk wn = w.next(cx.G, cx.n_units);
        const bool next_real = real && wn.g < cx.total;
        const UnitRegs nxt = fetch_unit(P, wn.u, next_real, lane);   // the next unit's record, meanwhile
        Unit un = decode_unit(P, cx, bcast_rec(cur), w.item);
        if (!real) un.run = false;   // past the end: only the last unit's expand jobs are left
        if (i == 0) {
            if (P.early) {
                // The kernel before this one may still be running: the pool may be read (the host
                // vouches for it), the activations not yet.  Weight tiles of the first jobs now, their
                // token rows after the wait; everything else of this and the next unit as L2 hints.
                skip = !un.run ? 0 : un.na < S ? un.na : S;
                for (int32_t j = 0; j < skip; ++j) request_job(P, cx, un, j, j, cur.rowid, lane, 1);
            }
            if (P.prefetch) prefetch_unit(P, un, skip, cur.rowid, lane);
        }
        const bool hint_next = P.prefetch && next_real;
        const bool hint_first = i == 0 && !waited;   // time to spare before the wait returns
        Unit un_next;
        if (hint_next) un_next = decode_unit(P, cx, bcast_rec(nxt), wn.item);
        if (hint_next && hint_first) prefetch_unit(P, un_next, 0, nxt.rowid, lane);
        if (!waited) {
            griddep_wait();
            waited = true;
            for (int32_t j = 0; j < skip; ++j) {
                request_job(P, cx, un, j, j, cur.rowid, lane, 2);
                ring_advance(P, cx);
            }
            if (lane == 0) *issued = skip;
            q = skip;
        }
        // this step's jobs in ring order: the unit's shrink chunks, then the pending unit's expand chunks
        const int32_t ja = un.run ? un.na : 0, jb = have_pend ? pend.nb : 0;
        for (int32_t k = (i == 0 ? skip : 0); k < ja + jb; ++k) {
            if (k == ja && hint_next && !hint_first) prefetch_unit(P, un_next, 0, nxt.rowid, lane);
            if (q >= S && cx.ok) {
                cx.ok = mbar_wait(&cx.empty[cx.st], (cx.ph - 1u) & 1u);
                if (!cx.ok) *dead = 1;
            }
            if (cx.ok && !*dead) {
                if (k < ja) request_job(P, cx, un, k, cx.st, cur.rowid, lane, 0);
                else request_job(P, cx, pend, pend.na + k - ja, cx.st, pend_rowid, lane, 0);
                if (lane == 0) *issued = q + 1;
            }
            ++q;
            ring_advance(P, cx);
        }
        if (jb == 0 && hint_next && !hint_first) prefetch_unit(P, un_next, 0, nxt.rowid, lane);
        have_pend = un.run;
        pend = un;
        pend_rowid = cur.rowid;
        if (!real) break;
        cur = nxt;
        w = wn;
    }
    if (!waited) griddep_wait();
    if (!cx.ok && lane == 0) atomicAdd(&P.pool.status[STATUS_TIMEOUTS], 1);
}

// ---------------------------------------------------------------------------------------------
// the consumer warps
// ---------------------------------------------------------------------------------------------
// wait for the data of the next job; returns its stage number
__device__ __forceinline__ int acquire_job(const FusedParams &P, Ctx &cx) {
    if (cx.ok) {
        cx.ok = mbar_wait(&cx.full[cx.st], cx.ph & 1u);
        if (!cx.ok) *dead_flag(cx.smem) = 1;
    }
    return cx.st;
}
// this warp is done with the job's stage
__device__ __forceinline__ void release_job(const FusedParams &P, Ctx &cx, int lane) {
    __syncwarp();
    if (lane == 0 && cx.ok) mbar_arrive(&cx.empty[cx.st]);
    ring_advance(P, cx);
}

// Shrink of one unit over this block's slice of d_in, then the block's partial is made available
// to the cluster (buffer set kp & 1).  RP: rank bucket; H: 1 when a unit holds at most 8 rows,
// 2 when rows 8..15 can be occupied.
template <int RP, int H>
__device__ __forceinline__ void shrink_unit(const FusedParams &P, const Unit &un, Ctx &cx) {
    constexpr int CW = 4096 / RP;      // columns per job
    constexpr int PW = TOK_PITCH;      // row pitch of the token rows
    // the four warps split the rank tiles WN ways and the chunk's columns WK ways, so that every
    // warp owns two rank tiles of 8 and 64 columns of every job (one column block), whatever the bucket
    constexpr int WN = RP / 16, WK = 4 / WN;
    constexpr int mrows = 8 * H;
    constexpr bool hi_rows = H == 2;
    static_assert(CW / WK == 64, "a warp's share of a job is one block of 64 columns");

    unsigned char *smem = cx.smem;
    float *part = reinterpret_cast<float *>(smem + P.off_part);     // [WK][mrows][RP] = mrows x 64 floats
    const int b = cx.kp & 1;
    float *vbuf = reinterpret_cast<float *>(smem + P.off_vpart + b * P.vbuf_bytes);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, t = lane & 3;
    const int32_t rows = un.rows;
    // A weight tile is stored as blocks of 64 columns, rb rows of 128 bytes each, the 16-byte
    // chunks of a row exchanged by the row number's low three bits (128-byte swizzle).
    const uint32_t blk_bytes = (uint32_t)un.rb * 128u;

    // warp (wk, wn) takes column block wk of every chunk and rank tiles 2wn, 2wn+1
    const int wk = warp % WK, wn = warp / WK;
    // Operand fragments come by ldmatrix.  Lane l names row (l & 7) of 8x8 matrix (l >> 3).
    //  weights: matrices (tile 2wn, k 0-7) (tile 2wn, k 8-15) (tile 2wn+1, k 0-7) (tile 2wn+1, k 8-15);
    //           rank row n = 16 wn + 8 (mi >> 1) + r sits at n * 128 bytes of the column block, its
    //           16-byte chunk c at ((c ^ r) << 4); c = 2 (ks / 16) + (mi & 1), whose even part is
    //           folded in per step with one XOR
    //  tokens:  matrices (rows 0-7, k 0-7) (rows 8-15, k 0-7) (rows 0-7, k 8-15) (rows 8-15, k 8-15)
    const int mi = lane >> 3, r = lane & 7;
    const uint32_t w_lane = (uint32_t)(16 * wn + 8 * (mi >> 1) + r) * 128u + (uint32_t)(((mi & 1) ^ r) << 4);
    const uint32_t x_lane = hi_rows ? (uint32_t)(((mi & 1) * 8 + r) * PW + (mi >> 1) * 8) * 2u
                                    : (uint32_t)(r * PW + (mi & 1) * 8) * 2u;
    float acc[2][4];
#pragma unroll
    for (int i = 0; i < 2; ++i) acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0.0f;
    for (int32_t c = 0; c < un.na; ++c) {
        const int st = acquire_job(P, cx);
        const uint32_t As = smem_u32(smem + P.off_w + st * W_BYTES) + (uint32_t)wk * blk_bytes + w_lane;
        const uint32_t X = smem_u32(smem + P.off_tok + st * P.tok_bytes) + (uint32_t)(wk * 64 * 2) + x_lane;
        const int32_t ncols = min(CW, un.a_hi - (un.a_lo + c * CW)) - wk * 64;   // of this warp's block
        if (cx.ok && ncols >= 64) {
#pragma unroll
            for (int ks = 0; ks < 64; ks += 16) {
                uint32_t a[4], bw[4];
                if (hi_rows) {
                    ldmatrix_x4(a, X + ks * 2);
                } else {
                    ldmatrix_x2(a[0], a[2], X + ks * 2);
                    a[1] = a[3] = 0u;
                }
                ldmatrix_x4(bw, As ^ (uint32_t)((ks >> 3) << 4));
                mma16816(acc[0], a, bw[0], bw[1]);
                mma16816(acc[1], a, bw[2], bw[3]);
            }
        } else if (cx.ok && ncols > 0) {
            // ragged end of the slice: columns past the end hold neither x nor this adapter's weights
#pragma unroll
            for (int ks = 0; ks < 64; ks += 16) {
                if (ks < ncols) {
                    const bool full = ncols - ks >= 16;   // else only 8 columns are left
                    uint32_t a[4], bw[4];
                    if (hi_rows) {
                        ldmatrix_x4(a, X + ks * 2);
                    } else {
                        ldmatrix_x2(a[0], a[2], X + ks * 2);
                        a[1] = a[3] = 0u;
                    }
                    ldmatrix_x4(bw, As ^ (uint32_t)((ks >> 3) << 4));
                    if (!full) a[2] = a[3] = bw[1] = bw[3] = 0u;
                    mma16816(acc[0], a, bw[0], bw[1]);
                    mma16816(acc[1], a, bw[2], bw[3]);
                }
            }
        }
        release_job(P, cx, lane);
    }
    // The exchange is signalled with mbarriers in the blocks' shared memory instead of the
    // cluster-wide hardware barrier: every block of the cluster arrives on every block's barrier,
    // once when its partial is published, once when it has read the partials.  Buffer set b was
    // last used two units ago: the peers have finished reading it before it is overwritten.
    uint64_t *xbar = reinterpret_cast<uint64_t *>(smem + SM_XBAR) + b;
    uint64_t *ybar = reinterpret_cast<uint64_t *>(smem + SM_YBAR) + b;
    if (cx.kp >= 2 && cx.ok) {
        cx.ok = mbar_wait_cluster(ybar, (uint32_t)((cx.kp - 2) >> 1) & 1u);
        if (!cx.ok) *dead_flag(smem) = 1;
    }
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        float *p0 = part + (wk * mrows + g) * RP + (wn * 2 + i) * 8 + 2 * t;
        *reinterpret_cast<float2 *>(p0) = make_float2(acc[i][0], acc[i][1]);
        if (hi_rows) *reinterpret_cast<float2 *>(p0 + 8 * RP) = make_float2(acc[i][2], acc[i][3]);
    }
    consumer_sync();
    if (*dead_flag(smem)) cx.ok = false;
    // block partial: the column splits' sums in order
    if (cx.ok) {
        for (int i = tid; i < mrows * RP; i += FT) {
            const int rr = i / RP;
            if (rr < rows) {
                float v = part[i];
#pragma unroll
                for (int w = 1; w < WK; ++w) v += part[w * mrows * RP + i];
                if (P.push) {
                    // small units: every block hands its partial to all blocks (remote stores need no
                    // answer), so that after the signal the sum is taken from local shared memory
                    const uint32_t dst = smem_u32(vbuf + ((int)cx.crank * mrows * RP + i));
                    for (uint32_t q = 0; q < cx.csize; ++q) st_peer_f32(dst, q, v);
                } else {
                    vbuf[i] = v;
                }
            }
        }
    }
    // one arrival per block and peer: thread q tells block q, after the block's threads have met
    // (its release then covers all their writes)
    consumer_sync();
    if (cx.ok && tid < (int)cx.csize) mbar_arrive_peer(xbar, (uint32_t)tid);
    ++cx.kp;
}

// The other half of a unit: the cluster's partials are summed in block order (buffer set kr & 1),
// then the expand over this block's slice of d_out with the fused epilogue.
template <int RP, int H>
__device__ __forceinline__ void expand_unit(const FusedParams &P, const Unit &un, const int32_t *rowidx,
                                         Ctx &cx) {
    constexpr int CW = 4096 / RP;      // columns per job
    constexpr int PW = TOK_PITCH;
    constexpr int PV = RP + 8;         // pitch of the bf16 copies of v
    constexpr int NW = CW / 4;         // columns per warp and job
    constexpr int NT_E = NW / 8;       // column tiles of 8 per warp
    constexpr int KT = RP / 16;        // k steps of 16 ranks the bucket can have
    constexpr int mrows = 8 * H;
    constexpr bool hi_rows = H == 2;

    unsigned char *smem = cx.smem;
    const FusedItem &it = P.item[un.item];
    const int b = cx.kr & 1;
    const float *vbuf = reinterpret_cast<const float *>(smem + P.off_vpart + b * P.vbuf_bytes);
    __nv_bfloat16 *Vh = reinterpret_cast<__nv_bfloat16 *>(smem + P.off_vh);   // [mrows][PV]
    __nv_bfloat16 *Vl = reinterpret_cast<__nv_bfloat16 *>(smem + P.off_vl);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, t = lane & 3;
    const int32_t rows = un.rows, rank = un.rank;
    const int32_t rank16 = (rank + 15) & ~15;
    const uint32_t blk_bytes = (uint32_t)un.rb * 128u;
    uint64_t *xbar = reinterpret_cast<uint64_t *>(smem + SM_XBAR) + b;
    uint64_t *ybar = reinterpret_cast<uint64_t *>(smem + SM_YBAR) + b;

    // ---- exchange: every block sums all blocks' partials in block order -------------------------
    if (cx.ok) {
        cx.ok = mbar_wait_cluster(xbar, (uint32_t)(cx.kr >> 1) & 1u);
        if (!cx.ok) *dead_flag(smem) = 1;
    }
    if (cx.ok) {
        const uint32_t vp_addr = smem_u32(vbuf);
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
                            : P.push     ? vbuf[(int)q * mrows * RP + m * RP + k]
                                         : ld_peer_f32(vp_addr + (uint32_t)(m * RP + k) * 4u, q);
#pragma unroll
                for (uint32_t q = 0; q < 8; ++q) v += pv[q];
            }
            const __nv_bfloat16 hi = __float2bfloat16_rn(v);
            Vh[m * PV + k] = hi;
            Vl[m * PV + k] = __float2bfloat16_rn(v - __bfloat162float(hi));
        }
    }
    consumer_sync();
    if (*dead_flag(smem)) cx.ok = false;
    // done reading the partials; the matching wait comes before buffer set b is written again
    if (cx.ok && tid < (int)cx.csize) mbar_arrive_peer(ybar, (uint32_t)tid);
    ++cx.kr;

    // ---- expand: warp w takes columns [w*NW, (w+1)*NW) of every chunk ---------------------------
    // v as MMA row operand, high and low parts; for the smallest bucket (one step of 16 ranks) the
    // fragments stay in registers for all of the unit's jobs
    uint32_t ah[KT == 1 ? 4 : 1], al[KT == 1 ? 4 : 1];
    const __nv_bfloat16 *vh = Vh + g * PV + 2 * t;
    const __nv_bfloat16 *vl = Vl + g * PV + 2 * t;
    if (KT == 1) {
        ah[0] = lds32(vh);
        ah[1] = hi_rows ? lds32(vh + 8 * PV) : 0u;
        ah[2] = lds32(vh + 8);
        ah[3] = hi_rows ? lds32(vh + 8 * PV + 8) : 0u;
        al[0] = lds32(vl);
        al[1] = hi_rows ? lds32(vl + 8 * PV) : 0u;
        al[2] = lds32(vl + 8);
        al[3] = hi_rows ? lds32(vl + 8 * PV + 8) : 0u;
    }
    // B_i fragments by ldmatrix (transposing): lane l names rank row ks + 8 (mi & 1) + r of column
    // tile 2 np + (mi >> 1); the tile's 16-byte chunk c sits at ((c ^ r) << 4), the even part of c
    // is folded in per tile pair with one XOR
    const int mi = lane >> 3, r = lane & 7;
    const uint32_t b_lane = (uint32_t)((mi & 1) * 8 + r) * 128u + (uint32_t)(((mi >> 1) ^ r) << 4);
    // this lane's output rows: g (and g + 8), columns 2t, 2t+1 of every column tile
    const bool row0 = g < rows, row1 = hi_rows && g + 8 < rows;
    __nv_bfloat16 *y0p = it.y + (int64_t)(row0 ? rowidx[g] : 0) * it.ldy + un.b_lo + warp * NW + 2 * t;
    __nv_bfloat16 *y1p = it.y + (int64_t)(row1 ? rowidx[g + 8] : 0) * it.ldy + un.b_lo + warp * NW + 2 * t;
    const uint32_t ys_lane = (uint32_t)(g * PW + warp * NW + 2 * t) * 2u;
    const float s = un.scale;
    // the column block of this warp's first tile and the tile's chunk number inside it
    constexpr int TPB = 8;   // column tiles per 64-column block
    for (int32_t c = 0; c < un.nb; ++c) {
        const int st = acquire_job(P, cx);
        const uint32_t Bs = smem_u32(smem + P.off_w + st * W_BYTES) + b_lane;
        const uint32_t Ys = smem_u32(smem + P.off_tok + st * P.tok_bytes) + ys_lane;
        const int32_t ncols = min(CW, un.b_hi - (un.b_lo + c * CW)) - warp * NW;   // of this warp's columns
        if (cx.ok && ncols > 0) {
#pragma unroll
            for (int np = 0; np < NT_E / 2; ++np) {
                // tiles 2np, 2np+1 of this warp: columns warp*NW + 16 np .. + 15 of the chunk
                if (NT_E > 2 && 16 * np >= ncols) break;
                const int tile0 = 0;   // (placeholder for readability: tile index inside the warp's columns is 2 np)
                (void)tile0;
                float ex[2][4];
#pragma unroll
                for (int j = 0; j < 2; ++j) ex[j][0] = ex[j][1] = ex[j][2] = ex[j][3] = 0.0f;
                // absolute tile number in the chunk: warp * NT_E + 2 np; its column block and chunk
                const uint32_t tabs = (uint32_t)(warp * NT_E + 2 * np);
                const uint32_t baddr = Bs + (tabs / TPB) * blk_bytes;
                const uint32_t cx4 = (tabs % TPB) << 4;
#pragma unroll
                for (int kt = 0; kt < KT; ++kt) {
                    const int ks = kt * 16;
                    if (KT > 1 && ks >= rank16) break;
                    uint32_t fh[4], fl[4];
                    if (KT == 1) {
#pragma unroll
                        for (int q = 0; q < 4; ++q) { fh[q] = ah[q]; fl[q] = al[q]; }
                    } else {
                        fh[0] = lds32(vh + ks);
                        fh[1] = hi_rows ? lds32(vh + 8 * PV + ks) : 0u;
                        fh[2] = lds32(vh + ks + 8);
                        fh[3] = hi_rows ? lds32(vh + 8 * PV + ks + 8) : 0u;
                        fl[0] = lds32(vl + ks);
                        fl[1] = hi_rows ? lds32(vl + 8 * PV + ks) : 0u;
                        fl[2] = lds32(vl + ks + 8);
                        fl[3] = hi_rows ? lds32(vl + 8 * PV + ks + 8) : 0u;
                    }
                    uint32_t bb[4];
                    ldmatrix_x4_trans(bb, (baddr + (uint32_t)ks * 128u) ^ cx4);
                    // Rank rows ks+8 .. ks+15 were only copied when the tile has them; what the
                    // stage holds there otherwise belongs to an earlier job (possibly another
                    // adapter's weights) and must not meet the MMA, not even multiplied by zero.
                    if (ks + 8 >= un.rb) bb[1] = bb[3] = 0u;
                    mma16816(ex[0], fh, bb[0], bb[1]);
                    mma16816(ex[0], fl, bb[0], bb[1]);
                    mma16816(ex[1], fh, bb[2], bb[3]);
                    mma16816(ex[1], fl, bb[2], bb[3]);
                }
                // epilogue straight from the accumulator layout: each lane owns two adjacent columns of
                // a row per column tile; a quad covers 16 contiguous bytes
#pragma unroll
                for (int j = 0; j < 2; ++j) {
                    const int coff = (2 * np + j) * 8;   // column offset inside the warp's columns
                    if (coff < ncols) {
                        if (row0) {
                            uint32_t w;
                            asm volatile("ld.shared.b32 %0, [%1];" : "=r"(w) : "r"(Ys + coff * 2));
                            const float a0 = fmaf(s, ex[j][0], __uint_as_float(w << 16));
                            const float a1 = fmaf(s, ex[j][1], __uint_as_float(w & 0xffff0000u));
                            *reinterpret_cast<uint32_t *>(y0p + c * CW + coff) = pack2(a0, a1);
                        }
                        if (row1) {
                            uint32_t w;
                            asm volatile("ld.shared.b32 %0, [%1];" : "=r"(w) : "r"(Ys + (8 * PW + coff) * 2));
                            const float a0 = fmaf(s, ex[j][2], __uint_as_float(w << 16));
                            const float a1 = fmaf(s, ex[j][3], __uint_as_float(w & 0xffff0000u));
                            *reinterpret_cast<uint32_t *>(y1p + c * CW + coff) = pack2(a0, a1);
                        }
                    }
                }
            }
        }
        release_job(P, cx, lane);
    }
}

template <int H>
__device__ __forceinline__ void shrink_dispatch(const FusedParams &P, const Unit &un, Ctx &cx) {
    if (un.RP == 16) shrink_unit<16, H>(P, un, cx);
    else if (un.RP == 32) shrink_unit<32, H>(P, un, cx);
    else shrink_unit<64, H>(P, un, cx);
}
template <int H>
__device__ __forceinline__ void expand_dispatch(const FusedParams &P, const Unit &un, const int32_t *rowidx,
                                                Ctx &cx) {
    if (un.RP == 16) expand_unit<16, H>(P, un, rowidx, cx);
    else if (un.RP == 32) expand_unit<32, H>(P, un, rowidx, cx);
    else expand_unit<64, H>(P, un, rowidx, cx);
}

// y_base -> y for rows that take no adapter (out-of-place projections only); the columns are
// split over the blocks of the cluster, the consumer threads do the copying.
__device__ __forceinline__ void copy_rows_item(const FusedItem &it, const int32_t *rowidx, int32_t rows,
                                               int32_t part, int32_t parts) {
    const int32_t vecs = it.d_out / 8;
    for (int32_t m = 0; m < rows; ++m) {
        const __nv_bfloat16 *src = it.yb + (int64_t)rowidx[m] * it.ldyb;
        __nv_bfloat16 *dst = it.y + (int64_t)rowidx[m] * it.ldy;
        for (int32_t v = part * FT + threadIdx.x; v < vecs; v += parts * FT)
            reinterpret_cast<uint4 *>(dst)[v] = ldg16(src + (int64_t)v * 8);
    }
}

template <int H>
__device__ __forceinline__ void consumer_warps(const FusedParams &P, Ctx &cx) {
    unsigned char *smem = cx.smem;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    Walk w;
    {
        // the number of units and (speculatively, as if the table were full) the records of this
        // cluster's first two units, side by side
        const int32_t n_hdr = P.meta ? ldg_int(P.meta + H_NPIECE) : P.T;
        UnitRegs m0, m1;
        const bool spec = P.n_items == 1;
        if (warp == 3) {
            m0 = fetch_unit(P, cx.cid, spec && cx.cid < P.units_cap, lane);
            m1 = fetch_unit(P, cx.cid + cx.G, spec && cx.cid + cx.G < P.units_cap, lane);
        }
        set_counts(P, cx, n_hdr);
        w.start(cx.cid, cx.n_units);
        const Walk w1 = w.next(cx.G, cx.n_units);
        if (warp == 3) {
            if (!spec) {
                m0 = fetch_unit(P, w.u, w.g < cx.total, lane);
                m1 = fetch_unit(P, w1.u, w1.g < cx.total, lane);
            }
            store_unit(smem, 0, m0, w.g < cx.total, lane);
            store_unit(smem, 1, m1, w1.g < cx.total, lane);
        }
    }
    consumer_sync();
    if (P.early) griddep_wait();

    // the unit whose expand half is still to run: its ring entry and projection
    int32_t pend_i = -1, pend_item = 0;
    auto entry_of = [&](int32_t i) { return smem + SM_RING + (i & (UNIT_RING - 1)) * RING_ENTRY; };
    auto run_pending = [&]() {
        if (pend_i < 0) return;
        const unsigned char *e = entry_of(pend_i);
        const Unit up = decode_unit(P, cx, *reinterpret_cast<const int4 *>(e), pend_item);
        expand_dispatch<H>(P, up, reinterpret_cast<const int32_t *>(e + 16), cx);
        pend_i = -1;
    };
    Walk w1 = w.next(cx.G, cx.n_units);
    for (int32_t i = 0; w.g < cx.total; ++i) {
        // the record of the unit after next is requested now and stored when this step is done
        const Walk w2 = w1.next(cx.G, cx.n_units);
        UnitRegs mn;
        if (warp == 3) mn = fetch_unit(P, w2.u, w2.g < cx.total, lane);
        const unsigned char *e = entry_of(i);
        const int4 rec = *reinterpret_cast<const int4 *>(e);
        const Unit un = decode_unit(P, cx, rec, w.item);
        if (un.run) shrink_dispatch<H>(P, un, cx);
        run_pending();
        if (un.run) {
            pend_i = i;
            pend_item = w.item;
        } else if (!P.meta && rec.x == -1) {   // per-token mode: this token has no adapter
            if (cx.crank == 0 && tid == 0 && rec.y && un.item == 0)
                atomicAdd(&P.pool.status[STATUS_INVALID_TOKENS], 1);
            if (!P.item[un.item].in_place)
                copy_rows_item(P.item[un.item], reinterpret_cast<const int32_t *>(e + 16), 1,
                               (int32_t)cx.crank, (int32_t)cx.csize);
        }
        if (warp == 3) store_unit(smem, i + 2, mn, true, lane);
        consumer_sync();   // the new record is visible; nobody reads the overwritten one any more
        w = w1;
        w1 = w2;
    }
    run_pending();
    if (!cx.ok) {
        *dead_flag(smem) = 1;
        if (tid == 0) atomicAdd(&P.pool.status[STATUS_TIMEOUTS], 1);
    }

    // rows that take no adapter: y_base -> y, 16 rows per cluster step (grouped mode, out of place)
    if (P.meta) {
        int32_t *rowidx = reinterpret_cast<int32_t *>(smem + SM_RING + 16);
        const int32_t n_idle = P.T - __ldg(P.meta + H_NACTIVE);
        const int32_t chunks = (n_idle + 15) / 16;
        for (int32_t k = cx.cid; k < chunks * P.n_items; k += cx.G) {
            const int32_t item = k / chunks, first = (k - item * chunks) * 16;
            if (P.item[item].in_place) continue;
            const int32_t rows = min(16, n_idle - first);
            consumer_sync();
            if (tid < rows) rowidx[tid] = __ldg(P.meta + P.moff_perm + (P.T - n_idle) + first + tid);
            consumer_sync();
            copy_rows_item(P.item[item], rowidx, rows, (int32_t)cx.crank, (int32_t)cx.csize);
        }
    }
}

// H: 1 when a unit holds at most 8 rows (decode tiles, single tokens), 2 otherwise.
template <int H>
__global__ void __launch_bounds__(FT_ALL, LORA_FUSED_MIN_BLOCKS)
fused_kernel(const __grid_constant__ FusedParams P) {
    extern __shared__ __align__(1024) unsigned char smem[];
    Ctx cx;
    cx.smem = smem;
    cx.full = reinterpret_cast<uint64_t *>(smem);
    cx.empty = cx.full + MAX_STAGES;
    cx.csize = cluster_nctarank();
    cx.crank = cluster_ctarank();
    cx.cid = (int32_t)(blockIdx.x / cx.csize);
    cx.G = (int32_t)(gridDim.x / cx.csize);
    cx.st = 0;
    cx.ph = 0;
    cx.kp = cx.kr = 0;
    cx.n_units = 1;
    cx.total = 0;
    cx.ok = true;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // The next kernel of the stream may become resident from now on.  It touches nothing this
    // kernel writes before its own griddepcontrol.wait, which returns only when this kernel (and,
    // through this kernel's own wait below, everything before it) is complete.
    griddep_launch_dependents();
    // the swizzled tiles want 1024-byte aligned stages; the carve-up assumes an aligned base (the
    // same in every block, so either all blocks of the launch leave here or none)
    if (smem_u32(smem) & 1023u) {
        if (tid == 0 && blockIdx.x == 0) atomicAdd(&P.pool.status[STATUS_TIMEOUTS], 1);
        griddep_wait();
        return;
    }
    // barriers; the next lines touch no memory another kernel writes
    if (tid == 0) {
        for (int s = 0; s < P.n_stages; ++s) {
            mbar_init(&cx.full[s], 1);
            mbar_init(&cx.empty[s], 4);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(reinterpret_cast<uint64_t *>(smem + SM_XBAR) + b, cx.csize);
            mbar_init(reinterpret_cast<uint64_t *>(smem + SM_YBAR) + b, cx.csize);
        }
        *reinterpret_cast<int32_t *>(smem + SM_DEAD) = 0;
        *reinterpret_cast<int32_t *>(smem + SM_ISSUED) = 0;
        fence_mbar_init();
    }
    // no block signals a peer whose barriers are not set up
    cluster_arrive();
    if (warp == 4 && lane < MAPS_PER_TARGET) prefetch_tensormap(P.maps + P.item[0].map_base + lane);
    // Under programmatic dependent launch this kernel may start while the one before it on the
    // stream is still running.  Activations are only touched after griddep_wait().  The unit
    // records and the pool were complete before that kernel started when P.early is set (the host
    // sets it only then), so they are read, and the first weight tiles requested, ahead of the wait.
    if (!P.early) griddep_wait();
    __syncthreads();
    cluster_wait();
    if (warp == 4) producer_warp(P, cx, lane);
    else consumer_warps<H>(P, cx);
    // A block that gave up may still have copies on their way into its shared memory; they must
    // land before the block leaves.  All five warps meet (the requesting warp has published how
    // many jobs it asked for), then one thread waits, bounded, for what has not been consumed.
    __syncthreads();
    if (*dead_flag(smem) && tid == 0) {
        const int32_t issued = *reinterpret_cast<volatile int32_t *>(smem + SM_ISSUED);
        // the most recent job of every stage: all earlier ones were waited for before a refill
        for (int32_t q = max(issued - P.n_stages, 0); q < issued; ++q)
            mbar_wait(&cx.full[q % P.n_stages], (uint32_t)(q / P.n_stages) & 1u);
    }
    // No block leaves while a peer may still read its partials, write into its buffers or signal
    // its barriers: the closing barrier is the hardware one, which every block reaches whatever
    // happened before.
    cluster_arrive();
    cluster_wait();
}

}  // namespace lora

#include "decode_kernel.cuh"

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
            const int blocks = rows <= 16 ? 4 : rows <= 32 ? 2 : 1;   // chunk width 256 / 128 / 64
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
    else if (H == 1) kern = fused_kernel<1>;
    else kern = fused_kernel<2>;
    const int32_t mrows = H == 2 ? 16 : 8;
    const int32_t RPmax = (pool->bucket_mask & 8u) ? 64 : (pool->bucket_mask & 4u) ? 32 : 16;
    int32_t S = pool->tuning[5];
    if (S < 2 || S > MAX_STAGES) S = 2;   // two stages and more resident blocks beat deeper rings
    int32_t o = SM_HEADER;
    P.off_part = o;   o += mrows * 64 * 4;
    // the partials of all blocks of the cluster fit beside each other when units are small: then
    // they are pushed to every block instead of fetched by every block
    P.push = (8 * mrows * RPmax * 4 <= 4096 && pool->tuning[6] != 1) ? 1 : 0;
    P.vbuf_bytes = (P.push ? 8 : 1) * mrows * RPmax * 4;
    P.off_vpart = o;  o += 2 * P.vbuf_bytes;
    P.off_vh = o;     o += mrows * (RPmax + 8) * 2;
    P.off_vl = o;     o += mrows * (RPmax + 8) * 2;
    o = (o + 1023) & ~1023;
    P.off_w = o;      o += S * W_BYTES;
    P.tok_bytes = mrows * TOK_PITCH * 2;
    P.off_tok = o;    o += S * P.tok_bytes;
    P.n_stages = S;
    const int32_t smem = H == 0 ? dec::smem_bytes(S) : o;
    P.prefetch = pool->tuning[8] == 1 ? 0 : 1;
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
    // Programmatic dependent launch (tuning key 2: 0 = when allowed, 2 = never).  Reading the table
    // and the pool ahead of the preceding kernel's end is allowed for grouped batches whose table
    // has already been read by an earlier apply: that apply was fully ordered behind the build, so
    // the table is complete before this kernel can start.
    const bool fresh = meta_key ? pool->take_fresh(meta_key) : true;
    P.early = (meta_key && !fresh && pool->tuning[2] != 2) ? 1 : 0;
    // Without `early` the attribute still lets the blocks become resident and set up their shared
    // memory while the kernel before them drains; they read nothing until it has completed.
    const unsigned n_attrs = pool->tuning[2] != 2 ? 2 : 1;

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
        C = 8;
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
