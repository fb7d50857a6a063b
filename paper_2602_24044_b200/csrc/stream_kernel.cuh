// The general form of the fused LoRA forward (paper Section 2.2), included by apply_fused.cu: every
// rank up to 64, units of up to 16 token rows, widths that are not whole 64-column blocks, batches
// indexed per token.  (Decode batches of small ranks take decode_kernel, the same design with
// everything fixed at compile time.)
//
// A unit is at most 16 token rows of one adapter in one projection.  A thread-block cluster owns
// one unit at a time; block c of the cluster takes the c-th slice of d_in for the shrink phase and
// the c-th slice of d_out for the expand phase.  The requesting warp walks the cluster's units and
// places jobs in a ring of shared-memory stages, software-pipelined by one unit:
//     shrink(u0) shrink(u1) expand(u0) shrink(u2) expand(u1) ... end
// A job is one column chunk: the rank rows of A_i (or B_i) by ONE tiled bulk copy (TMA, 128-byte
// swizzle), the unit's rows of x (or y_base) by one bulk copy per row, and a 16-byte header (kind,
// first / last chunk of its unit, columns, unit entry).  The four consumer warps hold no control
// logic: they follow the headers.  A chunk is 256 columns wide up to rank 32 and 128 above, so a
// weight tile is at most 16 KB and a stage has one size for every rank.
//   shrink   bf16 MMA (m16n8k16), fp32 accumulators carried across a unit's chunks in registers;
//   exchange every block keeps its partial in its own shared memory and tells the cluster; every
//            block then reads all partials (distributed shared memory) and sums them in block order;
//            two sets of buffers and barriers alternate between consecutive units;
//   expand   v as the sum of two bf16 numbers (high and low part); scale and residual add fused,
//            one rounding to bf16 at the store.
// A block without columns in a phase still gets a header-only job, so that it takes part in the
// exchange.  Every wait is bounded; a wait that runs out marks the block dead: it stops, drains
// its own copies and goes to the closing cluster barrier.
#pragma once

namespace lora {
namespace gen {

constexpr int SM_FULL = 0;       // mbarriers: a job's data has landed              [MAX_STAGES]
constexpr int SM_EMPTY = 32;     // mbarriers: the consumer warps have left a stage  [MAX_STAGES]
constexpr int SM_XB = 64;        // two mbarriers: every block has published its partial
constexpr int SM_YB = 80;        // two mbarriers: every block has read the partials
constexpr int SM_FLAG = 96;      // int32: a bounded wait of this block has expired
constexpr int SM_COUNT = 100;    // int32: jobs requested so far
constexpr int SM_CBAR = 104;     // mbarrier: the consumer threads meet (bounded, unlike bar.sync)
constexpr int SM_JOB = 128;      // job headers, 16 bytes per stage
constexpr int SM_UNIT = 192;     // unit entries, ring of eight
constexpr int UNIT_ENTRIES = 8;
constexpr int UNIT_BYTES = 96;
constexpr int PV = 72;           // elements between rows of the bf16 copies of v
static_assert(SM_UNIT + UNIT_ENTRIES * UNIT_BYTES <= SM_HEADER, "fixed part fits before the carved-up buffers");

// columns of a job for rank bucket 16 << sh: the weight tile is at most 16 KB
__host__ __device__ constexpr int chunk_cols(int sh) { return sh == 2 ? 128 : 256; }

enum { J_SHRINK = 1, J_FIRST = 2, J_LAST = 4, J_END = 8 /* no data, stream over */,
       J_FINAL = 16 /* last job of the stream */, J_COPY = 32 /* y_base -> y for one row */ };

struct UnitEntry {          // 96 bytes
    int32_t rows, rb, rank, item;
    float scale;
    int32_t b_lo;           // first column of this block's slice of d_out
    int32_t sh;             // rank bucket: 16 << sh
    int32_t pad;
    int32_t rowid[16];
};

// ---------------------------------------------------------------------------------------------
// the requesting warp
// ---------------------------------------------------------------------------------------------
struct PUnit {              // what the requesting warp keeps of a unit
    int32_t slot, rows, rb, rank, item, sh;
    int32_t na, nb, a_lo, a_hi, b_lo, b_hi;
    float scale;
    bool run;
    bool copy;              // per-token mode: a token without adapter whose row has to be copied
};

// record: {slot (-1: token without adapter, -2: past the end), position, rows | tile rows << 8 |
// consecutive ids << 16 | rank << 17, scale bits}
__device__ __forceinline__ PUnit p_decode(const FusedParams &P, uint32_t crank, const int4 rec, int32_t item) {
    PUnit u;
    u.slot = rec.x;
    u.rows = rec.z & 0xff;
    const int32_t tile_rows = (rec.z >> 8) & 0xff, contiguous = (rec.z >> 16) & 1;
    u.rank = (rec.z >> 17) & 0x7f;
    u.rb = (u.rank + 7) & ~7;
    u.scale = __int_as_float(rec.w);
    u.item = min(item, P.n_items - 1);
    const FusedItem &it = P.item[u.item];
    u.a_lo = min((int32_t)crank * it.wa, it.d_in);
    u.a_hi = min(u.a_lo + it.wa, it.d_in);
    u.b_lo = min((int32_t)crank * it.wb, it.d_out);
    u.b_hi = min(u.b_lo + it.wb, it.d_out);
    // runs of consecutive tokens belong to the tensor-core kernels when those ran
    u.run = rec.x >= 0 && u.rows > 0 && u.rank > 0 &&
            !(P.path_filter && contiguous && tile_rows >= P.path_filter);
    u.copy = !P.meta && rec.x == -1 && !it.in_place;
    u.sh = u.rank <= 16 ? 0 : u.rank <= 32 ? 1 : 2;
    const int32_t cw = chunk_cols(u.sh);
    // at least one job per phase: a block without columns still takes part in the exchange
    u.na = max(1, (u.a_hi - u.a_lo + cw - 1) / cw);
    u.nb = max(1, (u.b_hi - u.b_lo + cw - 1) / cw);
    return u;
}

// The record of unit u of the batch, on its way to the requesting warp's registers (lane 16: the
// record, lanes 0-15: the unit's token ids).
__device__ __forceinline__ void p_fetch(const FusedParams &P, int32_t u, bool valid, int lane, int4 &rec,
                                        int32_t &rowid) {
    rec = make_int4(-2, 0, 0, 0);
    rowid = 0;
    if (!valid) return;
    if (P.meta) {
        if (lane == 16) rec = ldg_int4(P.meta + P.moff_udesc + 4 * (int64_t)u);
        else if (lane < 16) rowid = ldg_int(P.meta + P.moff_uperm + 16 * (int64_t)u + lane);
    } else {
        rowid = u;
        if (lane == 16) {
            const int32_t s = ldg_int(P.slot_idx + u);
            rec = make_int4(-1, s != -1 ? 1 : 0, 0, 0);   // y = 1: not an adapter-less token either
            if (s >= 0 && s < P.pool.num_slots) {
                const SlotEntry e = P.pool.table[s];
                if (e.loaded)
                    rec = make_int4(s, u, 1 | (1 << 8) | (1 << 16) | (e.rank << 17), __float_as_int(e.scale));
            }
        }
    }
}

// One job into stage st: header, weight tile, token rows.  mode 0: all; 1: header and tile (with the
// byte count of the whole job); 2: the token rows of a job started in mode 1.
__device__ __forceinline__ void p_request(const FusedParams &P, unsigned char *smem, const PUnit &un,
                                          int32_t j, int32_t entry, int st, int32_t rowid, int lane, int mode,
                                          bool final_job) {
    const FusedItem &it = P.item[un.item];
    uint64_t *full = reinterpret_cast<uint64_t *>(smem + SM_FULL) + st;
    const bool shrink = j < un.na;
    const int32_t c = shrink ? j : j - un.na;
    const int32_t cw = chunk_cols(un.sh);
    const int32_t col0 = (shrink ? un.a_lo : un.b_lo) + c * cw;   // a multiple of 64
    const int32_t ncols = max(0, min(cw, (shrink ? un.a_hi : un.b_hi) - col0));
    if (lane == 0 && mode != 2) {
        const int32_t last = shrink ? un.na - 1 : un.nb - 1;
        *reinterpret_cast<int4 *>(smem + SM_JOB + 16 * st) =
            make_int4((shrink ? J_SHRINK : 0) | (c == 0 ? J_FIRST : 0) | (c == last ? J_LAST : 0) |
                          (final_job ? J_FINAL : 0), entry, c, ncols);
        if (ncols > 0) {
            const CUtensorMap *map = P.maps + it.map_base + (shrink ? 0 : 8) + (un.rb >> 3) - 1;
            // the tile load always delivers its whole box: rb rows of cw columns
            mbar_expect_tx(full, (uint32_t)un.rb * (uint32_t)cw * 2u + (uint32_t)un.rows * (uint32_t)ncols * 2u);
            tma_load_4d(smem + P.off_w + st * P.w_bytes, map, 0, 0, col0 >> 6, un.slot, full);
        } else {
            mbar_arrive(full);   // header only
        }
    }
    __syncwarp();
    if (lane < un.rows && mode != 1 && ncols > 0) {
        const __nv_bfloat16 *tok = (shrink ? it.x : it.yb) + col0 + (int64_t)rowid * (shrink ? it.ldx : it.ldyb);
        bulk_g2s(smem + P.off_tok + st * P.tok_bytes + lane * (TOK_PITCH * 2), tok, (uint32_t)ncols * 2u, full);
    }
}

// Walks the cluster's units (it reads the records itself, one unit ahead) and keeps the ring full:
// a job is requested as soon as the four consumer warps have left its stage.
__device__ __forceinline__ void producer(const FusedParams &P, unsigned char *smem, int32_t cid, int32_t G,
                                         uint32_t crank, int lane) {
    const int32_t S = P.n_stages;
    volatile int32_t *dead = reinterpret_cast<volatile int32_t *>(smem + SM_FLAG);
    volatile int32_t *count = reinterpret_cast<volatile int32_t *>(smem + SM_COUNT);
    uint64_t *empty = reinterpret_cast<uint64_t *>(smem + SM_EMPTY);
    uint64_t *full = reinterpret_cast<uint64_t *>(smem + SM_FULL);
    auto bcast = [&](int4 r) {
        r.x = __shfl_sync(0xffffffffu, r.x, 16);
        r.y = __shfl_sync(0xffffffffu, r.y, 16);
        r.z = __shfl_sync(0xffffffffu, r.z, 16);
        r.w = __shfl_sync(0xffffffffu, r.w, 16);
        return r;
    };
    // the unit count and (speculatively, as if the table were full) the first record, side by side
    int32_t n_units = P.meta ? ldg_int(P.meta + H_NPIECE) : P.T;
    int4 rec;
    int32_t rowid;
    p_fetch(P, cid, P.n_items == 1 && cid < P.units_cap, lane, rec, rowid);
    if (n_units > P.units_cap) n_units = P.units_cap;
    const int32_t total = n_units * P.n_items;
    if (n_units < 1) n_units = 1;
    // position in the launch's unit list: unit g is unit u of projection `item`
    int32_t g = cid, u = cid, item = 0;
    while (u >= n_units) { u -= n_units; ++item; }
    if (P.n_items > 1) p_fetch(P, u, g < total, lane, rec, rowid);

    int32_t q = 0, skip = 0, st = 0;
    uint32_t ph = 0;
    bool ok = true, have_pend = false, waited = !P.early, sent_final = false;
    PUnit pend;
    int32_t pend_rowid = 0, pend_entry = 0, n_run = 0;
    // waits until stage st may be refilled; false once a wait has run out
    auto stage_free = [&]() {
        if (q >= S && ok) {
            ok = mbar_wait(&empty[st], (ph - 1u) & 1u);
            if (!ok) *dead = 1;
        }
        return ok && !*dead;
    };
    auto advance = [&]() {
        ++q;
        if (++st == S) { st = 0; ++ph; }
    };
    for (int32_t i = 0;; ++i) {
        const bool real = g < total;
        if (!real && !have_pend) break;
        int32_t gn = g + G, un_ = u + G, itn = item;
        while (un_ >= n_units) { un_ -= n_units; ++itn; }
        const bool next_real = real && gn < total;
        int4 rec_n;
        int32_t rowid_n;
        p_fetch(P, un_, next_real, lane, rec_n, rowid_n);   // the next unit's record, meanwhile
        const int4 rb = bcast(rec);
        PUnit un = p_decode(P, crank, rb, item);
        if (!real) un.run = un.copy = false;   // past the end: only the last unit's expand jobs are left
        // per-token mode: a slot id that is neither -1 nor an occupied slot is counted once
        if (real && !P.meta && rb.x == -1 && rb.y && crank == 0 && un.item == 0 && lane == 0)
            atomicAdd(&P.pool.status[STATUS_INVALID_TOKENS], 1);
        // Entries are numbered by the units that run, not by the units walked: a cluster that
        // skips units between two that run must not come back to an entry still in use (the
        // entry of a unit is read until its last expand chunk, which follows the next running
        // unit's shrink chunks in the ring).
        const int32_t entry = n_run & (UNIT_ENTRIES - 1);
        if (un.run) ++n_run;
        if (un.run) {
            // the unit's entry; made visible to the consumers by the arrival on the barrier of
            // the unit's first job
            UnitEntry *e = reinterpret_cast<UnitEntry *>(smem + SM_UNIT + entry * UNIT_BYTES);
            if (lane == 16) {
                e->rows = un.rows; e->rb = un.rb; e->rank = un.rank; e->item = un.item;
                e->scale = un.scale; e->b_lo = un.b_lo; e->sh = un.sh;
            } else if (lane < 16) {
                e->rowid[lane] = rowid;
            }
            __syncwarp();
        }
        if (i == 0 && P.early) {
            // The kernel before this one may still be running: the pool may be read (the host
            // vouches for it), the activations not yet.  Weight tiles of the first jobs now, their
            // token rows after the wait.
            skip = !un.run ? 0 : un.na < S ? un.na : S;
            for (int32_t j = 0; j < skip; ++j) p_request(P, smem, un, j, entry, j, rowid, lane, 1, false);
        }
        if (!waited) {
            griddep_wait();
            waited = true;
            for (int32_t j = 0; j < skip; ++j) {
                p_request(P, smem, un, j, entry, j, rowid, lane, 2, false);
                advance();
            }
            if (lane == 0) *count = skip;
        }
        // this step's jobs in ring order: the unit's shrink chunks, then the pending unit's expand chunks
        const int32_t ja = un.run ? un.na : 0, jb = have_pend ? pend.nb : 0;
        for (int32_t k = (i == 0 ? skip : 0); k < ja + jb; ++k) {
            if (stage_free()) {
                if (k < ja) p_request(P, smem, un, k, entry, st, rowid, lane, 0, false);
                else p_request(P, smem, pend, pend.na + k - ja, pend_entry, st, pend_rowid, lane, 0,
                               !real && k == ja + jb - 1);   // nothing follows the last unit's last expand chunk
                if (lane == 0) *count = q + 1;
            }
            advance();
        }
        if (!real && jb > 0) sent_final = true;
        if (un.copy) {   // a row to copy: header only
            if (stage_free() && lane == 0) {
                *reinterpret_cast<int4 *>(smem + SM_JOB + 16 * st) = make_int4(J_COPY, un.item, rowid, 0);
                mbar_arrive(&full[st]);
            }
            advance();
        }
        have_pend = un.run;
        pend = un;
        pend_rowid = rowid;
        pend_entry = entry;
        if (!real) break;
        rec = rec_n;
        rowid = rowid_n;
        g = gn; u = un_; item = itn;
    }
    if (!waited) griddep_wait();
    // A stream whose last job is not an expand chunk is closed by a job without data.
    if (!sent_final) {
        if (stage_free() && lane == 0) {
            *reinterpret_cast<int4 *>(smem + SM_JOB + 16 * st) = make_int4(J_END, 0, 0, 0);
            mbar_arrive(&full[st]);
        }
    }
    if (!ok && lane == 0) atomicAdd(&P.pool.status[STATUS_TIMEOUTS], 1);
}

// ---------------------------------------------------------------------------------------------
// the consumer warps: job bodies
// ---------------------------------------------------------------------------------------------
// Per-thread constants of the consumer warps.
struct CLane {
    int tid, lane, warp, g, t, mi, r;
};

// One shrink chunk: acc += x[rows, chunk] . A_i[chunk, 16 ranks of this warp].  RP: rank bucket; H: 1
// when a unit holds at most 8 rows, 2 when rows 8..15 can be occupied.  The NWC consumer warps split the
// rank tiles WN ways and the chunk's 64-column blocks WK ways: every warp owns two rank tiles of 8
// and every WK-th column block.  Operand fragments come by ldmatrix; lane l names row (l & 7) of 8x8 matrix
// (l >> 3):
//   weights: (tile 2wn, k 0-7) (tile 2wn, k 8-15) (tile 2wn+1, k 0-7) (tile 2wn+1, k 8-15); rank row
//            n sits at n * 128 bytes of the column block, its 16-byte chunk c at ((c ^ (n & 7)) << 4);
//            the even part of c is folded in per step with one XOR
//   tokens:  (rows 0-7, k 0-7) (rows 8-15, k 0-7) (rows 0-7, k 8-15) (rows 8-15, k 8-15)
template <int RP, int H, int NWC>
__device__ __forceinline__ void shrink_job(const CLane &L, uint32_t w_stage, uint32_t t_stage, int32_t ncols,
                                           uint32_t blk_bytes, float (&acc)[2][4]) {
    constexpr int WN = RP / 16, WK = NWC / WN;   // a warp whose column block the job does not have stays idle
    constexpr int NB = chunk_cols(RP == 16 ? 0 : RP == 32 ? 1 : 2) / 64;   // column blocks of a job
    constexpr bool hi_rows = H == 2;
    const int wk = L.warp % WK, wn = L.warp / WK;
    const uint32_t w_lane = (uint32_t)(16 * wn + 8 * (L.mi >> 1) + L.r) * 128u + (uint32_t)(((L.mi & 1) ^ L.r) << 4);
    const uint32_t x_lane = hi_rows ? (uint32_t)(((L.mi & 1) * 8 + L.r) * TOK_PITCH + (L.mi >> 1) * 8) * 2u
                                    : (uint32_t)(L.r * TOK_PITCH + (L.mi & 1) * 8) * 2u;
#pragma unroll
    for (int cb = wk; cb < NB; cb += WK) {   // this warp's column blocks of the job
        const int32_t nc = ncols - cb * 64;
        if (nc <= 0) break;
        const uint32_t As = w_stage + (uint32_t)cb * blk_bytes + w_lane;
        const uint32_t X = t_stage + (uint32_t)cb * 128u + x_lane;
#pragma unroll
        for (int ks = 0; ks < 64; ks += 16) {
            if (ks < nc) {   // the ragged end of a slice: columns past it hold neither x nor these weights
                const bool full = nc - ks >= 16;   // else only 8 columns are left
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
}

// What a thread keeps of the unit whose expand chunks are running.
struct XUnit {
    __nv_bfloat16 *y0, *y1;   // this lane's output rows g and g + 8 at this warp's first column
    float scale;
    uint32_t blk_bytes;
    int32_t rank16, rb;
    bool row0, row1;
};

// One expand chunk: y[rows, chunk] = y_base + s * v . B_i[ranks, chunk] for this warp's columns.
// B_i fragments by ldmatrix (transposing): lane l names rank row ks + 8 (mi & 1) + r of column tile
// 2 np + (mi >> 1); v fragments (high and low bf16 parts) by ldmatrix from the block's copies.
template <int RP, int H, int NWC>
__device__ __forceinline__ void expand_job(const CLane &L, uint32_t w_stage, uint32_t t_stage, uint32_t vh,
                                           uint32_t vl, int32_t ncols, int32_t c, const XUnit &xu) {
    constexpr int CW = chunk_cols(RP == 16 ? 0 : RP == 32 ? 1 : 2), NW = CW / NWC, NP = NW / 16, KT = RP / 16;
    constexpr bool hi_rows = H == 2;
    const int32_t nc = ncols - L.warp * NW;   // columns of this warp's share
    if (nc <= 0) return;
    const uint32_t b_lane = (uint32_t)((L.mi & 1) * 8 + L.r) * 128u + (uint32_t)(((L.mi >> 1) ^ L.r) << 4);
    const uint32_t v_lane = hi_rows ? (uint32_t)(((L.mi & 1) * 8 + L.r) * PV + (L.mi >> 1) * 8) * 2u
                                    : (uint32_t)(L.r * PV + (L.mi & 1) * 8) * 2u;
    const uint32_t Ys = t_stage + (uint32_t)(L.g * TOK_PITCH + L.warp * NW + 2 * L.t) * 2u;
    __nv_bfloat16 *y0 = xu.y0 + c * CW, *y1 = xu.y1 + c * CW;
#pragma unroll
    for (int np = 0; np < NP; ++np) {
        if (16 * np >= nc) break;
        const uint32_t tabs = (uint32_t)(L.warp * (NW / 8) + 2 * np);   // first tile of the pair in the chunk
        const uint32_t Bs = w_stage + (tabs >> 3) * xu.blk_bytes + b_lane;
        const uint32_t cx4 = (tabs & 7u) << 4;
        float ex[2][4];
#pragma unroll
        for (int j = 0; j < 2; ++j) ex[j][0] = ex[j][1] = ex[j][2] = ex[j][3] = 0.0f;
#pragma unroll
        for (int kt = 0; kt < KT; ++kt) {
            const int ks = kt * 16;
            if (KT > 1 && ks >= xu.rank16) break;
            uint32_t fh[4], fl[4], bb[4];
            if (hi_rows) {
                ldmatrix_x4(fh, vh + v_lane + ks * 2);
                ldmatrix_x4(fl, vl + v_lane + ks * 2);
            } else {
                ldmatrix_x2(fh[0], fh[2], vh + v_lane + ks * 2);
                ldmatrix_x2(fl[0], fl[2], vl + v_lane + ks * 2);
                fh[1] = fh[3] = fl[1] = fl[3] = 0u;
            }
            ldmatrix_x4_trans(bb, (Bs + (uint32_t)ks * 128u) ^ cx4);
            // Rank rows ks+8 .. ks+15 were only copied when the tile has them; what the stage holds
            // there otherwise belongs to an earlier job (possibly another adapter's weights) and
            // must not meet the MMA, not even multiplied by zero.
            if (ks + 8 >= xu.rb) bb[1] = bb[3] = 0u;
            mma16816(ex[0], fh, bb[0], bb[1]);
            mma16816(ex[0], fl, bb[0], bb[1]);
            mma16816(ex[1], fh, bb[2], bb[3]);
            mma16816(ex[1], fl, bb[2], bb[3]);
        }
        // epilogue straight from the accumulator layout: each lane owns two adjacent columns of a row
        // per column tile; a quad covers 16 contiguous bytes
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const int coff = (2 * np + j) * 8;
            if (coff < nc) {
                if (xu.row0) {
                    uint32_t w;
                    asm volatile("ld.shared.b32 %0, [%1];" : "=r"(w) : "r"(Ys + coff * 2));
                    *reinterpret_cast<uint32_t *>(y0 + coff) =
                        pack2(fmaf(xu.scale, ex[j][0], __uint_as_float(w << 16)),
                              fmaf(xu.scale, ex[j][1], __uint_as_float(w & 0xffff0000u)));
                }
                if (hi_rows && xu.row1) {
                    uint32_t w;
                    asm volatile("ld.shared.b32 %0, [%1];" : "=r"(w) : "r"(Ys + (8 * TOK_PITCH + coff) * 2));
                    *reinterpret_cast<uint32_t *>(y1 + coff) =
                        pack2(fmaf(xu.scale, ex[j][2], __uint_as_float(w << 16)),
                              fmaf(xu.scale, ex[j][3], __uint_as_float(w & 0xffff0000u)));
                }
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------
// the consumer warps: follow the job stream
// ---------------------------------------------------------------------------------------------
template <int H>
__device__ __forceinline__ void consumers(const FusedParams &P, unsigned char *smem, int32_t cid, int32_t G,
                                          uint32_t crank, uint32_t csize) {
    constexpr int mrows = 8 * H;
    constexpr int NWC = 4 * H, CT = 32 * NWC, LOG_NWC = H == 2 ? 3 : 2;   // consumer warps, threads
    CLane L;
    L.tid = threadIdx.x; L.lane = L.tid & 31; L.warp = L.tid >> 5; L.g = L.lane >> 2; L.t = L.lane & 3;
    L.mi = L.lane >> 3; L.r = L.lane & 7;
    const int tid = L.tid, lane = L.lane;
    uint64_t *full = reinterpret_cast<uint64_t *>(smem + SM_FULL);
    uint64_t *empty = reinterpret_cast<uint64_t *>(smem + SM_EMPTY);
    volatile int32_t *dead = reinterpret_cast<volatile int32_t *>(smem + SM_FLAG);
    float *part = reinterpret_cast<float *>(smem + P.off_part);     // [WK][mrows][RP] = mrows x 16 NWC floats
    __nv_bfloat16 *Vh = reinterpret_cast<__nv_bfloat16 *>(smem + P.off_vh);   // [mrows][PV]
    __nv_bfloat16 *Vl = reinterpret_cast<__nv_bfloat16 *>(smem + P.off_vl);
    const uint32_t w_base = smem_u32(smem + P.off_w), t_base = smem_u32(smem + P.off_tok);
    const uint32_t vh_addr = smem_u32(Vh), vl_addr = smem_u32(Vl);

    float acc[2][4];
#pragma unroll
    for (int i = 0; i < 2; ++i) acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0.0f;
    XUnit xu;
    xu.y0 = xu.y1 = nullptr; xu.scale = 0.0f; xu.blk_bytes = 0; xu.rank16 = 16; xu.rb = 16; xu.row0 = xu.row1 = false;
    int32_t st = 0, kp = 0, kr = 0;
    uint32_t ph = 0, cs = 0;
    bool ok = true, met_cluster = false;
    // rows without adapter are copied at the end (grouped mode, out-of-place projections)
    const int32_t n_active = (P.meta && P.copy_idle) ? ldg_int(P.meta + H_NACTIVE) : P.T;
    // The consumer threads meet on an mbarrier, not on bar.sync: a thread that has given up a wait
    // never arrives, and the others must not wait for it without a limit.
    auto meet = [&]() {
        uint64_t *cb = reinterpret_cast<uint64_t *>(smem + SM_CBAR);
        mbar_arrive(cb);
        const bool done = __all_sync(0xffffffffu, mbar_wait(cb, cs & 1u));
        ++cs;
        if (!done) *dead = 1;
        return done && !*dead;
    };
    if (P.early) griddep_wait();

    for (;;) {
        ok = __all_sync(0xffffffffu, mbar_wait(&full[st], ph & 1u));   // a warp stays together
        if (!ok) {
            *dead = 1;
            break;
        }
        const int4 job = *reinterpret_cast<const int4 *>(smem + SM_JOB + 16 * st);
        if (job.x & J_END) break;
        const uint32_t w_stage = w_base + st * P.w_bytes, t_stage = t_base + st * P.tok_bytes;
        if (job.x & J_COPY) {
            // per-token mode: row job.z of projection job.y takes no adapter
            const FusedItem &it = P.item[job.y];
            const __nv_bfloat16 *src = it.yb + (int64_t)job.z * it.ldyb;
            __nv_bfloat16 *dst = it.y + (int64_t)job.z * it.ldy;
            for (int32_t v = (int32_t)crank * CT + tid; v < it.d_out / 8; v += (int32_t)csize * CT)
                reinterpret_cast<uint4 *>(dst)[v] = ldg16(src + (int64_t)v * 8);
            __syncwarp();
            if (lane == 0) mbar_arrive(&empty[st]);
        } else if (job.x & J_SHRINK) {
            const UnitEntry *ue = reinterpret_cast<const UnitEntry *>(smem + SM_UNIT + job.y * UNIT_BYTES);
            const int32_t sh = ue->sh, rows = ue->rows;
            const uint32_t blk_bytes = (uint32_t)ue->rb * 128u;
            if (job.x & J_FIRST) {
#pragma unroll
                for (int i = 0; i < 2; ++i) acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0.0f;
            }
            if (sh == 0) shrink_job<16, H, NWC>(L, w_stage, t_stage, job.w, blk_bytes, acc);
            else if (sh == 1) shrink_job<32, H, NWC>(L, w_stage, t_stage, job.w, blk_bytes, acc);
            else shrink_job<64, H, NWC>(L, w_stage, t_stage, job.w, blk_bytes, acc);
            __syncwarp();
            if (lane == 0) mbar_arrive(&empty[st]);
            if (job.x & J_LAST) {
                // ---- the block's partial is made available to the cluster (buffer set kp & 1) ----
                const int b = kp & 1;
                const int RP = 16 << sh, WK = NWC >> sh;
                if (kp >= 2) {   // the peers have read what this set held two units ago
                    ok = __all_sync(0xffffffffu, mbar_wait_cluster(reinterpret_cast<uint64_t *>(smem + SM_YB) + b,
                                                                   (uint32_t)((kp - 2) >> 1) & 1u));
                    if (!ok) {
                        *dead = 1;
                        break;
                    }
                }
                const int wk = L.warp & (WK - 1), wn = L.warp >> (LOG_NWC - sh);
#pragma unroll
                for (int i = 0; i < 2; ++i) {
                    float *p0 = part + (wk * mrows + L.g) * RP + (wn * 2 + i) * 8 + 2 * L.t;
                    *reinterpret_cast<float2 *>(p0) = make_float2(acc[i][0], acc[i][1]);
                    if (H == 2) *reinterpret_cast<float2 *>(p0 + 8 * RP) = make_float2(acc[i][2], acc[i][3]);
                }
                if (!meet()) { ok = false; break; }
                // block partial: the column blocks' sums in order
                float *vbuf = reinterpret_cast<float *>(smem + P.off_vpart + b * P.vbuf_bytes);
                for (int i = tid; i < mrows * RP; i += CT) {
                    if ((i >> (4 + sh)) < rows) {
                        float v = part[i];
                        for (int w = 1; w < WK; ++w) v += part[w * mrows * RP + i];
                        vbuf[i] = v;
                    }
                }
                if (!met_cluster) {   // no block is signalled before its barriers are set up
                    cluster_wait();
                    met_cluster = true;
                }
                // one arrival per block and peer: thread q tells block q, after the block's threads
                // have met (its release then covers all their writes)
                if (!meet()) { ok = false; break; }
                if (tid < (int)csize) mbar_arrive_peer(reinterpret_cast<uint64_t *>(smem + SM_XB) + b, (uint32_t)tid);
                ++kp;
            }
        } else {
            const UnitEntry *ue = reinterpret_cast<const UnitEntry *>(smem + SM_UNIT + job.y * UNIT_BYTES);
            const int32_t sh = ue->sh;
            if (job.x & J_FIRST) {
                // ---- every block sums the cluster's partials in block order (buffer set kr & 1) ----
                const int b = kr & 1;
                const int RP = 16 << sh;
                ok = __all_sync(0xffffffffu, mbar_wait_cluster(reinterpret_cast<uint64_t *>(smem + SM_XB) + b,
                                                               (uint32_t)(kr >> 1) & 1u));
                if (!ok) {
                    *dead = 1;
                    break;
                }
                const int32_t rows = ue->rows, rank = ue->rank;
                const int32_t rank16 = (rank + 15) & ~15;
                // the previous unit's expand chunks have read their last fragment of v
                if (!meet()) { ok = false; break; }
                const uint32_t vp_addr = smem_u32(smem + P.off_vpart + b * P.vbuf_bytes);
                for (int i = tid; i < rows * rank16; i += CT) {
                    const int m = i / rank16, k = i - m * rank16;
                    float v = 0.0f;
                    if (k < rank) {
                        // all remote loads are issued before the first add; the sum is in block order
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
                if (!meet()) { ok = false; break; }
                // done reading the partials; the matching wait comes before the set is written again
                if (tid < (int)csize) mbar_arrive_peer(reinterpret_cast<uint64_t *>(smem + SM_YB) + b, (uint32_t)tid);
                ++kr;
                const FusedItem &it = P.item[ue->item];
                const int NW = chunk_cols(sh) / NWC;
                xu.row0 = L.g < rows;
                xu.row1 = H == 2 && L.g + 8 < rows;
                xu.y0 = it.y + (int64_t)(xu.row0 ? ue->rowid[L.g] : 0) * it.ldy + ue->b_lo + L.warp * NW + 2 * L.t;
                xu.y1 = it.y + (int64_t)(xu.row1 ? ue->rowid[L.g + 8] : 0) * it.ldy + ue->b_lo + L.warp * NW + 2 * L.t;
                xu.scale = ue->scale;
                xu.rb = ue->rb;
                xu.blk_bytes = (uint32_t)ue->rb * 128u;
                xu.rank16 = rank16;
            }
            if (sh == 0) expand_job<16, H, NWC>(L, w_stage, t_stage, vh_addr, vl_addr, job.w, job.z, xu);
            else if (sh == 1) expand_job<32, H, NWC>(L, w_stage, t_stage, vh_addr, vl_addr, job.w, job.z, xu);
            else expand_job<64, H, NWC>(L, w_stage, t_stage, vh_addr, vl_addr, job.w, job.z, xu);
            __syncwarp();
            if (lane == 0) mbar_arrive(&empty[st]);
            if (job.x & J_FINAL) break;
        }
        if (++st == P.n_stages) {
            st = 0;
            ++ph;
        }
    }
    if (!ok && tid == 0) atomicAdd(&P.pool.status[STATUS_TIMEOUTS], 1);
    // this block's last remote access is behind it: the closing cluster barrier is arrived at now
    // and waited for at the very end of the kernel
    if (!met_cluster) cluster_wait();
    cluster_arrive();

    // rows that take no adapter: y_base -> y, 16 rows per cluster step (grouped mode, out of place)
    if (ok && !*dead && n_active < P.T) {
        int32_t *rowidx = reinterpret_cast<int32_t *>(smem + P.off_part);
        const int32_t n_idle = P.T - n_active;
        const int32_t chunks = (n_idle + 15) / 16;
        for (int32_t k = cid; k < chunks * P.n_items; k += G) {
            const int32_t item = k / chunks, first = (k - item * chunks) * 16;
            const FusedItem &it = P.item[item];
            if (it.in_place) continue;
            const int32_t rows = min(16, n_idle - first);
            if (!meet()) break;
            if (tid < rows) rowidx[tid] = __ldg(P.meta + P.moff_perm + n_active + first + tid);
            if (!meet()) break;
            // the chunk's rows as one index space (row, 16-byte vector of this block's share), four
            // independent loads in flight per thread
            const int32_t vecs = it.d_out / 8;
            const int32_t per_blk = (vecs + (int32_t)csize - 1) / (int32_t)csize;
            const int32_t v_lo = (int32_t)crank * per_blk, v_n = max(0, min(per_blk, vecs - v_lo));
            const int32_t total = rows * v_n;
            for (int32_t i0 = tid; i0 < total; i0 += 4 * CT) {
                uint4 val[4];
                int64_t off[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const int32_t i = i0 + q * CT;
                    const int32_t m = i < total ? i / v_n : 0, v = i < total ? v_lo + i - m * v_n : 0;
                    off[q] = (int64_t)rowidx[m];
                    val[q] = make_uint4(0, 0, 0, 0);
                    if (i < total) val[q] = ldg16(it.yb + off[q] * it.ldyb + (int64_t)v * 8);
                    off[q] = off[q] * it.ldy + (int64_t)v * 8;
                }
#pragma unroll
                for (int q = 0; q < 4; ++q)
                    if (i0 + q * CT < total) *reinterpret_cast<uint4 *>(it.y + off[q]) = val[q];
            }
        }
    }
}

}  // namespace gen

// H: 1 when a unit holds at most 8 rows (decode tiles, single tokens), 2 otherwise.
// Four consumer warps at H = 1, eight at H = 2 (a 16-row job is twice the work, and the batches that
// come here keep few blocks per SM: the launch is bound by the consumer warps' own chains), plus
// the requesting warp.
template <int H>
__global__ void __launch_bounds__(32 * (4 * H + 1), H == 2 ? 3 : LORA_FUSED_MIN_BLOCKS)
stream_kernel(const __grid_constant__ FusedParams P) {
    extern __shared__ __align__(1024) unsigned char smem[];
    const uint32_t csize = cluster_nctarank(), crank = cluster_ctarank();
    const int32_t cid = (int32_t)(blockIdx.x / csize), G = (int32_t)(gridDim.x / csize);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // The next kernel of the stream may become resident from now on.  It touches nothing this
    // kernel writes before its own griddepcontrol.wait, which returns only when this kernel (and,
    // through this kernel's own wait below, everything before it) is complete.
    if (!P.late_trigger) griddep_launch_dependents();
    // the swizzled tiles want 1024-byte aligned stages (the base is the same in every block, so
    // either all blocks of the launch leave here or none)
    if (smem_u32(smem) & 1023u) {
        if (tid == 0 && blockIdx.x == 0) atomicAdd(&P.pool.status[STATUS_TIMEOUTS], 1);
        griddep_wait();
        return;
    }
    constexpr int NWC = 4 * H;   // consumer warps; warp NWC requests the jobs
    if (warp == NWC && lane < MAPS_PER_TARGET) prefetch_tensormap(P.maps + P.item[0].map_base + lane);
    if (tid == 0) {
        uint64_t *full = reinterpret_cast<uint64_t *>(smem + gen::SM_FULL);
        uint64_t *empty = reinterpret_cast<uint64_t *>(smem + gen::SM_EMPTY);
        for (int s = 0; s < P.n_stages; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], NWC);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(reinterpret_cast<uint64_t *>(smem + gen::SM_XB) + b, csize);
            mbar_init(reinterpret_cast<uint64_t *>(smem + gen::SM_YB) + b, csize);
        }
        mbar_init(reinterpret_cast<uint64_t *>(smem + gen::SM_CBAR), 32 * NWC);
        *reinterpret_cast<int32_t *>(smem + gen::SM_FLAG) = 0;
        *reinterpret_cast<int32_t *>(smem + gen::SM_COUNT) = 0;
        fence_mbar_init();
    }
    __syncthreads();
    // Opening cluster barrier: arrived at here, waited for only where a block first touches a peer.
    // Warp 0 (which set the barriers up) arrives with release; the others have nothing to publish.
    if (warp == 0) cluster_arrive();
    else cluster_arrive_relaxed();
    // Activations are only touched after griddep_wait().  The unit records and the pool were
    // complete before the preceding kernel started when P.early is set (the host sets it only
    // then), so they are read, and the first weight tiles requested, ahead of the wait.
    if (!P.early) griddep_wait();
    if (warp == NWC) {
        gen::producer(P, smem, cid, G, crank, lane);
        cluster_wait();     // the opening barrier (this warp touches no peer)
        cluster_arrive();   // the closing one
    } else {
        gen::consumers<H>(P, smem, cid, G, crank, csize);
    }
    // A block that gave up may still have copies on their way into its shared memory; they must
    // land before the block leaves: all five warps meet, then one thread waits, bounded, for the
    // most recent job of every stage.
    __syncthreads();
    if (*reinterpret_cast<volatile int32_t *>(smem + gen::SM_FLAG) && tid == 0) {
        const int32_t issued = *reinterpret_cast<volatile int32_t *>(smem + gen::SM_COUNT);
        for (int32_t q = max(issued - P.n_stages, 0); q < issued; ++q)
            mbar_wait(reinterpret_cast<uint64_t *>(smem + gen::SM_FULL) + q % P.n_stages,
                      (uint32_t)(q / P.n_stages) & 1u);
    }
    // No block leaves while a peer may still read its partials or signal its barriers: every block
    // of the cluster has arrived at the closing barrier (the hardware one, which each block reaches
    // whatever happened before) only after its last access to a peer.
    cluster_wait();
}

}  // namespace lora
