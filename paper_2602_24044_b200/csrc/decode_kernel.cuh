// The decode form of the fused LoRA forward (paper Section 2.2), included by apply_fused.cu.
//
// Decode batches are what a serving step mostly consists of: a handful of tokens per adapter, ranks
// of 16 or less, grouped metadata.  For them this kernel replaces the general fused kernel with one
// whose consumers hold no control logic at all: the requesting warp walks the units, and every job
// it places in the ring carries a 16-byte header (shrink or expand chunk, first / last of its unit,
// columns, which unit entry), so the four consumer warps simply follow the stream
//     shrink(u0) shrink(u1) expand(u0) shrink(u2) expand(u1) ... end
// A unit entry (rows, rank rows, scale, projection, token ids) sits in a small ring in shared
// memory, written by the requesting warp before the unit's first job is signalled.
//
// Same decomposition as the general kernel: a cluster of blocks owns a unit of at most 8 token rows
// of one adapter in one projection; block c takes the c-th slice of d_in (shrink) and of d_out
// (expand); the block partials are pushed into every block of the cluster and summed there in block
// order (by every warp for its own MMA fragments); v goes into the expand MMAs as the sum of two bf16 numbers; scale and residual add are
// fused; one rounding at the store.  Requirements (checked by the host, which otherwise uses the
// general kernel): grouped metadata with tile_m <= 8, every occupied slot of rank <= 16, d_in and
// d_out multiples of 64.
#pragma once

namespace lora {
namespace dec {

constexpr int SM_FULL = 0;       // mbarriers: a job's data has landed            [MAX_STAGES]
constexpr int SM_EMPTY = 32;     // mbarriers: the consumer warps have left a stage [MAX_STAGES]
constexpr int SM_XB = 64;        // two mbarriers: every block has published its partial
constexpr int SM_YB = 80;        // two mbarriers: every block has read the partials
constexpr int SM_FLAG = 96;      // int32: a bounded wait of this block has expired
constexpr int SM_COUNT = 100;    // int32: jobs requested so far
constexpr int SM_CBAR = 104;     // mbarrier: the 128 consumer threads meet (bounded, unlike bar.sync)
constexpr int SM_JOB = 128;      // job headers, 16 bytes per stage
constexpr int SM_UNIT = 192;     // unit entries, 64 bytes each, ring of eight
constexpr int UNIT_ENTRIES = 8;
constexpr int SM_PART = 704;     // [4 column blocks][8 rows][16 ranks] fp32: the warps' partial sums
constexpr int SM_VALL = SM_PART + 2048;          // two sets of [8 blocks][8 rows][16 ranks] fp32
constexpr int SM_W = 11264;                      // weight tiles, W_BYTES per stage
constexpr int TOK_BYTES = 8 * TOK_PITCH * 2;     // token rows of a stage
static_assert(SM_VALL + 2 * 4096 <= SM_W && SM_W % 1024 == 0, "header fits");

enum { J_SHRINK = 1, J_FIRST = 2, J_LAST = 4, J_END = 8 /* no data, stream over */, J_FINAL = 16 /* last job of the stream */ };

struct UnitEntry {          // 64 bytes
    int32_t rows, rb, rank, item;
    float scale;
    int32_t b_lo;           // first column of this block's slice of d_out
    int32_t pad[2];
    int32_t rowid[8];
};

inline int smem_bytes(int stages) { return SM_W + stages * (W_BYTES + TOK_BYTES); }

// ---------------------------------------------------------------------------------------------
// the requesting warp
// ---------------------------------------------------------------------------------------------
struct PUnit {              // what the requesting warp keeps of a unit
    int32_t slot, rows, rb, rank, item;
    int32_t na, nb, a_lo, a_hi, b_lo, b_hi;
    float scale;
    bool run;
};

__device__ __forceinline__ PUnit p_decode(const FusedParams &P, uint32_t crank, const int4 rec, int32_t item) {
    PUnit u;
    u.slot = rec.x;
    u.rows = rec.z & 0xff;
    u.rank = (rec.z >> 17) & 0x7f;
    u.rb = (u.rank + 7) & ~7;
    u.scale = __int_as_float(rec.w);
    u.item = min(item, P.n_items - 1);
    const FusedItem &it = P.item[u.item];
    u.a_lo = min((int32_t)crank * it.wa, it.d_in);
    u.a_hi = min(u.a_lo + it.wa, it.d_in);
    u.b_lo = min((int32_t)crank * it.wb, it.d_out);
    u.b_hi = min(u.b_lo + it.wb, it.d_out);
    u.run = rec.x >= 0 && u.rows > 0 && u.rank > 0;
    u.na = (u.a_hi - u.a_lo + 255) >> 8;
    u.nb = (u.b_hi - u.b_lo + 255) >> 8;
    return u;
}

// One job into stage st: header, weight tile, token rows.  mode 0: all; 1: header and tile (with the
// byte count of the whole job); 2: the token rows of a job started in mode 1.
__device__ __forceinline__ void p_request(const FusedParams &P, unsigned char *smem, const PUnit &un,
                                          int32_t j, int32_t entry, int st, int32_t rowid, int lane, int mode,
                                          bool final_job = false) {
    const FusedItem &it = P.item[un.item];
    uint64_t *full = reinterpret_cast<uint64_t *>(smem + SM_FULL) + st;
    const bool shrink = j < un.na;
    const int32_t c = shrink ? j : j - un.na;
    const int32_t col0 = (shrink ? un.a_lo : un.b_lo) + c * 256;
    const int32_t ncols = min(256, (shrink ? un.a_hi : un.b_hi) - col0);
    if (lane == 0 && mode != 2) {
        const int32_t last = shrink ? un.na - 1 : un.nb - 1;
        *reinterpret_cast<int4 *>(smem + SM_JOB + 16 * st) =
            make_int4((shrink ? J_SHRINK : 0) | (c == 0 ? J_FIRST : 0) | (c == last ? J_LAST : 0) |
                          (final_job ? J_FINAL : 0), entry, c, ncols);
        const CUtensorMap *map = P.maps + it.map_base + (shrink ? 0 : 8) + (un.rb >> 3) - 1;
        // the tile load always delivers its whole box: rb rows of 256 columns
        mbar_expect_tx(full, (uint32_t)un.rb * 512u + (uint32_t)un.rows * (uint32_t)ncols * 2u);
        tma_load_4d(smem + SM_W + st * W_BYTES, map, 0, 0, col0 >> 6, un.slot, full);
    }
    __syncwarp();
    if (lane < un.rows && mode != 1) {
        const __nv_bfloat16 *tok = (shrink ? it.x : it.yb) + col0 + (int64_t)rowid * (shrink ? it.ldx : it.ldyb);
        bulk_g2s(smem + SM_W + P.n_stages * W_BYTES + st * TOK_BYTES + lane * (TOK_PITCH * 2), tok,
                 (uint32_t)ncols * 2u, full);
    }
}

// The first global loads of the requesting warp: the unit count and (speculatively, as if the
// table were full) the cluster's first record, side by side.  Issued at the very top of the kernel
// when the table may be read ahead of the preceding kernel's end, else after the wait.
struct FirstLoads {
    int32_t n_units;
    int4 rec;
    int32_t rowid;
};
__device__ __forceinline__ FirstLoads first_loads(const FusedParams &P, int32_t cid, int lane) {
    FirstLoads f;
    f.n_units = ldg_int(P.meta + H_NPIECE);
    f.rec = make_int4(-2, 0, 0, 0);
    f.rowid = 0;
    if (P.n_items == 1 && cid < P.units_cap) {
        if (lane == 16) f.rec = ldg_int4(P.meta + P.moff_udesc + 4 * (int64_t)cid);
        else if (lane < 16) f.rowid = ldg_int(P.meta + P.moff_uperm + 16 * (int64_t)cid + lane);
    }
    return f;
}

__device__ __forceinline__ void producer(const FusedParams &P, unsigned char *smem, int32_t cid, int32_t G,
                                         uint32_t crank, int lane, const FirstLoads &fl) {
    const int32_t S = P.n_stages;
    volatile int32_t *dead = reinterpret_cast<volatile int32_t *>(smem + SM_FLAG);
    volatile int32_t *count = reinterpret_cast<volatile int32_t *>(smem + SM_COUNT);
    uint64_t *empty = reinterpret_cast<uint64_t *>(smem + SM_EMPTY);
    int32_t n_units = fl.n_units;
    int4 rec = fl.rec;
    int32_t rowid = fl.rowid;
    auto fetch = [&](int32_t u, bool valid, int4 &r, int32_t &id) {
        r = make_int4(-2, 0, 0, 0);
        id = 0;
        if (valid) {
            if (lane == 16) r = ldg_int4(P.meta + P.moff_udesc + 4 * (int64_t)u);
            else if (lane < 16) id = ldg_int(P.meta + P.moff_uperm + 16 * (int64_t)u + lane);
        }
    };
    auto bcast = [&](int4 r) {
        r.x = __shfl_sync(0xffffffffu, r.x, 16);
        r.y = __shfl_sync(0xffffffffu, r.y, 16);
        r.z = __shfl_sync(0xffffffffu, r.z, 16);
        r.w = __shfl_sync(0xffffffffu, r.w, 16);
        return r;
    };
    if (n_units > P.units_cap) n_units = P.units_cap;
    const int32_t total = n_units * P.n_items;
    if (n_units < 1) n_units = 1;
    // position in the launch's unit list: unit g is unit u of projection `item`
    int32_t g = cid, u = cid, item = 0;
    while (u >= n_units) { u -= n_units; ++item; }
    if (P.n_items > 1) fetch(u, g < total, rec, rowid);

    int32_t q = 0, skip = 0, st = 0;
    uint32_t ph = 0;
    bool ok = true, have_pend = false, waited = !P.early;
    PUnit pend;
    int32_t pend_rowid = 0, pend_entry = 0, n_run = 0;
    bool sent_final = false;
    for (int32_t i = 0;; ++i) {
        const bool real = g < total;
        if (!real && !have_pend) break;
        int32_t gn = g + G, un_ = u + G, itn = item;
        while (un_ >= n_units) { un_ -= n_units; ++itn; }
        const bool next_real = real && gn < total;
        int4 rec_n;
        int32_t rowid_n;
        fetch(un_, next_real, rec_n, rowid_n);   // the next unit's record, meanwhile
        PUnit un = p_decode(P, crank, bcast(rec), item);
        if (!real) un.run = false;   // past the end: only the last unit's expand jobs are left
        // Entries are numbered by the units that run, not by the units walked: a cluster that
        // skips units between two that run must not come back to an entry still in use (the
        // entry of a unit is read until its last expand chunk, which follows the next running
        // unit's shrink chunks in the ring).
        const int32_t entry = n_run & (UNIT_ENTRIES - 1);
        if (un.run) ++n_run;
        if (un.run) {
            // the unit's entry; made visible to the consumers by the arrival on the barrier of
            // the unit's first job
            UnitEntry *e = reinterpret_cast<UnitEntry *>(smem + SM_UNIT) + entry;
            if (lane == 16) {
                e->rows = un.rows; e->rb = un.rb; e->rank = un.rank; e->item = un.item;
                e->scale = un.scale; e->b_lo = un.b_lo;
            } else if (lane < 8) {
                e->rowid[lane] = rowid;
            }
            __syncwarp();
        }
        if (i == 0) {
            if (P.early) {
                // The kernel before this one may still be running: the pool may be read (the host
                // vouches for it), the activations not yet.  Weight tiles of the first jobs now, their
                // token rows after the wait.
                skip = !un.run ? 0 : un.na < S ? un.na : S;
                for (int32_t j = 0; j < skip; ++j) p_request(P, smem, un, j, entry, j, rowid, lane, 1);
                // and a hint to L2 for the block's slices of the unit's rows (no value is consumed)
                if (un.run && lane < un.rows) {
                    const FusedItem &it = P.item[un.item];
                    if (un.a_hi > un.a_lo)
                        bulk_prefetch_l2(it.x + (int64_t)rowid * it.ldx + un.a_lo, (uint32_t)(un.a_hi - un.a_lo) * 2u);
                    if (un.b_hi > un.b_lo)
                        bulk_prefetch_l2(it.yb + (int64_t)rowid * it.ldyb + un.b_lo, (uint32_t)(un.b_hi - un.b_lo) * 2u);
                }
            }
        }
        if (!waited) {
            griddep_wait();
            waited = true;
            for (int32_t j = 0; j < skip; ++j) {
                p_request(P, smem, un, j, entry, j, rowid, lane, 2);
                if (++st == S) { st = 0; ++ph; }
            }
            if (lane == 0) *count = skip;
            q = skip;
        }
        // this step's jobs in ring order: the unit's shrink chunks, then the pending unit's expand chunks
        const int32_t ja = un.run ? un.na : 0, jb = have_pend ? pend.nb : 0;
        for (int32_t k = (i == 0 ? skip : 0); k < ja + jb; ++k) {
            if (q >= S && ok) {
                ok = mbar_wait(&empty[st], (ph - 1u) & 1u);
                if (!ok) *dead = 1;
            }
            if (ok && !*dead) {
                if (k < ja) p_request(P, smem, un, k, entry, st, rowid, lane, 0);
                else p_request(P, smem, pend, pend.na + k - ja, pend_entry, st, pend_rowid, lane, 0,
                               !real && k == ja + jb - 1);   // nothing follows the last unit's last expand chunk
                if (lane == 0) *count = q + 1;
            }
            ++q;
            if (++st == S) { st = 0; ++ph; }
        }
        if (!real && jb > 0) sent_final = true;
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
    // A stream without any job (no unit for this cluster, or units without expand chunks at its
    // end) is closed by a job without data; otherwise the last expand chunk carried the mark.
    if (!sent_final) {
        if (q >= S && ok) {
            ok = mbar_wait(&empty[st], (ph - 1u) & 1u);
            if (!ok) *dead = 1;
        }
        if (ok && !*dead && lane == 0) {
            *reinterpret_cast<int4 *>(smem + SM_JOB + 16 * st) = make_int4(J_END, 0, 0, 0);
            mbar_arrive(reinterpret_cast<uint64_t *>(smem + SM_FULL) + st);
        }
    }
    if (!ok && lane == 0) atomicAdd(&P.pool.status[STATUS_TIMEOUTS], 1);
}

// ---------------------------------------------------------------------------------------------
// the consumer warps: follow the job stream
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void consumers(const FusedParams &P, unsigned char *smem, int32_t cid, int32_t G,
                                          uint32_t crank, uint32_t csize) {
    constexpr int PW = TOK_PITCH;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, t = lane & 3;
    const int mi = lane >> 3, r = lane & 7;
    uint64_t *full = reinterpret_cast<uint64_t *>(smem + SM_FULL);
    uint64_t *empty = reinterpret_cast<uint64_t *>(smem + SM_EMPTY);
    volatile int32_t *dead = reinterpret_cast<volatile int32_t *>(smem + SM_FLAG);
    float *part = reinterpret_cast<float *>(smem + SM_PART);
    const uint32_t w_base = smem_u32(smem + SM_W), t_base = w_base + (uint32_t)P.n_stages * W_BYTES;
    // Operand fragments come by ldmatrix; lane l names row (l & 7) of 8x8 matrix (l >> 3).
    //  shrink, weights: matrices (ranks 0-7, k 0-7) (ranks 0-7, k 8-15) (ranks 8-15, k 0-7) (ranks 8-15,
    //          k 8-15) of this warp's column block; rank row n sits at n * 128 bytes, its 16-byte
    //          chunk c at ((c ^ (n & 7)) << 4); the even part of c is folded in per step with one XOR
    //  shrink, tokens: matrices (rows 0-7, k 0-7) (rows 0-7, k 8-15)
    //  expand, weights (transposing): rank row 8 (mi & 1) + r of column tile 2 np + (mi >> 1)
    const uint32_t wsh_lane = (uint32_t)(8 * (mi >> 1) + r) * 128u + (uint32_t)(((mi & 1) ^ r) << 4);
    const uint32_t xsh_lane = (uint32_t)(r * PW + (mi & 1) * 8) * 2u + (uint32_t)warp * 128u;
    const uint32_t wex_lane = (uint32_t)((mi & 1) * 8 + r) * 128u + (uint32_t)(((mi >> 1) ^ r) << 4);
    const uint32_t yex_lane = (uint32_t)(g * PW + warp * 64 + 2 * t) * 2u;

    float acc[2][4];
#pragma unroll
    for (int i = 0; i < 2; ++i) acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0.0f;
    uint32_t ah[4] = {0u, 0u, 0u, 0u}, al[4] = {0u, 0u, 0u, 0u};
    __nv_bfloat16 *yp = nullptr;
    float scale = 0.0f;
    bool row_ok = false, upper = true;
    int32_t st = 0, kp = 0, kr = 0;
    uint32_t ph = 0, blk_bytes = 0;
    bool ok = true;
    bool met_cluster = false;   // the opening cluster barrier has been waited for (needed before the first remote access)
    // rows without adapter are copied at the end (out-of-place projections): their number, asked for now
    const int32_t n_active = P.copy_idle ? ldg_int(P.meta + H_NACTIVE) : P.T;
    // The consumer threads meet on an mbarrier, not on bar.sync: a thread that has given up a wait
    // never arrives, and the others must not wait for it without a limit.
    uint32_t cs = 0;
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
        const UnitEntry *ue = reinterpret_cast<const UnitEntry *>(smem + SM_UNIT) + job.y;
        const int32_t ncols = job.w - warp * 64;   // of this warp's 64 columns
        if (job.x & J_SHRINK) {
            if (job.x & J_FIRST) {
#pragma unroll
                for (int i = 0; i < 2; ++i) acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0.0f;
            }
            if (ncols > 0) {
                const uint32_t As = w_base + st * W_BYTES + (uint32_t)warp * ((uint32_t)ue->rb * 128u) + wsh_lane;
                const uint32_t X = t_base + st * TOK_BYTES + xsh_lane;
#pragma unroll
                for (int ks = 0; ks < 64; ks += 16) {
                    uint32_t a[4], bw[4];
                    ldmatrix_x2(a[0], a[2], X + ks * 2);
                    a[1] = a[3] = 0u;
                    ldmatrix_x4(bw, As ^ (uint32_t)((ks >> 3) << 4));
                    mma16816(acc[0], a, bw[0], bw[1]);
                    mma16816(acc[1], a, bw[2], bw[3]);
                }
            }
            const int32_t rows = ue->rows;
            __syncwarp();
            if (lane == 0) mbar_arrive(&empty[st]);
            if (job.x & J_LAST) {
                // ---- the block's partial goes to every block of the cluster (buffer set kp & 1) ----
                const int b = kp & 1;
                if (kp >= 2) {   // the peers have read what this set held two units ago
                    ok = __all_sync(0xffffffffu, mbar_wait_cluster(reinterpret_cast<uint64_t *>(smem + SM_YB) + b,
                                                                   (uint32_t)((kp - 2) >> 1) & 1u));
                    if (!ok) {
                        *dead = 1;
                        break;
                    }
                }
                float *p0 = part + (warp * 8 + g) * 16 + 2 * t;
                *reinterpret_cast<float2 *>(p0) = make_float2(acc[0][0], acc[0][1]);
                *reinterpret_cast<float2 *>(p0 + 8) = make_float2(acc[1][0], acc[1][1]);
                if (!met_cluster) {   // no block is written to before its barriers are set up
                    cluster_wait();
                    met_cluster = true;
                }
                // this block will receive rows x 16 floats from every block of the cluster
                if (tid == 0) mbar_expect_tx(reinterpret_cast<uint64_t *>(smem + SM_XB) + b, csize * (uint32_t)rows * 64u);
                if (!meet()) { ok = false; break; }
                // thread (row, rank): the four column blocks' sums in order, sent to every block; each
                // store counts its bytes on the receiver's barrier, so data and signal travel together
                if ((tid >> 4) < rows) {
                    const float v = ((part[tid] + part[128 + tid]) + part[256 + tid]) + part[384 + tid];
                    const uint32_t dst = smem_u32(smem + SM_VALL + b * 4096 + ((int)crank * 128 + tid) * 4);
                    const uint32_t bar = smem_u32(smem + SM_XB + 8 * b);
                    for (uint32_t q = 0; q < csize; ++q) st_async_peer_f32(dst, bar, q, v);
                }
                ++kp;
            }
        } else {
            if (job.x & J_FIRST) {
                // ---- every block sums the cluster's partials in block order (buffer set kr & 1) ----
                const int b = kr & 1;
                ok = __all_sync(0xffffffffu, mbar_wait_cluster(reinterpret_cast<uint64_t *>(smem + SM_XB) + b,
                                                               (uint32_t)(kr >> 1) & 1u));
                if (!ok) {
                    *dead = 1;
                    break;
                }
                const int32_t rows = ue->rows, rank = ue->rank;
                {
                    // This lane's four elements of v (row g; ranks 2t, 2t+1, 2t+8, 2t+9: its MMA row
                    // fragments), each the sum of the blocks' partials in block order.  Every warp
                    // takes the same sums from the block's own shared memory, so nothing has to be
                    // handed from thread to thread.  All loads are issued before the first add.
                    const float *vs = reinterpret_cast<const float *>(smem + SM_VALL + b * 4096) + g * 16 + 2 * t;
                    float2 p0[8], p1[8];
#pragma unroll
                    for (uint32_t q = 0; q < 8; ++q) {
                        p0[q] = q < csize ? *reinterpret_cast<const float2 *>(vs + q * 128) : make_float2(0.0f, 0.0f);
                        p1[q] = q < csize ? *reinterpret_cast<const float2 *>(vs + q * 128 + 8) : make_float2(0.0f, 0.0f);
                    }
                    float v0 = 0.0f, v1 = 0.0f, v2 = 0.0f, v3 = 0.0f;
#pragma unroll
                    for (uint32_t q = 0; q < 8; ++q) {
                        v0 += p0[q].x; v1 += p0[q].y; v2 += p1[q].x; v3 += p1[q].y;
                    }
                    // ranks the adapter does not have carry no meaning (and may hold anything)
                    if (2 * t >= rank) v0 = 0.0f;
                    if (2 * t + 1 >= rank) v1 = 0.0f;
                    if (2 * t + 8 >= rank) v2 = 0.0f;
                    if (2 * t + 9 >= rank) v3 = 0.0f;
                    // v as MMA row operand, high and low bf16 parts (rows 8..15 of the MMA stay
                    // zero), kept in registers for all of the unit's jobs
                    const __nv_bfloat162 h01 = __floats2bfloat162_rn(v0, v1), h23 = __floats2bfloat162_rn(v2, v3);
                    ah[0] = *reinterpret_cast<const uint32_t *>(&h01);
                    ah[2] = *reinterpret_cast<const uint32_t *>(&h23);
                    al[0] = pack2(v0 - __low2float(h01), v1 - __high2float(h01));
                    al[2] = pack2(v2 - __low2float(h23), v3 - __high2float(h23));
                }
                // done reading the partials (every warp tells every block on its own); the matching
                // wait comes before the set is written again
                __syncwarp();
                if (lane < (int)csize) mbar_arrive_peer(reinterpret_cast<uint64_t *>(smem + SM_YB) + b, (uint32_t)lane);
                ++kr;
                const FusedItem &it = P.item[ue->item];
                row_ok = g < rows;
                yp = it.y + (int64_t)(row_ok ? ue->rowid[g] : 0) * it.ldy + ue->b_lo + warp * 64 + 2 * t;
                scale = ue->scale;
                blk_bytes = (uint32_t)ue->rb * 128u;
                // Rank rows 8..15 were only copied when the tile has them; what the stage holds there
                // otherwise belongs to an earlier job (possibly another adapter's weights) and must
                // not meet the MMA, not even multiplied by zero.
                upper = ue->rb > 8;
            }
            if (ncols > 0) {
                const uint32_t Bs = w_base + st * W_BYTES + (uint32_t)warp * blk_bytes + wex_lane;
                const uint32_t Ys = t_base + st * TOK_BYTES + yex_lane;
                __nv_bfloat16 *yj = yp + job.z * 256;
#pragma unroll
                for (int np = 0; np < 4; ++np) {
                    float ex[2][4];
                    uint32_t bb[4];
                    ldmatrix_x4_trans(bb, Bs ^ (uint32_t)(np << 5));
                    if (!upper) bb[1] = bb[3] = 0u;
                    mma16816_first(ex[0], ah, bb[0], bb[1]);
                    mma16816_first(ex[1], ah, bb[2], bb[3]);
                    mma16816(ex[0], al, bb[0], bb[1]);
                    mma16816(ex[1], al, bb[2], bb[3]);
                    // epilogue straight from the accumulator layout: each lane owns two adjacent
                    // columns of row g per column tile; a quad covers 16 contiguous bytes
                    if (row_ok) {
#pragma unroll
                        for (int j = 0; j < 2; ++j) {
                            const int coff = (2 * np + j) * 8;
                            uint32_t w;
                            asm volatile("ld.shared.b32 %0, [%1];" : "=r"(w) : "r"(Ys + coff * 2));
                            const float a0 = fmaf(scale, ex[j][0], __uint_as_float(w << 16));
                            const float a1 = fmaf(scale, ex[j][1], __uint_as_float(w & 0xffff0000u));
                            *reinterpret_cast<uint32_t *>(yj + coff) = pack2(a0, a1);
                        }
                    }
                }
            }
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

    // rows that take no adapter: y_base -> y, 16 rows per cluster step (out-of-place projections)
    if (ok && !*dead && n_active < P.T) {
        int32_t *rowidx = reinterpret_cast<int32_t *>(smem + SM_PART);
        const int32_t n_idle = P.T - n_active;
        const int32_t chunks = (n_idle + 15) / 16;
        for (int32_t k = cid; k < chunks * P.n_items; k += G) {
            const int32_t item = k / chunks, first = (k - item * chunks) * 16;
            const FusedItem &it = P.item[item];
            if (it.in_place) continue;
            const int32_t rows = min(16, n_idle - first);
            if (!meet()) break;
            if (tid < rows) rowidx[tid] = __ldg(P.meta + P.moff_perm + (P.T - n_idle) + first + tid);
            if (!meet()) break;
            // the chunk's rows as one index space (row, 16-byte vector of this block's share), four
            // independent loads in flight per thread
            const int32_t vecs = it.d_out / 8;
            const int32_t per_blk = (vecs + (int32_t)csize - 1) / (int32_t)csize;
            const int32_t v_lo = (int32_t)crank * per_blk, v_n = max(0, min(per_blk, vecs - v_lo));
            const int32_t total = rows * v_n;
            for (int32_t i0 = tid; i0 < total; i0 += 4 * FT) {
                uint4 val[4];
                int64_t off[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const int32_t i = i0 + q * FT;
                    const int32_t m = i < total ? i / v_n : 0, v = i < total ? v_lo + i - m * v_n : 0;
                    off[q] = (int64_t)rowidx[m];
                    val[q] = make_uint4(0, 0, 0, 0);
                    if (i < total) val[q] = ldg16(it.yb + off[q] * it.ldyb + (int64_t)v * 8);
                    off[q] = off[q] * it.ldy + (int64_t)v * 8;
                }
#pragma unroll
                for (int q = 0; q < 4; ++q)
                    if (i0 + q * FT < total) *reinterpret_cast<uint4 *>(it.y + off[q]) = val[q];
            }
        }
    }
}

}  // namespace dec

__global__ void __launch_bounds__(FT_ALL, LORA_FUSED_MIN_BLOCKS)
decode_kernel(const __grid_constant__ FusedParams P) {
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
    // what the requesting warp needs first from global memory, asked for before anything else when
    // the table may be read now
    dec::FirstLoads fl;
    fl.n_units = 0;
    fl.rec = make_int4(-2, 0, 0, 0);
    fl.rowid = 0;
    if (warp == 4 && P.early) fl = dec::first_loads(P, cid, lane);
    if (warp == 4 && lane < MAPS_PER_TARGET) prefetch_tensormap(P.maps + P.item[0].map_base + lane);
    if (tid == 0) {
        uint64_t *full = reinterpret_cast<uint64_t *>(smem + dec::SM_FULL);
        uint64_t *empty = reinterpret_cast<uint64_t *>(smem + dec::SM_EMPTY);
        for (int s = 0; s < P.n_stages; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], 4);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(reinterpret_cast<uint64_t *>(smem + dec::SM_XB) + b, 1);
            mbar_init(reinterpret_cast<uint64_t *>(smem + dec::SM_YB) + b, 4 * csize);
        }
        mbar_init(reinterpret_cast<uint64_t *>(smem + dec::SM_CBAR), FT);
        *reinterpret_cast<int32_t *>(smem + dec::SM_FLAG) = 0;
        *reinterpret_cast<int32_t *>(smem + dec::SM_COUNT) = 0;
        fence_mbar_init();
    }
    __syncthreads();
    // Opening cluster barrier: arrived at here, waited for only where a block first touches a peer.
    // Warp 0 (which set the barriers up) arrives with release; the others have nothing to publish
    // and must not wait for their loads in flight.
    if (warp == 0) cluster_arrive();
    else cluster_arrive_relaxed();
    // Activations are only touched after griddep_wait().  The unit records and the pool were
    // complete before the preceding kernel started when P.early is set (the host sets it only
    // then), so they are read, and the first weight tiles requested, ahead of the wait.
    if (!P.early) {
        griddep_wait();
        if (warp == 4) fl = dec::first_loads(P, cid, lane);
    }
    if (warp == 4) {
        dec::producer(P, smem, cid, G, crank, lane, fl);
        cluster_wait();     // the opening barrier (this warp touches no peer)
        cluster_arrive();   // the closing one
    } else {
        dec::consumers(P, smem, cid, G, crank, csize);
    }
    // A block that gave up may still have copies on their way into its shared memory; they must
    // land before the block leaves: all five warps meet, then one thread waits, bounded, for the
    // most recent job of every stage.
    __syncthreads();
    if (*reinterpret_cast<volatile int32_t *>(smem + dec::SM_FLAG) && tid == 0) {
        const int32_t issued = *reinterpret_cast<volatile int32_t *>(smem + dec::SM_COUNT);
        for (int32_t q = max(issued - P.n_stages, 0); q < issued; ++q)
            mbar_wait(reinterpret_cast<uint64_t *>(smem + dec::SM_FULL) + q % P.n_stages,
                      (uint32_t)(q / P.n_stages) & 1u);
    }
    // No block leaves while a peer may still write into its buffers or signal its barriers: every
    // block of the cluster has arrived at the closing barrier (the hardware one, which each block
    // reaches whatever happened before) only after its last access to a peer.
    cluster_wait();
}

}  // namespace lora
