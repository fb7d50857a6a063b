// Segment metadata: a stable group-by-slot of the batch's tokens (several adapters are served
// inside one batch, paper Section 2.2; each request names its adapter, Section 5), cut into row
// tiles.  Integer work only; the result is a unique function of the inputs.
//
// One launch, no inter-block communication: every block recomputes the per-slot histogram and
// its prefix sums (O(T + N) integer work from L2), then each warp owns whole slots and writes
// that slot's run of `perm` by scanning the token list in order with warp ballots, which makes
// the order inside a run ascending by construction.
#include "apply_common.cuh"

namespace lora {

constexpr int SEG_THREADS = 256;
constexpr int SEG_WARPS = SEG_THREADS / 32;

__global__ void __launch_bounds__(SEG_THREADS)
build_segments_kernel(PoolView pool, const int32_t *__restrict__ slot_idx_g, int32_t T,
                      int32_t tile_m, int32_t long_min, int32_t *meta, int32_t staged) {
    extern __shared__ int32_t sm[];
    const int32_t N = pool.num_slots;
    int32_t *cnt = sm;             // [N] tokens per slot
    int32_t *start = cnt + N;      // [N] first position in perm
    int32_t *segid = start + N;    // [N] segment number
    int32_t *tile0 = segid + N;    // [N] first tile number
    int32_t *occ = tile0 + N;      // [N] slot occupied (copy of the slot table's flag)
    int32_t *piece0 = occ + N;     // [N] first 16-row piece number
    const MetaLayout L = meta_layout(T, N, tile_m);
    int32_t *tfirst = piece0 + N;          // [cap_tile] first token id of a tile
    int32_t *tlast = tfirst + L.cap_tile;  // [cap_tile] last token id of a tile
    int32_t *tok = tlast + L.cap_tile;     // [T] copy of the token list (only when `staged`)
    __shared__ int32_t warp_tot[4][SEG_WARPS];
    __shared__ int32_t totals[4];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // programmatic dependent launch: the next kernel of the stream may be scheduled now; this one
    // waits until everything queued before it is complete (no-ops without the launch attribute)
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");

    // ---- 1. histogram of active tokens ------------------------------------------------------
    // The slot flags and (for batches that fit) the token list are copied to shared memory with
    // independent loads first, so that the scans below do not pay a global round trip per step.
    for (int32_t s = tid; s < N; s += SEG_THREADS) {
        cnt[s] = 0;
        occ[s] = pool.table[s].loaded;
    }
    if (staged)
        for (int32_t t = tid; t < T; t += SEG_THREADS) tok[t] = slot_idx_g[t];
    const int32_t *slot_idx = staged ? tok : slot_idx_g;
    __syncthreads();
    // one shared-memory atomic per distinct slot per warp step: prefill batches are long runs of
    // one slot, which would otherwise serialise on a single counter
    for (int32_t base = warp * 32; base < T; base += SEG_THREADS) {
        const int32_t t = base + lane;
        const int32_t s = t < T ? slot_idx[t] : -1;
        const bool act = s >= 0 && s < N && occ[s];
        const uint32_t peers = __match_any_sync(0xffffffffu, act ? s : N + lane);
        if (act && lane == __ffs(peers) - 1) atomicAdd(&cnt[s], __popc(peers));
    }
    __syncthreads();

    // ---- 2. exclusive prefix sums over slots: positions, segment numbers, tile numbers ------
    const int32_t per = (N + SEG_THREADS - 1) / SEG_THREADS;
    const int32_t lo = min(tid * per, N), hi = min(lo + per, N);
    // 16-row pieces of a segment of n tokens: full tiles have ppt pieces, the last tile fewer
    const int32_t ppt = (tile_m + 15) / 16;
    auto pieces_of = [&](int32_t n) {
        return (n / tile_m) * ppt + ((n % tile_m) + 15) / 16;
    };
    int32_t c = 0, z = 0, tl = 0, pc = 0;
    for (int32_t s = lo; s < hi; ++s) {
        c += cnt[s];
        z += cnt[s] > 0;
        tl += (cnt[s] + tile_m - 1) / tile_m;
        pc += pieces_of(cnt[s]);
    }
    int32_t ic = c, iz = z, it = tl, ip = pc;   // inclusive warp scans
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int32_t a = __shfl_up_sync(0xffffffffu, ic, o);
        const int32_t b = __shfl_up_sync(0xffffffffu, iz, o);
        const int32_t d = __shfl_up_sync(0xffffffffu, it, o);
        const int32_t e = __shfl_up_sync(0xffffffffu, ip, o);
        if (lane >= o) { ic += a; iz += b; it += d; ip += e; }
    }
    if (lane == 31) {
        warp_tot[0][warp] = ic; warp_tot[1][warp] = iz; warp_tot[2][warp] = it; warp_tot[3][warp] = ip;
    }
    __syncthreads();
    int32_t bc = 0, bz = 0, bt = 0, bp = 0;
    for (int w = 0; w < warp; ++w) {
        bc += warp_tot[0][w]; bz += warp_tot[1][w]; bt += warp_tot[2][w]; bp += warp_tot[3][w];
    }
    int32_t rc = bc + ic - c, rz = bz + iz - z, rt = bt + it - tl, rp = bp + ip - pc;
    for (int32_t s = lo; s < hi; ++s) {
        start[s] = rc;
        segid[s] = rz;
        tile0[s] = rt;
        piece0[s] = rp;
        rc += cnt[s];
        rz += cnt[s] > 0;
        rt += (cnt[s] + tile_m - 1) / tile_m;
        rp += pieces_of(cnt[s]);
    }
    if (tid == SEG_THREADS - 1) { totals[0] = rc; totals[1] = rz; totals[2] = rt; totals[3] = rp; }
    __syncthreads();
    const int32_t n_active = totals[0], n_seg = totals[1], n_tile = totals[2], n_piece = totals[3];

    int32_t *perm = meta + L.perm;
    // ---- 3. one warp per occupied slot: write its run of perm, its segment and its tiles ----
    for (int32_t s = blockIdx.x * SEG_WARPS + warp; s < N; s += gridDim.x * SEG_WARPS) {
        const int32_t n = cnt[s];
        if (n == 0) continue;
        const int32_t p0 = start[s], seg = segid[s];
        // the slot's rank and scale for the records below: asked for now, needed after the scan, so
        // that this trip to global memory is off the critical path
        const int4 slot_entry = __ldg(reinterpret_cast<const int4 *>(pool.table + s));
        int32_t run = 0;
        // 128 tokens per step: the four loads are independent, the ballots keep token order
        for (int32_t base = 0; base < T && run < n; base += 128) {
            int32_t sv[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int32_t t = base + q * 32 + lane;
                sv[q] = t < T ? slot_idx[t] : -2;
            }
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int32_t t = base + q * 32 + lane;
                const bool hit = sv[q] == s;
                const uint32_t m = __ballot_sync(0xffffffffu, hit);
                if (hit) {
                    const int32_t j = run + __popc(m & ((1u << lane) - 1u));
                    perm[p0 + j] = t;
                    // private copy laid out by unit (16-row piece of a tile), 16 ids per unit
                    const int32_t k = j / tile_m, jj = j - k * tile_m;
                    meta[L.unit_perm + 16 * (int64_t)(piece0[s] + k * ppt + (jj >> 4)) + (jj & 15)] = t;
                    // first and last token of every tile, kept on chip: what was just stored to
                    // global memory is not read back
                    if (jj == 0) tfirst[tile0[s] + k] = t;
                    if (jj == tile_m - 1 || j == n - 1) tlast[tile0[s] + k] = t;
                }
                run += __popc(m);
            }
        }
        __syncwarp();
        const int32_t nt = (n + tile_m - 1) / tile_m;
        const int32_t first = tfirst[tile0[s]], last = tlast[tile0[s] + nt - 1];
        if (lane == 0) {
            meta[L.seg_slot + seg] = s;
            meta[L.seg_start + seg] = p0;
            meta[L.seg_rank + seg] = slot_entry.x;
            meta[L.seg_flags + seg] = (last - first + 1 == n ? 1 : 0) | (n >= long_min ? 2 : 0);
        }
        for (int32_t k = lane; k < nt; k += 32) {
            const int32_t r0 = p0 + k * tile_m;
            const int32_t rows = min(tile_m, p0 + n - r0);
            const int32_t idx = tile0[s] + k;
            meta[L.tile_seg + idx] = seg;
            meta[L.tile_row0 + idx] = r0;
            meta[L.tile_rows + idx] = rows;
            const int32_t contiguous = (tlast[idx] - tfirst[idx] + 1 == rows) ? 1 : 0;
            meta[L.tile_flags + idx] = contiguous;
            SlotEntry e;
            e.rank = slot_entry.x;
            e.scale = __int_as_float(slot_entry.y);
            // private record: slot, position, rows (bits 0-14) | consecutive ids (bit 15) | rank, scale
            *reinterpret_cast<int4 *>(meta + L.tile_desc + 4 * (int64_t)idx) =
                make_int4(s, r0, rows | (contiguous << 15) | (e.rank << 16), __float_as_int(e.scale));
            // private unit records: the tile's pieces of at most 16 rows (all earlier tiles of the
            // segment are full, so they have ppt pieces each)
            for (int32_t i = 0; i < (rows + 15) / 16; ++i)
                *reinterpret_cast<int4 *>(meta + L.unit_desc + 4 * (int64_t)(piece0[s] + k * ppt + i)) =
                    make_int4(s, r0 + 16 * i,
                              min(16, rows - 16 * i) | (rows << 8) | (contiguous << 16) | (e.rank << 17),
                              __float_as_int(e.scale));
        }
    }

    // ---- 4. last block: header, the inactive tail of perm, -1 in unused entries -------------
    if (blockIdx.x != gridDim.x - 1) return;
    if (warp == 0) {
        int32_t run = 0, n_invalid = 0;
        for (int32_t base = 0; base < T; base += 32) {
            const int32_t t = base + lane;
            const int32_t s = t < T ? slot_idx[t] : -1;
            const bool inact = t < T && !(s >= 0 && s < N && occ[s]);
            const uint32_t m = __ballot_sync(0xffffffffu, inact);
            const uint32_t bad = __ballot_sync(0xffffffffu, inact && s != -1);
            if (inact) perm[n_active + run + __popc(m & ((1u << lane) - 1u))] = t;
            run += __popc(m);
            n_invalid += __popc(bad);
        }
        if (lane == 0) {
            meta[H_T] = T;
            meta[H_NACTIVE] = n_active;
            meta[H_NINVALID] = n_invalid;
            meta[H_NSEG] = n_seg;
            meta[H_NTILE] = n_tile;
            meta[H_TILE_M] = tile_m;
            meta[H_LONG_MIN] = long_min;
            meta[H_NSLOTS] = N;
            meta[H_CAP_SEG] = L.cap_seg;
            meta[H_CAP_TILE] = L.cap_tile;
            meta[H_NPIECE] = n_piece;
            for (int i = H_NPIECE + 1; i < META_HEADER_WORDS; ++i) meta[i] = 0;
            meta[L.seg_start + n_seg] = n_active;
            if (n_invalid) atomicAdd(&pool.status[STATUS_INVALID_TOKENS], n_invalid);
        }
    } else {
        const int t0 = tid - 32, nt = SEG_THREADS - 32;
        for (int32_t i = n_seg + t0; i < L.cap_seg; i += nt) {
            meta[L.seg_slot + i] = -1;
            meta[L.seg_rank + i] = -1;
            meta[L.seg_flags + i] = -1;
        }
        for (int32_t i = n_seg + 1 + t0; i <= L.cap_seg; i += nt) meta[L.seg_start + i] = -1;
        for (int32_t i = n_tile + t0; i < L.cap_tile; i += nt) {
            meta[L.tile_seg + i] = -1;
            meta[L.tile_row0 + i] = -1;
            meta[L.tile_rows + i] = -1;
            meta[L.tile_flags + i] = -1;
            *reinterpret_cast<int4 *>(meta + L.tile_desc + 4 * (int64_t)i) = make_int4(-1, 0, 0, 0);
        }
    }
}

// The same table for long batches (prefill): the token list is cut into chunks and the position
// of every token inside its slot's run comes from per-chunk, per-slot counts, so the work per block
// is O(T) instead of O(T) per occupied slot.  Every block builds the small tables in shared memory
// (counts, prefix sums, first and last token of every tile); the writes to global memory are
// divided: a block writes the perm entries of its own chunks and the records of its own slots.
// Tokens without an occupied slot are counted in an extra column and land behind the active ones.
// The two passes over the token list are chains of shared-memory updates per warp, so their length
// is the number of chunks a warp owns: 32 warps for the longest batches, 8 below that (where the
// larger block only costs more at its barriers).
template <int SEGC_THREADS>
__global__ void __launch_bounds__(SEGC_THREADS)
build_segments_chunked_kernel(PoolView pool, const int32_t *__restrict__ slot_idx_g, int32_t T,
                              int32_t tile_m, int32_t long_min, int32_t *meta, int32_t CH, int32_t C) {
    extern __shared__ int32_t sm[];
    constexpr int SEGC_WARPS = SEGC_THREADS / 32;
    const int32_t N = pool.num_slots, N1 = N + 1;
    const MetaLayout L = meta_layout(T, N, tile_m);
    int32_t *cnt = sm;             // [N] tokens per slot
    int32_t *start = cnt + N;      // [N] first position in perm
    int32_t *segid = start + N;    // [N] segment number
    int32_t *tile0 = segid + N;    // [N] first tile number
    int32_t *occ = tile0 + N;      // [N] slot occupied
    int32_t *piece0 = occ + N;     // [N] first unit number
    int32_t *tok = piece0 + N;     // [T] the token list
    int32_t *cnt2 = tok + T;       // [C][N + 1] per chunk and slot: count, then running position
    int32_t *tfirst = cnt2 + (int64_t)C * N1;   // [cap_tile] first token id of a tile
    int32_t *tlast = tfirst + L.cap_tile;       // [cap_tile] last token id of a tile
    __shared__ int32_t warp_tot[4][SEGC_WARPS];
    __shared__ int32_t totals[4];
    __shared__ int32_t n_invalid_s;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");

    for (int32_t s = tid; s < N; s += SEGC_THREADS) {
        cnt[s] = 0;
        occ[s] = pool.table[s].loaded;
    }
    for (int32_t i = tid; i < C * N1; i += SEGC_THREADS) cnt2[i] = 0;
    for (int32_t t = tid; t < T; t += SEGC_THREADS) tok[t] = slot_idx_g[t];
    if (tid == 0) n_invalid_s = 0;
    __syncthreads();

    // column of a token: its slot when that is occupied, else the extra column N
    auto classify = [&](int32_t t, int32_t t1, int32_t &s, bool &valid, bool &act) {
        valid = t < t1;
        s = valid ? tok[t] : -1;
        act = valid && s >= 0 && s < N && occ[s];
        return valid ? (act ? s : N) : -1 - lane;   // distinct keys for lanes past the end
    };

    // ---- 1. counts per chunk and column --------------------------------------------------------
    for (int32_t c = warp; c < C; c += SEGC_WARPS) {
        const int32_t t0 = c * CH, t1 = min(T, t0 + CH);
        for (int32_t base = t0; base < t1; base += 32) {
            int32_t s; bool valid, act;
            const int32_t col = classify(base + lane, t1, s, valid, act);
            const uint32_t peers = __match_any_sync(0xffffffffu, col);
            if (valid && lane == __ffs(peers) - 1) cnt2[c * N1 + col] += __popc(peers);
            const uint32_t bad = __ballot_sync(0xffffffffu, valid && !act && s != -1);
            if (lane == 0 && bad) atomicAdd(&n_invalid_s, __popc(bad));
            __syncwarp();
        }
    }
    __syncthreads();
    // ---- 2. per column: exclusive prefix over the chunks; per slot: totals and prefix sums -------
    for (int32_t col = tid; col < N1; col += SEGC_THREADS) {
        int32_t run = 0;
        for (int32_t c = 0; c < C; ++c) {
            const int32_t v = cnt2[c * N1 + col];
            cnt2[c * N1 + col] = run;
            run += v;
        }
        if (col < N) cnt[col] = run;
    }
    __syncthreads();
    const int32_t per = (N + SEGC_THREADS - 1) / SEGC_THREADS;
    const int32_t lo = min(tid * per, N), hi = min(lo + per, N);
    const int32_t ppt = (tile_m + 15) / 16;
    auto pieces_of = [&](int32_t n) { return (n / tile_m) * ppt + ((n % tile_m) + 15) / 16; };
    int32_t c_ = 0, z = 0, tl = 0, pc = 0;
    for (int32_t s = lo; s < hi; ++s) {
        c_ += cnt[s];
        z += cnt[s] > 0;
        tl += (cnt[s] + tile_m - 1) / tile_m;
        pc += pieces_of(cnt[s]);
    }
    int32_t ic = c_, iz = z, it = tl, ip = pc;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int32_t a = __shfl_up_sync(0xffffffffu, ic, o);
        const int32_t b = __shfl_up_sync(0xffffffffu, iz, o);
        const int32_t d = __shfl_up_sync(0xffffffffu, it, o);
        const int32_t e = __shfl_up_sync(0xffffffffu, ip, o);
        if (lane >= o) { ic += a; iz += b; it += d; ip += e; }
    }
    if (lane == 31) {
        warp_tot[0][warp] = ic; warp_tot[1][warp] = iz; warp_tot[2][warp] = it; warp_tot[3][warp] = ip;
    }
    __syncthreads();
    int32_t bc = 0, bz = 0, bt = 0, bp = 0;
    for (int w = 0; w < warp; ++w) {
        bc += warp_tot[0][w]; bz += warp_tot[1][w]; bt += warp_tot[2][w]; bp += warp_tot[3][w];
    }
    int32_t rc = bc + ic - c_, rz = bz + iz - z, rt = bt + it - tl, rp = bp + ip - pc;
    for (int32_t s = lo; s < hi; ++s) {
        start[s] = rc;
        segid[s] = rz;
        tile0[s] = rt;
        piece0[s] = rp;
        rc += cnt[s];
        rz += cnt[s] > 0;
        rt += (cnt[s] + tile_m - 1) / tile_m;
        rp += pieces_of(cnt[s]);
    }
    if (tid == SEGC_THREADS - 1) { totals[0] = rc; totals[1] = rz; totals[2] = rt; totals[3] = rp; }
    __syncthreads();
    const int32_t n_active = totals[0], n_seg = totals[1], n_tile = totals[2], n_piece = totals[3];

    // ---- 3. position of every token; first and last token of every tile --------------------------
    int32_t *perm = meta + L.perm;
    for (int32_t c = warp; c < C; c += SEGC_WARPS) {
        const int32_t t0 = c * CH, t1 = min(T, t0 + CH);
        const bool mine = (c % (int32_t)gridDim.x) == (int32_t)blockIdx.x;
        for (int32_t base = t0; base < t1; base += 32) {
            const int32_t t = base + lane;
            int32_t s; bool valid, act;
            const int32_t col = classify(t, t1, s, valid, act);
            const uint32_t peers = __match_any_sync(0xffffffffu, col);
            int32_t j = 0;
            if (valid) j = cnt2[c * N1 + col] + __popc(peers & ((1u << lane) - 1u));
            __syncwarp();
            if (valid && lane == __ffs(peers) - 1) cnt2[c * N1 + col] += __popc(peers);
            __syncwarp();
            if (act) {
                const int32_t k = j / tile_m, jj = j - k * tile_m, idx = tile0[s] + k;
                if (jj == 0) tfirst[idx] = t;
                if (jj == tile_m - 1 || j == cnt[s] - 1) tlast[idx] = t;
                if (mine) {
                    perm[start[s] + j] = t;
                    meta[L.unit_perm + 16 * (int64_t)(piece0[s] + k * ppt + (jj >> 4)) + (jj & 15)] = t;
                }
            } else if (valid && mine) {
                perm[n_active + j] = t;
            }
        }
    }
    __syncthreads();

    // ---- 4. segment, tile and unit records of this block's slots ---------------------------------
    for (int32_t s = blockIdx.x * SEGC_WARPS + warp; s < N; s += gridDim.x * SEGC_WARPS) {
        const int32_t n = cnt[s];
        if (n == 0) continue;
        const int32_t p0 = start[s], seg = segid[s];
        const int32_t nt = (n + tile_m - 1) / tile_m;
        const SlotEntry e = pool.table[s];
        if (lane == 0) {
            const int32_t first = tfirst[tile0[s]], last = tlast[tile0[s] + nt - 1];
            meta[L.seg_slot + seg] = s;
            meta[L.seg_start + seg] = p0;
            meta[L.seg_rank + seg] = e.rank;
            meta[L.seg_flags + seg] = (last - first + 1 == n ? 1 : 0) | (n >= long_min ? 2 : 0);
        }
        for (int32_t k = lane; k < nt; k += 32) {
            const int32_t r0 = p0 + k * tile_m;
            const int32_t rows = min(tile_m, p0 + n - r0);
            const int32_t idx = tile0[s] + k;
            meta[L.tile_seg + idx] = seg;
            meta[L.tile_row0 + idx] = r0;
            meta[L.tile_rows + idx] = rows;
            const int32_t contiguous = (tlast[idx] - tfirst[idx] + 1 == rows) ? 1 : 0;
            meta[L.tile_flags + idx] = contiguous;
            *reinterpret_cast<int4 *>(meta + L.tile_desc + 4 * (int64_t)idx) =
                make_int4(s, r0, rows | (contiguous << 15) | (e.rank << 16), __float_as_int(e.scale));
            for (int32_t i = 0; i < (rows + 15) / 16; ++i)
                *reinterpret_cast<int4 *>(meta + L.unit_desc + 4 * (int64_t)(piece0[s] + k * ppt + i)) =
                    make_int4(s, r0 + 16 * i,
                              min(16, rows - 16 * i) | (rows << 8) | (contiguous << 16) | (e.rank << 17),
                              __float_as_int(e.scale));
        }
    }

    // ---- 5. last block: header, -1 in unused entries ---------------------------------------------
    if (blockIdx.x != gridDim.x - 1) return;
    if (tid == 0) {
        const int32_t n_invalid = n_invalid_s;
        meta[H_T] = T;
        meta[H_NACTIVE] = n_active;
        meta[H_NINVALID] = n_invalid;
        meta[H_NSEG] = n_seg;
        meta[H_NTILE] = n_tile;
        meta[H_TILE_M] = tile_m;
        meta[H_LONG_MIN] = long_min;
        meta[H_NSLOTS] = N;
        meta[H_CAP_SEG] = L.cap_seg;
        meta[H_CAP_TILE] = L.cap_tile;
        meta[H_NPIECE] = n_piece;
        for (int i = H_NPIECE + 1; i < META_HEADER_WORDS; ++i) meta[i] = 0;
        meta[L.seg_start + n_seg] = n_active;
        if (n_invalid) atomicAdd(&pool.status[STATUS_INVALID_TOKENS], n_invalid);
    }
    for (int32_t i = n_seg + tid; i < L.cap_seg; i += SEGC_THREADS) {
        meta[L.seg_slot + i] = -1;
        meta[L.seg_rank + i] = -1;
        meta[L.seg_flags + i] = -1;
    }
    for (int32_t i = n_seg + 1 + tid; i <= L.cap_seg; i += SEGC_THREADS) meta[L.seg_start + i] = -1;
    for (int32_t i = n_tile + tid; i < L.cap_tile; i += SEGC_THREADS) {
        meta[L.tile_seg + i] = -1;
        meta[L.tile_row0 + i] = -1;
        meta[L.tile_rows + i] = -1;
        meta[L.tile_flags + i] = -1;
        *reinterpret_cast<int4 *>(meta + L.tile_desc + 4 * (int64_t)i) = make_int4(-1, 0, 0, 0);
    }
}

lora_status_t launch_build_segments(lora_pool_t *pool, const int32_t *slot_idx_dev, int32_t T,
                                    int32_t tile_m, int32_t long_min, void *meta_dev,
                                    cudaStream_t stream) {
    const int32_t N = pool->num_slots;
    // long batches: the chunked kernel, when its tables fit in shared memory
    if (T >= 1024 && pool->tuning[7] != 1) {
        int32_t CH = ((T + 63) / 64 + 31) & ~31;   // about 64 chunks, multiples of 32 tokens
        if (CH < 128) CH = 128;
        const int32_t C = (T + CH - 1) / CH;
        const MetaLayout L = meta_layout(T, N, tile_m);
        const size_t words = 6 * (size_t)N + (size_t)T + (size_t)C * (N + 1) + 2 * (size_t)L.cap_tile;
        if (words * sizeof(int32_t) <= 200 * 1024) {
            const size_t smem = words * sizeof(int32_t);
            const bool wide = T >= 8192;
            size_t &attr_chunked = wide ? pool->seg_attr_chunked_wide : pool->seg_attr_chunked;
            if (attr_chunked == 0) attr_chunked = 48 * 1024;
            if (smem > attr_chunked) {
                cudaError_t e = wide ? cudaFuncSetAttribute(build_segments_chunked_kernel<1024>,
                                                            cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)
                                     : cudaFuncSetAttribute(build_segments_chunked_kernel<256>,
                                                            cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
                if (e != cudaSuccess) return cuda_fail(e);
                attr_chunked = smem;
            }
            // every block builds the tables; the blocks share the writes (chunks of perm, slots)
            const int warps = wide ? 32 : 8;
            int grid = (N + warps - 1) / warps;
            if (grid < (C + 7) / 8) grid = (C + 7) / 8;
            if (grid > pool->sm_count) grid = pool->sm_count;
            if (wide)
                build_segments_chunked_kernel<1024><<<grid, 1024, smem, stream>>>(
                    pool->view(), slot_idx_dev, T, tile_m, long_min, (int32_t *)meta_dev, CH, C);
            else
                build_segments_chunked_kernel<256><<<grid, 256, smem, stream>>>(
                    pool->view(), slot_idx_dev, T, tile_m, long_min, (int32_t *)meta_dev, CH, C);
            return count_launch();
        }
    }
    int grid = (N + SEG_WARPS - 1) / SEG_WARPS;
    if (grid > 2 * pool->sm_count) grid = 2 * pool->sm_count;
    if (grid < 1) grid = 1;
    // the token list is copied to shared memory when it fits beside the per-slot arrays
    const size_t fixed = 6 * (size_t)N + 2 * (size_t)meta_layout(T, N, tile_m).cap_tile;
    const int32_t staged = sizeof(int32_t) * (fixed + (size_t)T) <= 200 * 1024 ? 1 : 0;
    const size_t smem = sizeof(int32_t) * (fixed + (staged ? (size_t)T : 0));
    size_t &attr_smem = pool->seg_attr_smem;
    if (attr_smem == 0) attr_smem = 48 * 1024;
    if (smem > attr_smem) {
        cudaError_t e = cudaFuncSetAttribute(build_segments_kernel,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return cuda_fail(e);
        attr_smem = smem;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid, 1, 1);
    cfg.blockDim = dim3(SEG_THREADS, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    // Programmatic dependent launch: the blocks may become resident while the kernel before them on
    // the stream drains (they read nothing before griddepcontrol.wait); tuning key 2 = 2: never.
    cfg.numAttrs = pool->tuning[2] != 2 ? 1 : 0;
    LORA_CUDA_TRY(cudaLaunchKernelEx(&cfg, build_segments_kernel, pool->view(), slot_idx_dev, T,
                                     tile_m, long_min, (int32_t *)meta_dev, staged));
    return count_launch();
}

}  // namespace lora

using namespace lora;

extern "C" {

lora_status_t lora_segments_bytes(int32_t T, int32_t num_slots, int32_t tile_m, size_t *bytes) {
    if (!bytes) return LORA_ERR_INVALID_ARG;
    if (T < 0 || num_slots < 1 || tile_m < 1) return LORA_ERR_SHAPE;
    *bytes = (size_t)meta_layout(T, num_slots, tile_m).words * sizeof(int32_t);
    return LORA_OK;
}

lora_status_t lora_build_segments(lora_pool_t *pool, const int32_t *slot_idx_dev, int32_t T,
                                  int32_t tile_m, int32_t long_min, void *meta_dev,
                                  size_t meta_bytes, void *stream) {
    if (!pool || !meta_dev || (T > 0 && !slot_idx_dev)) return LORA_ERR_INVALID_ARG;
    if (T < 0 || tile_m < 1 || tile_m > 128 || long_min < 1) return LORA_ERR_SHAPE;
    if ((uintptr_t)meta_dev & 15) return LORA_ERR_INVALID_ARG;
    if (meta_bytes < (size_t)meta_layout(T, pool->num_slots, tile_m).words * sizeof(int32_t))
        return LORA_ERR_BUFFER_TOO_SMALL;
    DeviceGuard guard(pool->device);
    if (!guard.ok) return cuda_fail(cudaErrorInvalidDevice);
    lora_status_t s = launch_build_segments(pool, slot_idx_dev, T, tile_m, long_min, meta_dev,
                                            (cudaStream_t)stream);
    // batches that lora_sgmv_apply gives to its tensor-core kernels: the list of their tiles, once
    // per build (tuning key 4 is read here)
    const bool with_list = s == LORA_OK && tc_path_wanted(pool, T, tile_m);
    if (with_list) s = launch_tc_worklist(pool, T, tile_m, meta_dev, (cudaStream_t)stream);
    if (s == LORA_OK) pool->remember_meta(meta_dev, T, tile_m, long_min, with_list);
    return s;
}

}  // extern "C"
