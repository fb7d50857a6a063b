/*
 * CPU oracle for the unmerged multi-adapter LoRA forward.  TEST INFRASTRUCTURE:
 * only the test-suite, the smoke check and the benchmark's CPU-baseline leg may
 * build or call this file.  It shares no code with the CUDA library and is
 * never used to produce a product result.
 *
 * What it computes (paper Section 2.2: a LoRA adapter is two low-rank matrices
 * whose activations are added to the output of the backbone layer they adapt;
 * Section 1: adapters stay unmerged so many of them share one backbone; several
 * adapters are served inside one batch):
 *
 *     y[t, :] = y_base[t, :] + s_i * (x[t, :] . A_i) . B_i ,   i = slot_idx[t]
 *
 * with A_i of shape [d_in, r_i] and B_i of shape [r_i, d_out], in fp64, as the
 * plain definition: no blocking, no reordering, reductions in ascending index
 * order.  Tokens whose slot id is -1, out of range or names an empty slot get
 * y = y_base.
 *
 * The integer part groups the tokens of a batch by adapter slot (a stable
 * group-by) and cuts the groups into row tiles; every output is uniquely
 * defined, so it is written as the definition as well.
 *
 * Pins (tests/test_oracle_pins.py): merged-weight equivalence x.(W + s.A.B),
 * B = 0, rank-1 closed form, batch-permutation invariance, linearity in s,
 * additivity over a rank split, single-adapter reduction to two library
 * matmuls, exact small-integer cases, a hand-worked example stored under
 * tests/golden/.  The paper prints no worked numeric example of this
 * computation: parity is unpinned by paper-printed values and rests on those
 * closed forms.
 */
#include <stdint.h>
#include <stdlib.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* One token: v = x_t . A_i (d ascending), y_t = y_base_t + s_i * (v . B_i) (k ascending). */
static void oracle_token(int32_t d_in, int32_t d_out, int32_t r,
                         const double *xt, const double *ybt,
                         const double *A, const double *B, double s,
                         double *v, double *yt)
{
    for (int32_t k = 0; k < r; ++k) {
        double acc = 0.0;
        for (int32_t d = 0; d < d_in; ++d)
            acc += xt[d] * A[(int64_t)d * r + k];
        v[k] = acc;
    }
    for (int32_t j = 0; j < d_out; ++j) {
        double acc = 0.0;
        for (int32_t k = 0; k < r; ++k)
            acc += v[k] * B[(int64_t)k * d_out + j];
        yt[j] = ybt[j] + s * acc;
    }
}

/*
 * x      [T, ldx]   fp64 (bf16 inputs widened exactly by the caller)
 * y_base [T, ldyb]  fp64
 * A[i]   [d_in, rank[i]] row-major, B[i] [rank[i], d_out] row-major (NULL allowed for
 *        slots that are not loaded)
 * y      [T, ldy]   fp64 out (never rounded)
 * returns the number of invalid tokens (slot id not -1 and not an occupied slot), or -1 on
 * a bad argument.
 */
int64_t lora_oracle_apply(int32_t T, int32_t d_in, int32_t d_out, int32_t num_slots,
                          const double *x, int64_t ldx,
                          const double *y_base, int64_t ldyb,
                          const int32_t *slot_idx,
                          const double *const *A, const double *const *B,
                          const int32_t *rank, const double *scale, const int32_t *loaded,
                          double *y, int64_t ldy, int32_t num_threads)
{
    if (T < 0 || d_in < 1 || d_out < 1 || num_slots < 0) return -1;
    int32_t r_cap = 1;
    for (int32_t i = 0; i < num_slots; ++i)
        if (rank[i] > r_cap) r_cap = rank[i];
    int64_t n_invalid = 0;
#ifdef _OPENMP
    if (num_threads < 1) num_threads = 1;
#pragma omp parallel num_threads(num_threads) reduction(+ : n_invalid)
#endif
    {
        double *v = (double *)malloc(sizeof(double) * (size_t)r_cap);
#ifdef _OPENMP
#pragma omp for schedule(dynamic, 1)
#endif
        for (int32_t t = 0; t < T; ++t) {
            const int32_t i = slot_idx[t];
            const double *xt = x + (int64_t)t * ldx;
            const double *ybt = y_base + (int64_t)t * ldyb;
            double *yt = y + (int64_t)t * ldy;
            if (i < 0 || i >= num_slots || !loaded[i]) {
                if (i != -1) n_invalid += 1;
                for (int32_t j = 0; j < d_out; ++j) yt[j] = ybt[j];
                continue;
            }
            oracle_token(d_in, d_out, rank[i], xt, ybt, A[i], B[i], scale[i], v, yt);
        }
        free(v);
    }
    (void)num_threads;
    return n_invalid;
}

int32_t lora_oracle_max_threads(void)
{
#ifdef _OPENMP
    return (int32_t)omp_get_max_threads();
#else
    return 1;
#endif
}

/*
 * Segment metadata, step by step:
 *  1. token t is active iff 0 <= slot_idx[t] < num_slots and loaded[slot_idx[t]];
 *     invalid iff not active and slot_idx[t] != -1.
 *  2. perm[0:n_active] = active tokens ordered by (slot, t) ascending;
 *     perm[n_active:T] = the other tokens, t ascending.
 *  3. segments = maximal runs of one slot in perm[0:n_active]:
 *     seg_slot (strictly ascending), seg_start (n_seg + 1 entries), seg_rank.
 *  4. seg_flags bit0: rows of the segment are consecutive token ids;
 *     bit1: segment length >= long_min.
 *  5. tiles: each segment cut into pieces of at most tile_m rows, in order:
 *     (tile_seg, tile_row0, tile_rows).
 *  6. header = {T, n_active, n_invalid, n_seg, n_tile}; unused array entries = -1.
 * Capacities: perm T; seg arrays cap_seg (seg_start cap_seg + 1); tile arrays cap_tile.
 * Returns 0, or -1 on a bad argument or when a capacity is too small.
 */
int32_t lora_oracle_build_segments(int32_t T, int32_t num_slots,
                                   const int32_t *slot_idx, const int32_t *loaded,
                                   const int32_t *rank, int32_t tile_m, int32_t long_min,
                                   int32_t cap_seg, int32_t cap_tile,
                                   int32_t *header /*[5]*/, int32_t *perm,
                                   int32_t *seg_slot, int32_t *seg_start, int32_t *seg_rank,
                                   int32_t *seg_flags,
                                   int32_t *tile_seg, int32_t *tile_row0, int32_t *tile_rows)
{
    if (T < 0 || num_slots < 0 || tile_m < 1 || long_min < 1) return -1;
    for (int32_t t = 0; t < T; ++t) perm[t] = -1;
    for (int32_t s = 0; s < cap_seg; ++s)
        seg_slot[s] = seg_rank[s] = seg_flags[s] = -1;
    for (int32_t s = 0; s <= cap_seg; ++s) seg_start[s] = -1;
    for (int32_t k = 0; k < cap_tile; ++k)
        tile_seg[k] = tile_row0[k] = tile_rows[k] = -1;

    int32_t n_active = 0, n_invalid = 0, n_seg = 0, n_tile = 0;
    /* steps 1-3: for each slot in ascending order, take its tokens in ascending order */
    for (int32_t i = 0; i < num_slots; ++i) {
        if (!loaded[i]) continue;
        int32_t first = n_active;
        for (int32_t t = 0; t < T; ++t)
            if (slot_idx[t] == i) perm[n_active++] = t;
        if (n_active > first) {
            if (n_seg >= cap_seg) return -1;
            seg_slot[n_seg] = i;
            seg_start[n_seg] = first;
            seg_rank[n_seg] = rank[i];
            ++n_seg;
        }
    }
    seg_start[n_seg] = n_active;   /* cap_seg + 1 entries exist */
    /* the inactive tail, and the invalid count */
    int32_t tail = n_active;
    for (int32_t t = 0; t < T; ++t) {
        int32_t i = slot_idx[t];
        int active = (i >= 0 && i < num_slots && loaded[i]);
        if (!active) {
            perm[tail++] = t;
            if (i != -1) ++n_invalid;
        }
    }
    /* step 4 */
    for (int32_t s = 0; s < n_seg; ++s) {
        int32_t contiguous = 1;
        for (int32_t j = seg_start[s]; j + 1 < seg_start[s + 1]; ++j)
            if (perm[j + 1] != perm[j] + 1) contiguous = 0;
        int32_t len = seg_start[s + 1] - seg_start[s];
        seg_flags[s] = contiguous | ((len >= long_min) ? 2 : 0);
    }
    /* step 5 */
    for (int32_t s = 0; s < n_seg; ++s) {
        for (int32_t r0 = seg_start[s]; r0 < seg_start[s + 1]; r0 += tile_m) {
            if (n_tile >= cap_tile) return -1;
            int32_t rows = seg_start[s + 1] - r0;
            if (rows > tile_m) rows = tile_m;
            tile_seg[n_tile] = s;
            tile_row0[n_tile] = r0;
            tile_rows[n_tile] = rows;
            ++n_tile;
        }
    }
    header[0] = T;
    header[1] = n_active;
    header[2] = n_invalid;
    header[3] = n_seg;
    header[4] = n_tile;
    return 0;
}
