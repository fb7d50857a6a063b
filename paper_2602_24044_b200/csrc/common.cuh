// Shared declarations of the lora_b200 CUDA library (host handle, device views, metadata layout).
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>
#include <vector>

#include "lora_b200.h"

namespace lora {

// ---------------------------------------------------------------------------------------------
// error plumbing
// ---------------------------------------------------------------------------------------------
extern thread_local int32_t g_last_cuda_error;
extern std::atomic<int64_t> g_launch_count;

inline lora_status_t cuda_fail(cudaError_t e) {
    g_last_cuda_error = (int32_t)e;
    return LORA_ERR_CUDA;
}
#define LORA_CUDA_TRY(expr)                                   \
    do {                                                      \
        cudaError_t _e = (expr);                              \
        if (_e != cudaSuccess) return ::lora::cuda_fail(_e);  \
    } while (0)

inline lora_status_t count_launch() {
    g_launch_count.fetch_add(1, std::memory_order_relaxed);
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? LORA_OK : cuda_fail(e);
}

// ---------------------------------------------------------------------------------------------
// device-side pool description
// ---------------------------------------------------------------------------------------------
struct SlotEntry {       // one per slot, in the pool's control block
    int32_t rank;        // true rank, 0 when empty
    float scale;         // s_i
    int32_t loaded;      // 1 = occupied and complete
    int32_t reserved;
};

enum { STATUS_INVALID_TOKENS = 0, STATUS_TIMEOUTS = 1, STATUS_WORDS = 4 };

struct PoolView {                  // passed to kernels by value
    const __nv_bfloat16 *weights;  // slot 0 of the weight region
    int64_t slot_stride;           // elements between consecutive slots
    const SlotEntry *table;        // [num_slots]
    int32_t *status;               // [STATUS_WORDS]
    int32_t num_slots;
    int32_t r_max;
};

struct TargetView {    // one adapted projection inside a slot
    int64_t off_a;     // element offset of A [r_max, d_in] inside a slot
    int64_t off_b;     // element offset of B [r_max, d_out]
    int32_t d_in;
    int32_t d_out;
};

// ---------------------------------------------------------------------------------------------
// segment metadata layout (int32 words)
// ---------------------------------------------------------------------------------------------
enum { META_HEADER_WORDS = 16 };
enum { H_T = 0, H_NACTIVE = 1, H_NINVALID = 2, H_NSEG = 3, H_NTILE = 4, H_TILE_M = 5,
       H_LONG_MIN = 6, H_NSLOTS = 7, H_CAP_SEG = 8, H_CAP_TILE = 9, H_NPIECE = 10 /* private */ };

struct MetaLayout {
    int32_t cap_seg, cap_tile;
    int64_t perm, seg_slot, seg_start, seg_rank, seg_flags, tile_seg, tile_row0, tile_rows,
        tile_flags, tile_desc, unit_desc, unit_perm, long_list, words;
    int32_t cap_unit;
};

__host__ __device__ inline MetaLayout meta_layout(int32_t T, int32_t num_slots, int32_t tile_m) {
    MetaLayout L;
    L.cap_seg = T < num_slots ? T : num_slots;
    L.cap_tile = L.cap_seg + T / tile_m;
    int64_t o = META_HEADER_WORDS;
    L.perm = o;       o += T;
    L.seg_slot = o;   o += L.cap_seg;
    L.seg_start = o;  o += L.cap_seg + 1;
    L.seg_rank = o;   o += L.cap_seg;
    L.seg_flags = o;  o += L.cap_seg;
    L.tile_seg = o;   o += L.cap_tile;
    L.tile_row0 = o;  o += L.cap_tile;
    L.tile_rows = o;  o += L.cap_tile;
    L.tile_flags = o; o += L.cap_tile;
    o = (o + 3) & ~(int64_t)3;            // library-private part, 16-byte aligned records
    L.tile_desc = o;  o += 4 * (int64_t)L.cap_tile;   // {slot, row0, rows | rank << 16, scale bits}
    // Units of the fused kernel: every tile cut into pieces of at most 16 rows, in tile order
    // (a tile of tile_m <= 16 rows is one unit).  Header word H_NPIECE counts them.  One record
    // per unit {slot, position in perm, rows | tile rows << 8 | consecutive ids << 16 | rank << 17,
    // scale bits} and the unit's token ids at unit * 16.
    L.cap_unit = L.cap_tile * ((tile_m + 15) / 16);
    L.unit_desc = o;  o += 4 * (int64_t)L.cap_unit;
    L.unit_perm = o;  o += 16 * (int64_t)L.cap_unit;
    // Tiles for the tensor-core kernels of lora_sgmv_apply (runs of consecutive tokens), in tile
    // order: [0] = their number, then their tile numbers.  Written after the build when the batch
    // qualifies for those kernels, else left alone.
    L.long_list = o;  o += ((int64_t)L.cap_tile + 1 + 3) & ~(int64_t)3;
    L.words = o;
    return L;
}

// Kernel attributes (dynamic shared-memory limits) and occupancy figures are per device: the
// launchers keep what they have set or asked in small tables indexed by the device ordinal.
constexpr int DEVICE_TABLE = 64;
inline int device_index(int device) { return device >= 0 && device < DEVICE_TABLE ? device : 0; }

// rank bucket a slot's kernels are specialised for: 8, 16, 32 or 64
__host__ __device__ inline int32_t rank_bucket(int32_t r) {
    return r <= 8 ? 8 : r <= 16 ? 16 : r <= 32 ? 32 : 64;
}
__host__ __device__ inline int32_t round_up8(int32_t r) { return (r + 7) & ~7; }

}  // namespace lora

// ---------------------------------------------------------------------------------------------
// host handle
// ---------------------------------------------------------------------------------------------
struct lora_pool {
    int32_t device = 0, num_slots = 0, r_max = 0, num_targets = 0;
    std::vector<lora_target_t> targets;
    std::vector<lora::TargetView> target_views;
    char *base = nullptr;               // device_buf
    size_t bytes = 0;
    int32_t *status_dev = nullptr;      // [STATUS_WORDS]
    lora::SlotEntry *table_dev = nullptr;
    __nv_bfloat16 *staging_dev = nullptr;   // r_max * max_d_in elements, transpose input
    size_t staging_elems = 0;
    __nv_bfloat16 *weights_dev = nullptr;
    int64_t slot_stride = 0;            // elements
    std::vector<lora::SlotEntry> table_host;   // as of the last load / evict call
    std::vector<cudaEvent_t> ready;     // per slot, created on first load
    cudaEvent_t fence = nullptr;        // compute -> load ordering
    int32_t sm_count = 148;
    uint32_t bucket_mask = 0;           // rank buckets (8/16/32/64 -> bits 0..3) ever loaded into a slot
    int32_t tuning[16] = {0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0};
    // Tensor maps of the fused kernel in the pool's device buffer, written at creation: per
    // target 8 for A and 8 for B (one per number of rank rows 8, 16, .. 64 a tile load fetches).
    CUtensorMap *maps_dev = nullptr;
    // lora_sgmv_apply runs the tiles its tensor-core kernels leave over beside those kernels
    cudaStream_t side_stream = nullptr;
    cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
    // What the fused kernel's launcher has set or asked for this pool's device (dynamic
    // shared-memory limit, resident clusters), per kernel variant; part of the handle, so pools
    // used from different threads share nothing.
    struct FusedLaunchCache {
        int32_t attr_smem = 0, occ_smem = 0, occ_c = 0, occ_clusters = 0;
    };
    FusedLaunchCache fused_cache[3];
    // kernel attributes the other launchers have set for this pool's device
    bool twophase_attr_done = false;
    bool tc_attr_done[3] = {false, false, false};   // rank buckets 16, 32, 64
    size_t seg_attr_smem = 0, seg_attr_chunked = 0;
    size_t seg_attr_chunked_wide = 0;

    // Shapes of the metadata tables built through this handle (the table itself lives on the
    // device; apply calls need T and tile_m on the host to size their grids).
    struct MetaRecord {
        const void *ptr;
        int32_t T, tile_m, long_min;
        bool fresh;   // built, and no apply has been queued behind the build yet
        bool has_list;   // the list of long tiles was written behind the build
    };
    std::vector<MetaRecord> metas;
    void remember_meta(const void *ptr, int32_t T, int32_t tile_m, int32_t long_min, bool has_list) {
        for (MetaRecord &m : metas)
            if (m.ptr == ptr) {
                m.T = T; m.tile_m = tile_m; m.long_min = long_min; m.fresh = true; m.has_list = has_list;
                return;
            }
        if (metas.size() >= 256) metas.erase(metas.begin());
        metas.push_back({ptr, T, tile_m, long_min, true, has_list});
    }
    bool meta_has_list(const void *ptr) const {
        for (const MetaRecord &m : metas)
            if (m.ptr == ptr) return m.has_list;
        return false;
    }
    bool find_meta(const void *ptr, int32_t T, int32_t *tile_m) const {
        for (const MetaRecord &m : metas)
            if (m.ptr == ptr && m.T == T) {
                *tile_m = m.tile_m;
                return true;
            }
        return false;
    }

    // True once for a table after each build: the first kernel that reads the table must be
    // fully ordered behind the build; later ones may read it before their predecessor has finished.
    bool take_fresh(const void *ptr) {
        for (MetaRecord &m : metas)
            if (m.ptr == ptr) {
                const bool f = m.fresh;
                m.fresh = false;
                return f;
            }
        return true;
    }

    lora::PoolView view() const {
        lora::PoolView v;
        v.weights = weights_dev;
        v.slot_stride = slot_stride;
        v.table = table_dev;
        v.status = status_dev;
        v.num_slots = num_slots;
        v.r_max = r_max;
        return v;
    }
};

namespace lora {
// RAII-free device guard: remembers the current device, switches, restores in the destructor.
struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
        want = dev;
    }
    ~DeviceGuard() {
        if (prev >= 0 && prev != want) cudaSetDevice(prev);
    }
    int want = -1;
};
}  // namespace lora
