// Which adapter lives in which slot: the host-side bookkeeping of the adapter cache (paper
// Section 1: adapters are swapped between CPU and GPU memory according to their usage; Section
// 2.2: at most A_max adapters are loaded at once; Section 5: the adapter-cache stage of a step
// loads the adapters the scheduled batch needs).  Pure host code: it decides, the pool's
// load / evict calls move the bytes.
//
// Victim choice is least-recently-used among the slots that are neither pinned nor needed by the
// batch being admitted; empty slots are taken first, lowest index first.  "Recently used" is a
// logical clock advanced by every touch, so the order is a deterministic function of the call
// sequence.
#include <new>
#include <unordered_map>
#include <vector>

#include "common.cuh"

struct lora_policy {
    struct Slot {
        int64_t adapter = -1;   // -1: empty
        int64_t stamp = 0;      // logical time of the last use
        int32_t pins = 0;       // in-flight batches that reference the slot
    };
    std::vector<Slot> slots;
    std::unordered_map<int64_t, int32_t> where;   // adapter id -> slot
    int64_t clock = 0;
    int64_t hits = 0, misses = 0, evictions = 0;
};

namespace lora {

// The slot to (re)use next, ignoring slots whose `skip` flag is set: the lowest empty slot, else
// the unpinned slot with the oldest stamp (ties: lowest index).  -1 when there is none.
static int32_t pick_victim(const lora_policy &p, const std::vector<uint8_t> *skip) {
    int32_t best = -1;
    for (int32_t s = 0; s < (int32_t)p.slots.size(); ++s) {
        const lora_policy::Slot &e = p.slots[s];
        if (e.pins > 0 || (skip && (*skip)[s])) continue;
        if (e.adapter < 0) return s;
        if (best < 0 || e.stamp < p.slots[best].stamp) best = s;
    }
    return best;
}

}  // namespace lora

using namespace lora;

extern "C" {

lora_status_t lora_policy_create(int32_t num_slots, lora_policy_t **out) {
    if (!out) return LORA_ERR_INVALID_ARG;
    *out = nullptr;
    if (num_slots < 1 || num_slots > 8192) return LORA_ERR_INVALID_ARG;
    lora_policy_t *p = new (std::nothrow) lora_policy();
    if (!p) return LORA_ERR_INVALID_ARG;
    p->slots.resize(num_slots);
    *out = p;
    return LORA_OK;
}

lora_status_t lora_policy_destroy(lora_policy_t *p) {
    if (!p) return LORA_ERR_INVALID_ARG;
    delete p;
    return LORA_OK;
}

lora_status_t lora_policy_lookup(const lora_policy_t *p, int64_t adapter, int32_t *slot_out) {
    if (!p || !slot_out || adapter < 0) return LORA_ERR_INVALID_ARG;
    auto it = p->where.find(adapter);
    *slot_out = it == p->where.end() ? -1 : it->second;
    return LORA_OK;
}

lora_status_t lora_policy_slot(const lora_policy_t *p, int32_t slot, int64_t *adapter_out,
                               int32_t *pins_out) {
    if (!p) return LORA_ERR_INVALID_ARG;
    if (slot < 0 || slot >= (int32_t)p->slots.size()) return LORA_ERR_SLOT_RANGE;
    if (adapter_out) *adapter_out = p->slots[slot].adapter;
    if (pins_out) *pins_out = p->slots[slot].pins;
    return LORA_OK;
}

lora_status_t lora_policy_touch(lora_policy_t *p, int32_t slot) {
    if (!p) return LORA_ERR_INVALID_ARG;
    if (slot < 0 || slot >= (int32_t)p->slots.size()) return LORA_ERR_SLOT_RANGE;
    if (p->slots[slot].adapter < 0) return LORA_ERR_NOT_LOADED;
    p->slots[slot].stamp = ++p->clock;
    return LORA_OK;
}

lora_status_t lora_policy_pin(lora_policy_t *p, const int32_t *slots, int32_t n) {
    if (!p || n < 0 || (n > 0 && !slots)) return LORA_ERR_INVALID_ARG;
    for (int32_t i = 0; i < n; ++i) {
        if (slots[i] < 0 || slots[i] >= (int32_t)p->slots.size()) return LORA_ERR_SLOT_RANGE;
        if (p->slots[slots[i]].adapter < 0) return LORA_ERR_NOT_LOADED;
    }
    for (int32_t i = 0; i < n; ++i) ++p->slots[slots[i]].pins;
    return LORA_OK;
}

lora_status_t lora_policy_unpin(lora_policy_t *p, const int32_t *slots, int32_t n) {
    if (!p || n < 0 || (n > 0 && !slots)) return LORA_ERR_INVALID_ARG;
    // all or nothing: count how often each slot is named first
    std::vector<int32_t> need(p->slots.size(), 0);
    for (int32_t i = 0; i < n; ++i) {
        if (slots[i] < 0 || slots[i] >= (int32_t)p->slots.size()) return LORA_ERR_SLOT_RANGE;
        if (++need[slots[i]] > p->slots[slots[i]].pins) return LORA_ERR_INVALID_ARG;
    }
    for (int32_t i = 0; i < n; ++i) --p->slots[slots[i]].pins;
    return LORA_OK;
}

lora_status_t lora_policy_choose_victim(const lora_policy_t *p, int32_t *slot_out,
                                        int64_t *evicted_out) {
    if (!p || !slot_out) return LORA_ERR_INVALID_ARG;
    const int32_t v = pick_victim(*p, nullptr);
    if (v < 0) return LORA_ERR_BUSY;
    *slot_out = v;
    if (evicted_out) *evicted_out = p->slots[v].adapter;
    return LORA_OK;
}

lora_status_t lora_policy_assign(lora_policy_t *p, int32_t slot, int64_t adapter) {
    if (!p || adapter < 0) return LORA_ERR_INVALID_ARG;
    if (slot < 0 || slot >= (int32_t)p->slots.size()) return LORA_ERR_SLOT_RANGE;
    lora_policy::Slot &e = p->slots[slot];
    if (e.pins > 0) return LORA_ERR_BUSY;
    auto it = p->where.find(adapter);
    if (it != p->where.end() && it->second != slot) return LORA_ERR_INVALID_ARG;   // resident elsewhere
    if (e.adapter >= 0 && e.adapter != adapter) {
        p->where.erase(e.adapter);
        ++p->evictions;
    }
    e.adapter = adapter;
    e.stamp = ++p->clock;
    p->where[adapter] = slot;
    return LORA_OK;
}

lora_status_t lora_policy_release(lora_policy_t *p, int32_t slot) {
    if (!p) return LORA_ERR_INVALID_ARG;
    if (slot < 0 || slot >= (int32_t)p->slots.size()) return LORA_ERR_SLOT_RANGE;
    lora_policy::Slot &e = p->slots[slot];
    if (e.adapter < 0) return LORA_ERR_NOT_LOADED;
    if (e.pins > 0) return LORA_ERR_BUSY;
    p->where.erase(e.adapter);
    e.adapter = -1;
    e.stamp = 0;
    return LORA_OK;
}

lora_status_t lora_policy_admit(lora_policy_t *p, const int64_t *adapters, int32_t n,
                                int32_t *slot_idx_out, int32_t *miss_slots, int64_t *miss_adapters,
                                int32_t miss_cap, int32_t *n_miss_out) {
    if (!p || n < 0 || (n > 0 && (!adapters || !slot_idx_out)) || !n_miss_out || miss_cap < 0 ||
        (miss_cap > 0 && (!miss_slots || !miss_adapters)))
        return LORA_ERR_INVALID_ARG;
    const int32_t N = (int32_t)p->slots.size();
    // pass 1 (no state change): which slots the batch already holds, which adapters are missing
    std::vector<uint8_t> used(N, 0);
    std::vector<int64_t> missing;   // distinct, in order of first appearance
    std::unordered_map<int64_t, int32_t> miss_pos;
    for (int32_t i = 0; i < n; ++i) {
        const int64_t a = adapters[i];
        if (a < 0) continue;
        auto it = p->where.find(a);
        if (it != p->where.end()) used[it->second] = 1;
        else if (miss_pos.emplace(a, (int32_t)missing.size()).second) missing.push_back(a);
    }
    if ((int32_t)missing.size() > miss_cap) return LORA_ERR_BUFFER_TOO_SMALL;
    // victims for the missing adapters, chosen on a scratch copy so that failure changes nothing
    std::vector<int32_t> victims;
    {
        std::vector<uint8_t> skip = used;
        for (size_t k = 0; k < missing.size(); ++k) {
            const int32_t v = pick_victim(*p, &skip);
            if (v < 0) return LORA_ERR_BUSY;   // more distinct adapters than free or evictable slots
            skip[v] = 1;
            victims.push_back(v);
        }
    }
    // pass 2: commit
    for (size_t k = 0; k < missing.size(); ++k) {
        lora_policy::Slot &e = p->slots[victims[k]];
        if (e.adapter >= 0) {
            p->where.erase(e.adapter);
            ++p->evictions;
        }
        e.adapter = missing[k];
        p->where[missing[k]] = victims[k];
        miss_slots[k] = victims[k];
        miss_adapters[k] = missing[k];
    }
    p->misses += (int64_t)missing.size();
    std::vector<uint8_t> counted(N, 0);
    for (int32_t i = 0; i < n; ++i) {
        const int64_t a = adapters[i];
        if (a < 0) {
            slot_idx_out[i] = -1;
            continue;
        }
        const int32_t s = p->where[a];
        slot_idx_out[i] = s;
        p->slots[s].stamp = ++p->clock;
        if (!counted[s]) {
            counted[s] = 1;
            if (miss_pos.find(a) == miss_pos.end()) ++p->hits;
        }
    }
    *n_miss_out = (int32_t)missing.size();
    return LORA_OK;
}

lora_status_t lora_policy_stats(const lora_policy_t *p, int64_t *hits, int64_t *misses,
                                int64_t *evictions) {
    if (!p) return LORA_ERR_INVALID_ARG;
    if (hits) *hits = p->hits;
    if (misses) *misses = p->misses;
    if (evictions) *evictions = p->evictions;
    return LORA_OK;
}

lora_status_t lora_pool_plan(size_t bytes_budget, const lora_target_t *targets, int32_t num_targets,
                             int32_t r_max, int32_t *num_slots_out, size_t *bytes_per_slot_out) {
    if (!targets || !num_slots_out || num_targets < 1) return LORA_ERR_INVALID_ARG;
    lora_pool_desc_t d = {};
    d.num_slots = 1;
    d.r_max = r_max;
    d.num_targets = num_targets;
    d.targets = targets;
    size_t b1 = 0, b2 = 0;
    lora_status_t s = lora_pool_bytes(&d, &b1);
    if (s != LORA_OK) return s;
    d.num_slots = 2;
    if ((s = lora_pool_bytes(&d, &b2)) != LORA_OK) return s;
    const size_t per_slot = b2 - b1;   // weights of one slot; the rest is the control block
    if (bytes_per_slot_out) *bytes_per_slot_out = per_slot;
    // largest N with pool_bytes(N) <= budget; the control block grows by 16 bytes per slot in
    // 256-byte steps, so settle the last few slots by asking
    int64_t n = bytes_budget < b1 ? 0 : 1 + (int64_t)((bytes_budget - b1) / (per_slot + 16));
    if (n > 8192) n = 8192;
    while (n < 8192) {
        d.num_slots = (int32_t)n + 1;
        size_t b = 0;
        if (lora_pool_bytes(&d, &b) != LORA_OK || b > bytes_budget) break;
        ++n;
    }
    while (n > 0) {
        d.num_slots = (int32_t)n;
        size_t b = 0;
        if (lora_pool_bytes(&d, &b) == LORA_OK && b <= bytes_budget) break;
        --n;
    }
    *num_slots_out = (int32_t)n;
    return n > 0 ? LORA_OK : LORA_ERR_BUFFER_TOO_SMALL;
}

}  // extern "C"
