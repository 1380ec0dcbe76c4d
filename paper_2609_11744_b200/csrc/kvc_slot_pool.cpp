// Slot pool with the paper's scheduling rules for one shared staging pool (Sec. 6.4, 6.5), host
// bookkeeping only:
//   * loads, stores and speculative preloads draw from the same fixed set of slots;
//   * a number of slots equal to the I/O depth is reserved for foreground work: a preload gets a
//     slot only while more than that many are free, and only a bounded number of preloads may be
//     in flight at once;
//   * identical keys (chunk hashes) share one slot with a reference count: a second preload of
//     the same prefix, or a later demand load, joins the operation already holding the slot
//     instead of issuing another read; a demand load that joins a preload "claims" it;
//   * a foreground request that finds no free slot may take over a retained (cache) slot, least
//     recently used first, or a staged preload nobody has claimed;
//   * an unclaimed preload still in flight can be cancelled to give its bandwidth to demand work;
//   * completed slots can be retained as a DRAM cache (LRU) instead of being freed.
// The ring in kvc_ring.cu orders slots FIFO and ties reuse to CUDA events; this pool decides WHO
// gets a slot.  The two are independent: a slot index here can name a ring-sized region anywhere.
#include <new>
#include <unordered_map>
#include <vector>

#include "kvc.h"

namespace {

enum State { FREE = 0, IN_FLIGHT = 1, STAGED = 2, RETAINED = 3 };

struct PSlot {
    State state = FREE;
    uint64_t key = 0;
    uint32_t refs = 0;
    bool speculative = false;  // acquired by a preload and not claimed by foreground work yet
    uint64_t stamp = 0;        // last use, for LRU among retained slots
};

}  // namespace

struct kvc_slot_pool {
    std::vector<PSlot> slots;
    std::unordered_map<uint64_t, uint32_t> by_key;
    uint32_t reserve, max_spec;
    bool retain;
    uint64_t clock;
    kvc_slot_pool_counters c;
};

namespace {

uint32_t count_free(const kvc_slot_pool *p)
{
    uint32_t n = 0;
    for (const PSlot &s : p->slots)
        n += s.state == FREE;
    return n;
}

uint32_t speculative_in_flight(const kvc_slot_pool *p)
{
    uint32_t n = 0;
    for (const PSlot &s : p->slots)
        n += s.state == IN_FLIGHT && s.speculative;
    return n;
}

void forget(kvc_slot_pool *p, PSlot &s)
{
    auto it = p->by_key.find(s.key);
    if (it != p->by_key.end() && &p->slots[it->second] == &s)
        p->by_key.erase(it);
    s = PSlot();
}

}  // namespace

extern "C" {

kvc_status kvc_slot_pool_create(uint32_t n_slots, uint32_t foreground_reserve, uint32_t max_speculative,
                                int retain_completed, kvc_slot_pool **out)
{
    if (!out)
        return KVC_ERR_INVALID_ARG;
    *out = nullptr;
    if (n_slots == 0 || foreground_reserve > n_slots)
        return KVC_ERR_INVALID_ARG;
    kvc_slot_pool *p = new (std::nothrow) kvc_slot_pool();
    if (!p)
        return KVC_ERR_NOMEM;
    try {
        p->slots.resize(n_slots);
    } catch (const std::bad_alloc &) {
        delete p;
        return KVC_ERR_NOMEM;
    }
    p->reserve = foreground_reserve;
    p->max_spec = max_speculative;
    p->retain = retain_completed != 0;
    p->clock = 0;
    p->c = kvc_slot_pool_counters();
    *out = p;
    return KVC_OK;
}

kvc_status kvc_slot_pool_destroy(kvc_slot_pool *p)
{
    if (!p)
        return KVC_ERR_INVALID_ARG;
    delete p;
    return KVC_OK;
}

kvc_status kvc_slot_pool_acquire(kvc_slot_pool *p, kvc_slot_class cls, uint64_t key, uint32_t *slot,
                                 int *joined)
{
    if (!p || !slot || !joined ||
        (cls != KVC_CLASS_DEMAND_LOAD && cls != KVC_CLASS_STORE && cls != KVC_CLASS_PRELOAD))
        return KVC_ERR_INVALID_ARG;
    const bool foreground = cls != KVC_CLASS_PRELOAD;
    try {
        // 1. somebody already holds this chunk: join it
        auto it = p->by_key.find(key);
        if (it != p->by_key.end()) {
            PSlot &s = p->slots[it->second];
            if (s.state == RETAINED)
                s.state = STAGED;       // a cache hit brings the slot back into use
            ++s.refs;
            s.stamp = ++p->clock;
            if (foreground && s.speculative) {
                s.speculative = false;  // a demand request claims the preload
                ++p->c.claims;
            }
            ++p->c.joins;
            *slot = it->second;
            *joined = 1;
            return KVC_OK;
        }
        // 2. a free slot, within the class's allowance
        const uint32_t nfree = count_free(p);
        if (!foreground) {
            if (nfree <= p->reserve || (p->max_spec && speculative_in_flight(p) >= p->max_spec)) {
                ++p->c.preload_refusals;
                return KVC_ERR_WOULD_BLOCK;
            }
        }
        int take = -1;
        if (nfree) {
            for (uint32_t i = 0; i < p->slots.size(); ++i)
                if (p->slots[i].state == FREE) {
                    take = (int)i;
                    break;
                }
        } else if (foreground) {
            // 3. no free slot: foreground work may take over a retained slot (least recently
            //    used first), else a staged preload that nobody claimed
            uint64_t best = ~0ull;
            for (uint32_t i = 0; i < p->slots.size(); ++i) {
                const PSlot &s = p->slots[i];
                if (s.state == RETAINED && s.refs == 0 && s.stamp < best) {
                    best = s.stamp;
                    take = (int)i;
                }
            }
            if (take < 0) {
                best = ~0ull;
                for (uint32_t i = 0; i < p->slots.size(); ++i) {
                    const PSlot &s = p->slots[i];
                    // refs == 0: the preloader has let go of it and nobody joined; a staged preload
                    // that is still referenced has I/O or a copy in progress on its slot
                    if (s.state == STAGED && s.speculative && s.refs == 0 && s.stamp < best) {
                        best = s.stamp;
                        take = (int)i;
                    }
                }
            }
            if (take >= 0) {
                forget(p, p->slots[take]);
                ++p->c.reclaims;
            }
        }
        if (take < 0) {
            ++p->c.foreground_refusals;
            return KVC_ERR_WOULD_BLOCK;
        }
        p->by_key[key] = (uint32_t)take;  // first: if this allocation fails, the slot is still free
        PSlot &s = p->slots[take];
        s.state = IN_FLIGHT;
        s.key = key;
        s.refs = 1;
        s.speculative = !foreground;
        s.stamp = ++p->clock;
        ++p->c.acquires;
        *slot = (uint32_t)take;
        *joined = 0;
        return KVC_OK;
    } catch (const std::bad_alloc &) {
        return KVC_ERR_NOMEM;
    }
}

kvc_status kvc_slot_pool_mark_staged(kvc_slot_pool *p, uint32_t slot)
{
    if (!p || slot >= p->slots.size())
        return KVC_ERR_INVALID_ARG;
    PSlot &s = p->slots[slot];
    if (s.state != IN_FLIGHT)
        return KVC_ERR_STATE;
    s.state = STAGED;
    return KVC_OK;
}

kvc_status kvc_slot_pool_release(kvc_slot_pool *p, uint32_t slot)
{
    if (!p || slot >= p->slots.size())
        return KVC_ERR_INVALID_ARG;
    PSlot &s = p->slots[slot];
    if ((s.state != IN_FLIGHT && s.state != STAGED) || s.refs == 0)
        return KVC_ERR_STATE;
    if (--s.refs > 0)
        return KVC_OK;
    if (s.speculative && s.state == STAGED)
        return KVC_OK;  // a finished preload waits, unreferenced, for the demand load that claims it
    if (p->retain && s.state == STAGED) {
        s.state = RETAINED;
        s.stamp = ++p->clock;
    } else {
        forget(p, s);
    }
    return KVC_OK;
}

kvc_status kvc_slot_pool_cancel(kvc_slot_pool *p, uint32_t slot)
{
    if (!p || slot >= p->slots.size())
        return KVC_ERR_INVALID_ARG;
    PSlot &s = p->slots[slot];
    // only an unclaimed preload still in flight can be cancelled, and only by its sole holder:
    // other preload candidates that joined it still expect the chunk to arrive in this slot
    if (s.state != IN_FLIGHT || !s.speculative || s.refs != 1)
        return KVC_ERR_STATE;
    forget(p, s);
    ++p->c.cancels;
    return KVC_OK;
}

kvc_status kvc_slot_pool_slot_info(const kvc_slot_pool *p, uint32_t slot, uint32_t *state, uint32_t *refs,
                                   uint64_t *key, int *speculative)
{
    if (!p || slot >= p->slots.size())
        return KVC_ERR_INVALID_ARG;
    const PSlot &s = p->slots[slot];
    if (state)
        *state = (uint32_t)s.state;
    if (refs)
        *refs = s.refs;
    if (key)
        *key = s.key;
    if (speculative)
        *speculative = s.speculative ? 1 : 0;
    return KVC_OK;
}

kvc_status kvc_slot_pool_get_counters(const kvc_slot_pool *p, kvc_slot_pool_counters *out)
{
    if (!p || !out)
        return KVC_ERR_INVALID_ARG;
    *out = p->c;
    out->n_free = out->n_in_flight = out->n_staged = out->n_retained = 0;
    for (const PSlot &s : p->slots) {
        out->n_free += s.state == FREE;
        out->n_in_flight += s.state == IN_FLIGHT;
        out->n_staged += s.state == STAGED;
        out->n_retained += s.state == RETAINED;
    }
    return KVC_OK;
}

}  // extern "C"
