// Bounded staging ring (Sec. 6.4): a fixed pool of equal slots shared by every transfer; a
// slot returns to the pool only after the event recorded behind its last copy has completed.
// Host bookkeeping plus two events per slot; no kernel, no device-wide synchronisation.
#include <stdlib.h>

#include <chrono>
#include <mutex>
#include <new>
#include <thread>
#include <vector>

#include "kvc_internal.h"

namespace {

// ---- default event provider: CUDA events
int cu_create(void *, void **ev)
{
    cudaEvent_t e;
    if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess)
        return -1;
    *ev = e;
    return 0;
}
int cu_destroy(void *, void *ev) { return cudaEventDestroy((cudaEvent_t)ev) == cudaSuccess ? 0 : -1; }
int cu_record(void *, void *ev, void *st)
{
    return cudaEventRecord((cudaEvent_t)ev, (cudaStream_t)st) == cudaSuccess ? 0 : -1;
}
int cu_query(void *, void *ev)
{
    cudaError_t e = cudaEventQuery((cudaEvent_t)ev);
    if (e == cudaSuccess)
        return 0;
    if (e == cudaErrorNotReady) {
        (void)cudaGetLastError();
        return 1;
    }
    return -1;
}
int cu_stream_wait(void *, void *st, void *ev)
{
    return cudaStreamWaitEvent((cudaStream_t)st, (cudaEvent_t)ev, 0) == cudaSuccess ? 0 : -1;
}
int cu_sync(void *, void *ev) { return cudaEventSynchronize((cudaEvent_t)ev) == cudaSuccess ? 0 : -1; }

const kvc_event_provider kCudaEvents = {nullptr, cu_create, cu_destroy, cu_record,
                                        cu_query, cu_stream_wait, cu_sync};
// process-wide default for rings created from now on; rings copy it at creation
std::mutex g_events_mu;
kvc_event_provider g_events = kCudaEvents;
bool g_events_custom = false;

enum SlotState {
    SLOT_FREE = 0,      // never used, or seen drained
    SLOT_ACQUIRED = 1,  // handed to a producer
    SLOT_FILLED = 2,    // "filled" event recorded
    SLOT_DRAINING = 3   // "drained" event recorded, not yet seen complete
};

struct Slot {
    SlotState state = SLOT_FREE;
    void *filled = nullptr;
    void *drained = nullptr;
    bool filled_by_host = false;  // committed by kvc_staging_ring_commit_host: no event to wait for
    // pool mode: references released by consumers whose GPU work (guarded by `drained`) may still
    // be reading the slot; they are handed back to the slot policy once the event has completed
    uint32_t deferred = 0;
};

}  // namespace

struct kvc_ring {
    kvc_event_provider ev;
    bool custom_events;
    kvc_ring_kind kind;
    uint64_t slot_bytes;
    uint32_t n_slots;
    unsigned char *dev_base;   // address for kernels and async copies
    unsigned char *host_base;  // host address (HOST_MAPPED) or nullptr
    bool owns_mem;
    bool owns_host_part;       // DEVICE_STAGED: the pinned host half always belongs to the ring
    bool host_part_is_malloc;  // ... and is plain memory when a test's event provider stands in for CUDA
    std::vector<Slot> slots;
    uint32_t head;             // next slot to hand out
    uint64_t acquires, stalls;
    kvc_ring_trace_entry *trace;  // caller's buffer, or nullptr
    uint32_t trace_cap, trace_n;
    kvc_slot_pool *policy;     // pool mode: who gets which slot (nullptr = FIFO ring)
};

namespace {

void trace(kvc_ring *r, uint32_t slot, kvc_ring_trace_kind what)
{
    if (!r->trace)
        return;
    if (r->trace_n < r->trace_cap) {
        kvc_ring_trace_entry &e = r->trace[r->trace_n];
        e.t_ns = (uint64_t)std::chrono::duration_cast<std::chrono::nanoseconds>(
                     std::chrono::steady_clock::now().time_since_epoch())
                     .count();
        e.slot = slot;
        e.what = (uint32_t)what;
    }
    ++r->trace_n;  // keeps counting past the capacity so that the caller can see what was dropped
}

// FREE, or DRAINING whose event has completed.  Returns 0 free, 1 busy, <0 error.
int slot_is_free(kvc_ring *r, Slot &s)
{
    if (s.state == SLOT_FREE)
        return 0;
    if (s.state != SLOT_DRAINING)
        return 1;
    int q = r->ev.query(r->ev.ctx, s.drained);
    if (q == 0)
        s.state = SLOT_FREE;
    return q;
}

// Pool mode: a slot the policy has freed is free here too (a retained or unclaimed staged slot
// keeps its bytes and stays FILLED).
void sync_with_policy(kvc_ring *r, uint32_t slot)
{
    uint32_t state = 0;
    kvc_slot_pool_slot_info(r->policy, slot, &state, nullptr, nullptr, nullptr);
    if (state == KVC_SLOT_FREE)
        r->slots[slot].state = SLOT_FREE;
}

// Pool mode: hands references whose GPU work has completed back to the policy.
// Returns <0 on an event error.
int reap_deferred(kvc_ring *r)
{
    for (uint32_t i = 0; i < r->n_slots; ++i) {
        Slot &s = r->slots[i];
        if (!s.deferred)
            continue;
        const int q = r->ev.query(r->ev.ctx, s.drained);
        if (q < 0)
            return q;
        if (q != 0)
            continue;
        for (; s.deferred; --s.deferred)
            kvc_slot_pool_release(r->policy, i);
        sync_with_policy(r, i);
    }
    return 0;
}

}  // namespace

extern "C" {

kvc_status kvc_staging_ring_set_event_provider(const kvc_event_provider *p)
{
    if (p && (!p->create || !p->destroy || !p->record || !p->query || !p->stream_wait ||
              !p->synchronize))
        return KVC_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(g_events_mu);
    g_events = p ? *p : kCudaEvents;
    g_events_custom = p != nullptr;
    return KVC_OK;
}

kvc_status kvc_staging_ring_create(uint64_t slot_bytes, uint32_t n_slots, kvc_ring_kind kind,
                                   void *mem, uint64_t mem_bytes, kvc_ring **out)
{
    if (!out)
        return KVC_ERR_INVALID_ARG;
    *out = nullptr;
    if (slot_bytes == 0 || n_slots == 0 ||
        (kind != KVC_RING_DEVICE && kind != KVC_RING_HOST_MAPPED && kind != KVC_RING_DEVICE_STAGED))
        return KVC_ERR_INVALID_ARG;
    if (slot_bytes % 4096)
        return KVC_ERR_ALIGNMENT;
    const uint64_t total = slot_bytes * n_slots;
    if (total / n_slots != slot_bytes)
        return KVC_ERR_INVALID_ARG;
    if (mem) {
        if (mem_bytes < total)
            return KVC_ERR_INVALID_ARG;
        if ((uintptr_t)mem % 16)
            return KVC_ERR_ALIGNMENT;
    }
    kvc_ring *r = new (std::nothrow) kvc_ring();
    if (!r)
        return KVC_ERR_NOMEM;
    {
        std::lock_guard<std::mutex> lock(g_events_mu);
        r->ev = g_events;
        r->custom_events = g_events_custom;
    }
    r->kind = kind;
    r->slot_bytes = slot_bytes;
    r->n_slots = n_slots;
    r->dev_base = r->host_base = nullptr;
    r->owns_mem = false;
    r->owns_host_part = false;
    r->host_part_is_malloc = false;
    r->head = 0;
    r->acquires = r->stalls = 0;
    r->trace = nullptr;
    r->trace_cap = r->trace_n = 0;
    r->policy = nullptr;
    try {
        r->slots.resize(n_slots);
    } catch (const std::bad_alloc &) {
        delete r;
        return KVC_ERR_NOMEM;
    }
    kvc_status rc = KVC_OK;
    if (mem) {
        r->dev_base = static_cast<unsigned char *>(mem);
        if (kind == KVC_RING_HOST_MAPPED) {
            // the caller's pinned buffer: kernels use its device alias
            r->host_base = static_cast<unsigned char *>(mem);
            if (!r->custom_events) {
                void *d = nullptr;
                if (cudaHostGetDevicePointer(&d, mem, 0) != cudaSuccess) {
                    (void)cudaGetLastError();
                    rc = KVC_ERR_CUDA;
                } else {
                    r->dev_base = static_cast<unsigned char *>(d);
                }
            }
        }
    } else if (kind == KVC_RING_DEVICE || kind == KVC_RING_DEVICE_STAGED) {
        void *p = nullptr;
        if (cudaMalloc(&p, total) != cudaSuccess) {
            (void)cudaGetLastError();
            rc = KVC_ERR_NOMEM;
        }
        r->dev_base = static_cast<unsigned char *>(p);
        r->owns_mem = rc == KVC_OK;
    } else {
        void *h = nullptr, *d = nullptr;
        if (cudaHostAlloc(&h, total, cudaHostAllocMapped) != cudaSuccess) {
            (void)cudaGetLastError();
            rc = KVC_ERR_NOMEM;
        } else if (cudaHostGetDevicePointer(&d, h, 0) != cudaSuccess) {
            (void)cudaGetLastError();
            cudaFreeHost(h);
            rc = KVC_ERR_CUDA;
        } else {
            r->host_base = static_cast<unsigned char *>(h);
            r->dev_base = static_cast<unsigned char *>(d);
            r->owns_mem = true;
        }
    }
    if (rc == KVC_OK && kind == KVC_RING_DEVICE_STAGED) {
        // the host half of every slot: pinned memory the copy engines can reach at full speed
        void *h = nullptr;
        if (r->custom_events) {
            if (posix_memalign(&h, 4096, total) != 0)
                rc = KVC_ERR_NOMEM;
            r->host_part_is_malloc = rc == KVC_OK;
        } else if (cudaHostAlloc(&h, total, cudaHostAllocDefault) != cudaSuccess) {
            (void)cudaGetLastError();
            rc = KVC_ERR_NOMEM;
        }
        if (rc == KVC_OK) {
            r->host_base = static_cast<unsigned char *>(h);
            r->owns_host_part = true;
        }
    }
    for (uint32_t i = 0; rc == KVC_OK && i < n_slots; ++i) {
        if (r->ev.create(r->ev.ctx, &r->slots[i].filled) != 0 ||
            r->ev.create(r->ev.ctx, &r->slots[i].drained) != 0)
            rc = KVC_ERR_CUDA;
    }
    if (rc != KVC_OK) {
        kvc_staging_ring_destroy(r);
        return rc;
    }
    *out = r;
    return KVC_OK;
}

kvc_status kvc_staging_ring_destroy(kvc_ring *r)
{
    if (!r)
        return KVC_ERR_INVALID_ARG;
    kvc_status rc = KVC_OK;
    for (Slot &s : r->slots) {
        // work recorded behind a slot may still touch ring memory: wait for it before freeing
        if (s.state == SLOT_FILLED && s.filled && r->ev.synchronize(r->ev.ctx, s.filled) != 0)
            rc = KVC_ERR_CUDA;
        if ((s.state == SLOT_DRAINING || s.deferred) && s.drained &&
            r->ev.synchronize(r->ev.ctx, s.drained) != 0)
            rc = KVC_ERR_CUDA;
        if (s.filled)
            r->ev.destroy(r->ev.ctx, s.filled);
        if (s.drained)
            r->ev.destroy(r->ev.ctx, s.drained);
    }
    if (r->policy)
        kvc_slot_pool_destroy(r->policy);
    if (r->owns_mem) {
        if (r->kind == KVC_RING_HOST_MAPPED)
            cudaFreeHost(r->host_base);
        else
            cudaFree(r->dev_base);
    }
    if (r->owns_host_part) {
        if (r->host_part_is_malloc)
            free(r->host_base);
        else
            cudaFreeHost(r->host_base);
    }
    delete r;
    return rc;
}

kvc_status kvc_staging_ring_acquire(kvc_ring *r, int64_t timeout_us, uint32_t *slot, void **dev_ptr,
                                    void **host_ptr)
{
    if (!r || !slot || timeout_us < 0)
        return KVC_ERR_INVALID_ARG;
    if (r->policy)
        return KVC_ERR_STATE;  // pool mode: slots are handed out by kvc_staging_ring_acquire_for
    Slot &s = r->slots[r->head];
    const auto deadline =
        std::chrono::steady_clock::now() + std::chrono::microseconds(timeout_us);
    bool stall_logged = false;
    // Polling a slot whose "drained" event has not completed yet: a few immediate retries (the
    // event is often microseconds away), then sleeps that double from 2 to 20 microseconds, so a
    // waiting thread does not burn a core while the host link drains a 32 MiB slot (~600 us).
    uint32_t polls = 0, nap_us = 2;
    for (;;) {
        int q = slot_is_free(r, s);
        if (q < 0)
            return KVC_ERR_CUDA;
        if (q == 0)
            break;
        ++r->stalls;
        if (!stall_logged) {
            trace(r, r->head, KVC_TRACE_STALL);
            stall_logged = true;
        }
        if (timeout_us == 0)
            return KVC_ERR_WOULD_BLOCK;
        if (std::chrono::steady_clock::now() >= deadline)
            return KVC_ERR_TIMEOUT;
        if (s.state != SLOT_DRAINING) {
            // held by a producer or consumer of this same thread: only the caller can move it on
            std::this_thread::sleep_for(std::chrono::microseconds(50));
        } else if (++polls <= 8) {
            std::this_thread::yield();
        } else {
            std::this_thread::sleep_for(std::chrono::microseconds(nap_us));
            nap_us = nap_us * 2 > 20 ? 20 : nap_us * 2;
        }
    }
    s.state = SLOT_ACQUIRED;
    *slot = r->head;
    if (dev_ptr)
        *dev_ptr = r->dev_base + (uint64_t)r->head * r->slot_bytes;
    if (host_ptr)
        *host_ptr = r->host_base ? r->host_base + (uint64_t)r->head * r->slot_bytes : nullptr;
    trace(r, r->head, KVC_TRACE_ACQUIRE);
    r->head = (r->head + 1) % r->n_slots;
    ++r->acquires;
    return KVC_OK;
}

kvc_status kvc_staging_ring_commit(kvc_ring *r, uint32_t slot, void *producer_stream)
{
    if (!r || slot >= r->n_slots)
        return KVC_ERR_INVALID_ARG;
    Slot &s = r->slots[slot];
    if (s.state != SLOT_ACQUIRED)
        return KVC_ERR_STATE;
    if (r->ev.record(r->ev.ctx, s.filled, producer_stream) != 0)
        return KVC_ERR_CUDA;
    s.filled_by_host = false;
    s.state = SLOT_FILLED;
    if (r->policy)
        kvc_slot_pool_mark_staged(r->policy, slot);
    trace(r, slot, KVC_TRACE_COMMIT);
    return KVC_OK;
}

kvc_status kvc_staging_ring_wait_filled(kvc_ring *r, uint32_t slot, void *consumer_stream)
{
    if (!r || slot >= r->n_slots)
        return KVC_ERR_INVALID_ARG;
    Slot &s = r->slots[slot];
    if (s.state != SLOT_FILLED)
        return KVC_ERR_STATE;
    if (!s.filled_by_host && r->ev.stream_wait(r->ev.ctx, consumer_stream, s.filled) != 0)
        return KVC_ERR_CUDA;
    return KVC_OK;
}

kvc_status kvc_staging_ring_release(kvc_ring *r, uint32_t slot, void *consumer_stream)
{
    if (!r || slot >= r->n_slots)
        return KVC_ERR_INVALID_ARG;
    Slot &s = r->slots[slot];
    if (s.state != SLOT_FILLED)
        return KVC_ERR_STATE;
    if (r->policy) {
        // one consumer lets go; others may still hold the slot.  The event is re-recorded behind
        // every consumer's stream, each made to wait for the record before it, so its completion
        // means that all consumers released so far are done.
        uint32_t refs = 0;
        kvc_slot_pool_slot_info(r->policy, slot, nullptr, &refs, nullptr, nullptr);
        if (refs <= s.deferred)
            return KVC_ERR_STATE;  // more releases than references
        if (s.deferred && r->ev.stream_wait(r->ev.ctx, consumer_stream, s.drained) != 0)
            return KVC_ERR_CUDA;
        if (r->ev.record(r->ev.ctx, s.drained, consumer_stream) != 0)
            return KVC_ERR_CUDA;
        ++s.deferred;
        trace(r, slot, KVC_TRACE_RELEASE);
        return KVC_OK;
    }
    if (r->ev.record(r->ev.ctx, s.drained, consumer_stream) != 0)
        return KVC_ERR_CUDA;
    s.state = SLOT_DRAINING;
    trace(r, slot, KVC_TRACE_RELEASE);
    return KVC_OK;
}

kvc_status kvc_staging_ring_commit_host(kvc_ring *r, uint32_t slot)
{
    if (!r || slot >= r->n_slots)
        return KVC_ERR_INVALID_ARG;
    Slot &s = r->slots[slot];
    if (s.state != SLOT_ACQUIRED)
        return KVC_ERR_STATE;
    s.filled_by_host = true;
    s.state = SLOT_FILLED;
    if (r->policy)
        kvc_slot_pool_mark_staged(r->policy, slot);
    trace(r, slot, KVC_TRACE_COMMIT);
    return KVC_OK;
}

kvc_status kvc_staging_ring_sync_filled(kvc_ring *r, uint32_t slot)
{
    if (!r || slot >= r->n_slots)
        return KVC_ERR_INVALID_ARG;
    Slot &s = r->slots[slot];
    if (s.state != SLOT_FILLED)
        return KVC_ERR_STATE;
    if (!s.filled_by_host && r->ev.synchronize(r->ev.ctx, s.filled) != 0)
        return KVC_ERR_CUDA;
    return KVC_OK;
}

kvc_status kvc_staging_ring_release_host(kvc_ring *r, uint32_t slot)
{
    if (!r || slot >= r->n_slots)
        return KVC_ERR_INVALID_ARG;
    Slot &s = r->slots[slot];
    if (r->policy) {
        uint32_t refs = 0;
        kvc_slot_pool_slot_info(r->policy, slot, nullptr, &refs, nullptr, nullptr);
        // a filled slot: any holder may let go; a slot still being filled: only someone who
        // joined it (the filler's own reference has to stay until it commits or abandons)
        if (!(s.state == SLOT_FILLED && refs > s.deferred) && !(s.state == SLOT_ACQUIRED && refs > 1))
            return KVC_ERR_STATE;
        kvc_slot_pool_release(r->policy, slot);
        sync_with_policy(r, slot);
        trace(r, slot, KVC_TRACE_RELEASE);
        return KVC_OK;
    }
    if (s.state != SLOT_FILLED)
        return KVC_ERR_STATE;
    s.state = SLOT_FREE;
    trace(r, slot, KVC_TRACE_RELEASE);
    return KVC_OK;
}

kvc_status kvc_staging_ring_stats(const kvc_ring *r, uint32_t *in_flight, uint64_t *acquires,
                                  uint64_t *stalls)
{
    if (!r)
        return KVC_ERR_INVALID_ARG;
    if (in_flight) {
        // released slots whose event has completed meanwhile count as free: ask the events
        kvc_ring *rw = const_cast<kvc_ring *>(r);
        if (rw->policy)
            (void)reap_deferred(rw);
        uint32_t n = 0;
        for (Slot &s : rw->slots) {
            if (s.state == SLOT_DRAINING)
                (void)slot_is_free(rw, s);
            n += s.state != SLOT_FREE;
        }
        *in_flight = n;
    }
    if (acquires)
        *acquires = r->acquires;
    if (stalls)
        *stalls = r->stalls;
    return KVC_OK;
}

kvc_status kvc_staging_ring_set_trace(kvc_ring *r, kvc_ring_trace_entry *buf, uint32_t cap)
{
    if (!r || (buf && cap == 0))
        return KVC_ERR_INVALID_ARG;
    r->trace = buf;
    r->trace_cap = buf ? cap : 0;
    r->trace_n = 0;
    return KVC_OK;
}

uint32_t kvc_staging_ring_trace_count(const kvc_ring *r) { return r ? r->trace_n : 0; }

kvc_status kvc_staging_ring_set_policy(kvc_ring *r, uint32_t foreground_reserve, uint32_t max_speculative,
                                       int retain_completed)
{
    if (!r)
        return KVC_ERR_INVALID_ARG;
    if (r->policy && reap_deferred(r) < 0)
        return KVC_ERR_CUDA;
    for (Slot &s : r->slots) {
        if (s.state == SLOT_DRAINING && slot_is_free(r, s) < 0)
            return KVC_ERR_CUDA;
        if (s.state != SLOT_FREE || s.deferred)
            return KVC_ERR_STATE;  // only while every slot is free (no cached chunk either)
    }
    kvc_slot_pool *p = nullptr;
    kvc_status rc = kvc_slot_pool_create(r->n_slots, foreground_reserve, max_speculative, retain_completed, &p);
    if (rc != KVC_OK)
        return rc;
    if (r->policy)
        kvc_slot_pool_destroy(r->policy);
    r->policy = p;
    for (Slot &s : r->slots) {
        s.state = SLOT_FREE;
        s.deferred = 0;
    }
    r->head = 0;
    return KVC_OK;
}

kvc_status kvc_staging_ring_acquire_for(kvc_ring *r, kvc_slot_class cls, uint64_t key, int64_t timeout_us,
                                        uint32_t *slot, void **dev_ptr, void **host_ptr, int *joined)
{
    if (!r || !slot || !joined || timeout_us < 0)
        return KVC_ERR_INVALID_ARG;
    if (!r->policy)
        return KVC_ERR_STATE;
    const auto deadline = std::chrono::steady_clock::now() + std::chrono::microseconds(timeout_us);
    bool stall_logged = false;
    uint32_t polls = 0, nap_us = 2;
    for (;;) {
        if (reap_deferred(r) < 0)
            return KVC_ERR_CUDA;
        uint32_t got = 0;
        int j = 0;
        const kvc_status rc = kvc_slot_pool_acquire(r->policy, cls, key, &got, &j);
        if (rc == KVC_OK) {
            Slot &s = r->slots[got];
            if (!j) {
                // a fresh slot, or one taken over from a retained / unclaimed staged chunk: its old
                // references are all back (the policy only gives away unreferenced slots), so no
                // GPU work can still be touching it
                s.state = SLOT_ACQUIRED;
                s.filled_by_host = false;
                ++r->acquires;
                trace(r, got, KVC_TRACE_ACQUIRE);
            }
            *slot = got;
            *joined = j;
            if (dev_ptr)
                *dev_ptr = r->dev_base + (uint64_t)got * r->slot_bytes;
            if (host_ptr)
                *host_ptr = r->host_base ? r->host_base + (uint64_t)got * r->slot_bytes : nullptr;
            return KVC_OK;
        }
        if (rc != KVC_ERR_WOULD_BLOCK)
            return rc;
        ++r->stalls;
        if (!stall_logged) {
            trace(r, r->n_slots, KVC_TRACE_STALL);
            stall_logged = true;
        }
        if (timeout_us == 0)
            return KVC_ERR_WOULD_BLOCK;
        if (std::chrono::steady_clock::now() >= deadline)
            return KVC_ERR_TIMEOUT;
        if (++polls <= 8) {
            std::this_thread::yield();
        } else {
            std::this_thread::sleep_for(std::chrono::microseconds(nap_us));
            nap_us = nap_us * 2 > 20 ? 20 : nap_us * 2;
        }
    }
}

kvc_status kvc_staging_ring_slot_filled(kvc_ring *r, uint32_t slot, int *filled)
{
    if (!r || slot >= r->n_slots || !filled)
        return KVC_ERR_INVALID_ARG;
    *filled = r->slots[slot].state == SLOT_FILLED;
    return KVC_OK;
}

kvc_status kvc_staging_ring_cancel(kvc_ring *r, uint32_t slot)
{
    if (!r || slot >= r->n_slots)
        return KVC_ERR_INVALID_ARG;
    if (!r->policy || r->slots[slot].state != SLOT_ACQUIRED)
        return KVC_ERR_STATE;
    const kvc_status rc = kvc_slot_pool_cancel(r->policy, slot);
    if (rc == KVC_OK)
        r->slots[slot].state = SLOT_FREE;
    return rc;
}

kvc_status kvc_staging_ring_abandon(kvc_ring *r, uint32_t slot)
{
    if (!r || slot >= r->n_slots)
        return KVC_ERR_INVALID_ARG;
    Slot &s = r->slots[slot];
    if (s.state != SLOT_ACQUIRED)
        return KVC_ERR_STATE;
    if (!r->policy) {
        s.state = SLOT_FREE;
        return KVC_OK;
    }
    uint32_t refs = 0;
    kvc_slot_pool_slot_info(r->policy, slot, nullptr, &refs, nullptr, nullptr);
    if (refs != 1)
        return KVC_ERR_STATE;  // others joined and wait for the bytes
    kvc_slot_pool_release(r->policy, slot);  // in flight, last reference: the slot is freed
    sync_with_policy(r, slot);
    return KVC_OK;
}

kvc_status kvc_staging_ring_policy_counters(kvc_ring *r, kvc_slot_pool_counters *out)
{
    if (!r || !out)
        return KVC_ERR_INVALID_ARG;
    if (!r->policy)
        return KVC_ERR_STATE;
    if (reap_deferred(r) < 0)
        return KVC_ERR_CUDA;
    return kvc_slot_pool_get_counters(r->policy, out);
}

int kvc_staging_ring_pool_mode(const kvc_ring *r) { return r && r->policy ? 1 : 0; }
kvc_ring_kind kvc_staging_ring_kind(const kvc_ring *r) { return r ? r->kind : KVC_RING_DEVICE; }
uint64_t kvc_staging_ring_slot_bytes(const kvc_ring *r) { return r ? r->slot_bytes : 0; }
uint32_t kvc_staging_ring_num_slots(const kvc_ring *r) { return r ? r->n_slots : 0; }

}  // extern "C"
