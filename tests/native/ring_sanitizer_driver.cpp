// The staging ring (FIFO and pool mode) under AddressSanitizer / UBSan on a machine without a
// GPU: kvc_ring.cu is compiled as plain C++, the few CUDA runtime calls it names are replaced by
// the stand-ins below (never reached: the ring runs on caller memory with an event provider whose
// events complete on command), and a long random walk drives every entry point.
#include <cuda_runtime.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <vector>

#include "kvc.h"

extern "C" {
cudaError_t cudaEventCreateWithFlags(cudaEvent_t *, unsigned) { return cudaErrorNoDevice; }
cudaError_t cudaEventDestroy(cudaEvent_t) { return cudaErrorNoDevice; }
cudaError_t cudaEventRecord(cudaEvent_t, cudaStream_t) { return cudaErrorNoDevice; }
cudaError_t cudaEventQuery(cudaEvent_t) { return cudaErrorNoDevice; }
cudaError_t cudaEventSynchronize(cudaEvent_t) { return cudaErrorNoDevice; }
cudaError_t cudaStreamWaitEvent(cudaStream_t, cudaEvent_t, unsigned) { return cudaErrorNoDevice; }
cudaError_t cudaGetLastError(void) { return cudaSuccess; }
cudaError_t cudaMalloc(void **, size_t) { return cudaErrorNoDevice; }
cudaError_t cudaFree(void *) { return cudaErrorNoDevice; }
cudaError_t cudaHostAlloc(void **, size_t, unsigned) { return cudaErrorNoDevice; }
cudaError_t cudaFreeHost(void *) { return cudaErrorNoDevice; }
cudaError_t cudaHostGetDevicePointer(void **, void *, unsigned) { return cudaErrorNoDevice; }
}

#define CHECK(x)                                                      \
    do {                                                              \
        if (!(x)) {                                                   \
            printf("FAILED line %d: %s\n", __LINE__, #x);             \
            return 1;                                                 \
        }                                                             \
    } while (0)

namespace {
// events that complete when the driver says so
struct Ev {
    bool done = true;
};
std::vector<Ev *> g_all;
int ev_create(void *, void **out)
{
    Ev *e = new Ev();
    g_all.push_back(e);
    *out = e;
    return 0;
}
int ev_destroy(void *, void *e)
{
    for (Ev *&p : g_all)
        if (p == e)
            p = nullptr;
    delete static_cast<Ev *>(e);
    return 0;
}
int ev_record(void *, void *e, void *)
{
    static_cast<Ev *>(e)->done = false;
    return 0;
}
int ev_query(void *, void *e) { return static_cast<Ev *>(e)->done ? 0 : 1; }
int ev_wait(void *, void *, void *) { return 0; }
int ev_sync(void *, void *e)
{
    static_cast<Ev *>(e)->done = true;
    return 0;
}
uint32_t rnd(uint32_t *s)
{
    *s = *s * 1664525u + 1013904223u;
    return *s >> 8;
}
}  // namespace

int main()
{
    kvc_event_provider prov = {nullptr, ev_create, ev_destroy, ev_record, ev_query, ev_wait, ev_sync};
    CHECK(kvc_staging_ring_set_event_provider(&prov) == KVC_OK);
    const uint32_t n = 6;
    const uint64_t sb = 4096;
    void *mem = nullptr;
    CHECK(posix_memalign(&mem, 4096, n * sb) == 0);
    uint32_t seed = 12345;
    // ---- FIFO: stream many chunks through, with traces on
    kvc_ring *ring = nullptr;
    CHECK(kvc_staging_ring_create(sb, n, KVC_RING_DEVICE, mem, n * sb, &ring) == KVC_OK);
    std::vector<kvc_ring_trace_entry> trace(64);
    CHECK(kvc_staging_ring_set_trace(ring, trace.data(), (uint32_t)trace.size()) == KVC_OK);
    for (int i = 0; i < 500; ++i) {
        uint32_t slot = 0;
        void *dp = nullptr, *hp = nullptr;
        kvc_status s = kvc_staging_ring_acquire(ring, 0, &slot, &dp, &hp);
        if (s == KVC_ERR_WOULD_BLOCK) {
            for (Ev *e : g_all)
                if (e && rnd(&seed) % 2)
                    e->done = true;
            continue;
        }
        CHECK(s == KVC_OK && dp == (char *)mem + slot * sb);
        memset(dp, (int)i, sb);
        if (rnd(&seed) % 5 == 0) {
            CHECK(kvc_staging_ring_abandon(ring, slot) == KVC_OK);
            continue;
        }
        CHECK((rnd(&seed) % 2 ? kvc_staging_ring_commit(ring, slot, nullptr)
                              : kvc_staging_ring_commit_host(ring, slot)) == KVC_OK);
        CHECK(kvc_staging_ring_wait_filled(ring, slot, nullptr) == KVC_OK);
        CHECK(kvc_staging_ring_sync_filled(ring, slot) == KVC_OK);
        CHECK((rnd(&seed) % 2 ? kvc_staging_ring_release(ring, slot, nullptr)
                              : kvc_staging_ring_release_host(ring, slot)) == KVC_OK);
    }
    uint32_t in_flight = 0;
    uint64_t acq = 0, stalls = 0;
    CHECK(kvc_staging_ring_stats(ring, &in_flight, &acq, &stalls) == KVC_OK && acq > 100);
    CHECK(kvc_staging_ring_trace_count(ring) > trace.size());  // counted past the buffer, not written
    CHECK(kvc_staging_ring_destroy(ring) == KVC_OK);

    // ---- a staged ring: device half on caller memory, host half owned by the ring
    CHECK(kvc_staging_ring_create(sb, n, KVC_RING_DEVICE_STAGED, mem, n * sb, &ring) == KVC_OK);
    for (uint32_t i = 0; i < n; ++i) {
        uint32_t slot = 0;
        void *dp = nullptr, *hp = nullptr;
        CHECK(kvc_staging_ring_acquire(ring, 0, &slot, &dp, &hp) == KVC_OK && hp && hp != dp);
        memset(hp, 0x22, sb);
        memset(dp, 0x33, sb);
    }
    CHECK(kvc_staging_ring_kind(ring) == KVC_RING_DEVICE_STAGED);
    CHECK(kvc_staging_ring_destroy(ring) == KVC_OK);

    // ---- pool mode: random walk over classes, keys, joins, releases, cancels
    CHECK(kvc_staging_ring_create(sb, n, KVC_RING_DEVICE, mem, n * sb, &ring) == KVC_OK);
    CHECK(kvc_staging_ring_set_policy(ring, 2, 2, 1) == KVC_OK);
    std::vector<uint32_t> held(n, 0);
    std::vector<char> filled(n, 0), filler(n, 0);
    for (int i = 0; i < 5000; ++i) {
        const uint32_t op = rnd(&seed) % 7;
        if (op <= 1) {
            uint32_t slot = 0;
            int joined = 0;
            void *dp = nullptr, *hp = nullptr;
            const kvc_slot_class cls = (kvc_slot_class)(rnd(&seed) % 3);
            kvc_status s = kvc_staging_ring_acquire_for(ring, cls, rnd(&seed) % 9, 0, &slot, &dp, &hp, &joined);
            CHECK(s == KVC_OK || s == KVC_ERR_WOULD_BLOCK);
            if (s != KVC_OK)
                continue;
            if (!joined) {
                CHECK(held[slot] == 0);
                filled[slot] = 0;
                filler[slot] = 1;
                memset(dp, 0x11, sb);
            }
            ++held[slot];
        } else if (op == 2) {
            for (uint32_t sl = 0; sl < n; ++sl)
                if (held[sl] && !filled[sl] && filler[sl]) {
                    CHECK(kvc_staging_ring_commit_host(ring, sl) == KVC_OK);
                    filled[sl] = 1;
                    break;
                }
        } else if (op == 3) {
            const uint32_t sl = rnd(&seed) % n;
            if (held[sl] && filled[sl]) {
                CHECK((rnd(&seed) % 2 ? kvc_staging_ring_release(ring, sl, nullptr)
                                      : kvc_staging_ring_release_host(ring, sl)) == KVC_OK);
                --held[sl];
            }
        } else if (op == 4) {
            for (Ev *e : g_all)
                if (e && rnd(&seed) % 2)
                    e->done = true;
        } else if (op == 5) {
            const uint32_t sl = rnd(&seed) % n;
            if (held[sl] == 1 && !filled[sl] && filler[sl]) {
                kvc_status s = rnd(&seed) % 2 ? kvc_staging_ring_abandon(ring, sl) : kvc_staging_ring_cancel(ring, sl);
                CHECK(s == KVC_OK || s == KVC_ERR_STATE);
                if (s == KVC_OK) {
                    held[sl] = 0;
                    filler[sl] = 0;
                }
            }
        } else {
            int f = -1;
            CHECK(kvc_staging_ring_slot_filled(ring, rnd(&seed) % n, &f) == KVC_OK && (f == 0 || f == 1));
            CHECK(kvc_staging_ring_slot_filled(ring, n, &f) == KVC_ERR_INVALID_ARG);
        }
        kvc_slot_pool_counters c;
        CHECK(kvc_staging_ring_policy_counters(ring, &c) == KVC_OK);
        CHECK(c.n_free + c.n_in_flight + c.n_staged + c.n_retained == n);
    }
    CHECK(kvc_staging_ring_destroy(ring) == KVC_OK);  // with slots still held and events pending
    free(mem);
    CHECK(kvc_staging_ring_set_event_provider(nullptr) == KVC_OK);
    printf("ok\n");
    return 0;
}
