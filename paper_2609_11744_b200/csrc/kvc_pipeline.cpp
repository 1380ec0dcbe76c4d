// Store / load pipelines: a request's chunks go GPU -> mapped pinned ring slot -> file, and back.
// This is the reverse and forward pipeline of Sec. 6.4 reduced to what surrounds the GPU hot path:
// one job per chunk, each holding one slot of the bounded ring from the moment its copy is
// launched until its file I/O has completed; a request larger than the ring streams through it;
// I/O concurrency is a small fixed number of worker threads (the paper uses one io_uring reactor;
// with chunk-sized files the number of outstanding operations is what matters, not the mechanism).
// Loads stop at the first missing chunk: only the contiguous matching prefix is usable (Sec. 2.1).
//
// Built only from the public entry points of this library.
#include <chrono>
#include <condition_variable>
#include <deque>
#include <mutex>
#include <new>
#include <thread>
#include <vector>

#include "kvc.h"

namespace {

struct Job {
    uint32_t chunk, slot;
    void *host_ptr;
    void *dev_ptr;
    uint64_t bytes, hash;
    kvc_status status;
    bool existed;
};

// Work queue for the I/O threads and completion queue back to the calling thread.
struct Queues {
    std::mutex mu;
    std::condition_variable work_cv, done_cv;
    std::deque<Job> work, done;
    bool closing = false;
};

void io_worker(Queues *q, kvc_ring *ring, kvc_store *store, bool storing)
{
    for (;;) {
        Job j;
        {
            std::unique_lock<std::mutex> lk(q->mu);
            q->work_cv.wait(lk, [&] { return q->closing || !q->work.empty(); });
            if (q->work.empty())
                return;
            j = q->work.front();
            q->work.pop_front();
        }
        if (storing) {
            // the slot's copy was only enqueued: wait for its "filled" event, then write the file
            j.status = kvc_staging_ring_sync_filled(ring, j.slot);
            if (j.status == KVC_OK) {
                j.status = kvc_store_publish(store, j.hash, j.host_ptr, j.bytes);
                if (j.status == KVC_ERR_EXISTS) {
                    j.existed = true;
                    j.status = KVC_OK;
                }
            }
        } else {
            j.status = kvc_store_read(store, j.hash, j.host_ptr, j.bytes);
        }
        {
            std::lock_guard<std::mutex> lk(q->mu);
            q->done.push_back(j);
        }
        q->done_cv.notify_one();
    }
}

struct Workers {
    Queues q;
    std::vector<std::thread> threads;
    ~Workers()
    {
        {
            std::lock_guard<std::mutex> lk(q.mu);
            q.closing = true;
        }
        q.work_cv.notify_all();
        for (std::thread &t : threads)
            if (t.joinable())
                t.join();
    }
};

double now_s()
{
    return std::chrono::duration<double>(std::chrono::steady_clock::now().time_since_epoch()).count();
}

kvc_status run(kvc_layout *lay, kvc_ring *ring, kvc_store *store, const int32_t *ids, uint32_t n_blocks,
               const uint64_t *hashes, uint32_t n_hashes, uint32_t io_threads, int use_copy_engine,
               void *stream, bool storing, kvc_pipeline_stats *out)
{
    if (!lay || !ring || !store || (!ids && n_blocks) || (!hashes && n_hashes))
        return KVC_ERR_INVALID_ARG;
    kvc_pipeline_stats st = {};
    const double t0 = now_s();
    uint32_t n_chunks = 0;
    kvc_status rc = kvc_map_request(lay, n_blocks, 0, nullptr, 0, &n_chunks);
    if (rc != KVC_OK)
        return rc;
    if (n_hashes < n_chunks)
        return KVC_ERR_INVALID_ARG;
    std::vector<kvc_chunk_desc> descs;
    try {
        descs.resize(n_chunks ? n_chunks : 1);
    } catch (const std::bad_alloc &) {
        return KVC_ERR_NOMEM;
    }
    rc = kvc_map_request(lay, n_blocks, 0, descs.data(), n_chunks, &n_chunks);
    if (rc != KVC_OK)
        return rc;
    const uint64_t slot_bytes = kvc_staging_ring_slot_bytes(ring);
    for (uint32_t c = 0; c < n_chunks; ++c)
        if (descs[c].bytes > slot_bytes)
            return KVC_ERR_INVALID_ARG;
    if (!storing) {
        // only the contiguous prefix of chunks that are present (and of the right size) is loaded
        uint32_t have = 0;
        for (; have < n_chunks; ++have) {
            uint64_t sz = 0;
            if (kvc_store_lookup(store, hashes[have], &sz) != KVC_OK || sz != descs[have].bytes)
                break;
        }
        n_chunks = have;
    }
    Workers w;
    const uint32_t nthreads = io_threads ? io_threads : 4;
    try {
        for (uint32_t i = 0; i < nthreads; ++i)
            w.threads.emplace_back(io_worker, &w.q, ring, store, storing);
    } catch (...) {
        return KVC_ERR_NOMEM;
    }

    uint32_t issued = 0, finished = 0;
    kvc_status first_err = KVC_OK;
    // one completion: for a store the slot is free again; for a load the chunk is in its slot
    // and is unpacked on the stream, which then owns the slot until the kernel has run
    auto complete = [&](const Job &j) {
        ++finished;
        if (j.status != KVC_OK) {
            if (first_err == KVC_OK)
                first_err = j.status;
            if (storing)
                kvc_staging_ring_release_host(ring, j.slot);
            else if (kvc_staging_ring_commit_host(ring, j.slot) == KVC_OK)
                kvc_staging_ring_release_host(ring, j.slot);
            return;
        }
        st.bytes += j.bytes;
        if (storing) {
            j.existed ? ++st.already_present : ++st.published;
            kvc_staging_ring_release_host(ring, j.slot);
            return;
        }
        const kvc_chunk_desc &d = descs[j.chunk];
        kvc_status s = kvc_staging_ring_commit_host(ring, j.slot);
        if (s == KVC_OK)
            s = use_copy_engine
                    ? kvc_unpack_copy_engine(lay, j.host_ptr, j.bytes, ids + d.first, d.n_blocks, stream)
                    : kvc_unpack(lay, j.dev_ptr, j.bytes, ids + d.first, d.n_blocks, 0, stream);
        if (s == KVC_OK)
            s = kvc_staging_ring_release(ring, j.slot, stream);
        else
            kvc_staging_ring_release_host(ring, j.slot);
        if (s != KVC_OK && first_err == KVC_OK)
            first_err = s;
    };
    auto reap = [&](bool block) {
        std::unique_lock<std::mutex> lk(w.q.mu);
        if (block && w.q.done.empty() && finished < issued)
            w.q.done_cv.wait_for(lk, std::chrono::milliseconds(200));
        while (!w.q.done.empty()) {
            Job j = w.q.done.front();
            w.q.done.pop_front();
            lk.unlock();
            complete(j);
            lk.lock();
        }
    };

    const double deadline = now_s() + 600.0;  // a bounded wait, never forever
    for (uint32_t c = 0; c < n_chunks && first_err == KVC_OK; ++c) {
        uint32_t slot = 0;
        void *dptr = nullptr, *hptr = nullptr;
        for (;;) {
            reap(false);
            kvc_status s = kvc_staging_ring_acquire(ring, 0, &slot, &dptr, &hptr);
            if (s == KVC_OK)
                break;
            if (s != KVC_ERR_WOULD_BLOCK) {
                first_err = s;
                break;
            }
            ++st.ring_stalls;
            if (now_s() > deadline) {
                first_err = KVC_ERR_TIMEOUT;
                break;
            }
            if (finished < issued)
                reap(true);   // a slot comes back when one of the jobs in flight completes
            else
                std::this_thread::sleep_for(std::chrono::microseconds(50));  // waiting for a kernel
        }
        if (first_err != KVC_OK)
            break;
        if (!hptr) {  // the pipelines need slots the host can read and write
            kvc_staging_ring_commit_host(ring, slot);
            kvc_staging_ring_release_host(ring, slot);
            first_err = KVC_ERR_INVALID_ARG;
            break;
        }
        const kvc_chunk_desc &d = descs[c];
        Job j = {c, slot, hptr, dptr, d.bytes, hashes[c], KVC_OK, false};
        if (storing) {
            kvc_status s = use_copy_engine
                               ? kvc_pack_copy_engine(lay, ids + d.first, d.n_blocks, hptr, d.bytes, stream)
                               : kvc_pack(lay, ids + d.first, d.n_blocks, 0, dptr, d.bytes, stream);
            if (s == KVC_OK)
                s = kvc_staging_ring_commit(ring, slot, stream);
            if (s != KVC_OK) {
                first_err = s;
                break;
            }
        }
        {
            std::lock_guard<std::mutex> lk(w.q.mu);
            w.q.work.push_back(j);
        }
        w.q.work_cv.notify_one();
        ++issued;
        ++st.chunks;
    }
    while (finished < issued && now_s() < deadline)
        reap(true);
    if (finished < issued && first_err == KVC_OK)
        first_err = KVC_ERR_TIMEOUT;
    st.seconds = now_s() - t0;
    if (out)
        *out = st;
    return first_err;
}

}  // namespace

extern "C" {

kvc_status kvc_pipeline_store(kvc_layout *lay, kvc_ring *ring, kvc_store *store, const int32_t *ids,
                              uint32_t n_blocks, const uint64_t *hashes, uint32_t n_hashes,
                              uint32_t io_threads, int use_copy_engine, void *stream,
                              kvc_pipeline_stats *stats)
{
    return run(lay, ring, store, ids, n_blocks, hashes, n_hashes, io_threads, use_copy_engine, stream,
               true, stats);
}

kvc_status kvc_pipeline_load(kvc_layout *lay, kvc_ring *ring, kvc_store *store, const int32_t *ids,
                             uint32_t n_blocks, const uint64_t *hashes, uint32_t n_hashes,
                             uint32_t io_threads, int use_copy_engine, void *stream,
                             kvc_pipeline_stats *stats)
{
    return run(lay, ring, store, ids, n_blocks, hashes, n_hashes, io_threads, use_copy_engine, stream,
               false, stats);
}

}  // extern "C"
