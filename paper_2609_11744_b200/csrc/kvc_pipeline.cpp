// Store / load pipelines: a request's chunks go GPU -> mapped pinned staging slot -> file, and back.
// This is the forward and reverse pipeline of Sec. 6.4 reduced to what surrounds the GPU hot path:
// one job per chunk, each holding one slot of the bounded staging memory from the moment its copy
// is launched until its file I/O has completed; a request larger than the staging memory streams
// through it; I/O concurrency is a small fixed number of worker threads (the paper uses one
// io_uring reactor; with chunk-sized files the number of outstanding operations is what matters,
// not the mechanism).  Loads stop at the first missing chunk: only the contiguous matching prefix
// is usable (Sec. 2.1).
//
// With the staging memory in pool mode (Sec. 6.5) several requests are served at once: a chunk
// whose hash already holds a slot -- being read, read, or cached -- is joined instead of read
// again, demand loads go before preloads, and everything that became ready during one pass of
// the loop, for whichever requests, is scattered by ONE fused unpack launch (Sec. 6.4).
//
// Staging slots may be mapped pinned memory (the kernels cross the host link themselves) or
// device-plus-host pairs (KVC_RING_DEVICE_STAGED: the kernels fill the device half and one
// asynchronous copy per chunk, on a copy stream of the call's own, crosses the link).
//
// Built from the public entry points of this library, plus the CUDA runtime for those copies.
// Every exit, error exits included, hands every slot it took back to the staging memory.
#include <chrono>
#include <condition_variable>
#include <map>
#include <mutex>
#include <new>
#include <thread>
#include <vector>

#include <cuda_runtime.h>

#include "kvc.h"

namespace {

// DEVICE_STAGED rings: the call's own copy stream and one "copy done" event per slot.
struct StagedCopies {
    bool on = false;
    cudaStream_t stream = nullptr;
    std::vector<cudaEvent_t> done;
    kvc_status start(kvc_ring *ring)
    {
        on = kvc_staging_ring_kind(ring) == KVC_RING_DEVICE_STAGED;
        if (!on)
            return KVC_OK;
        if (cudaStreamCreateWithFlags(&stream, cudaStreamNonBlocking) != cudaSuccess)
            return KVC_ERR_CUDA;
        done.assign(kvc_staging_ring_num_slots(ring), nullptr);
        for (cudaEvent_t &e : done)
            if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess)
                return KVC_ERR_CUDA;
        return KVC_OK;
    }
    // dst <- src on the copy stream, then the slot's "copy done" event
    kvc_status copy(uint32_t slot, void *dst, const void *src, uint64_t bytes, cudaMemcpyKind kind)
    {
        if (cudaMemcpyAsync(dst, src, bytes, kind, stream) != cudaSuccess ||
            cudaEventRecord(done[slot], stream) != cudaSuccess) {
            (void)cudaGetLastError();
            return KVC_ERR_CUDA;
        }
        return KVC_OK;
    }
    ~StagedCopies()
    {
        if (stream)
            cudaStreamSynchronize(stream);
        for (cudaEvent_t e : done)
            if (e)
                cudaEventDestroy(e);
        if (stream)
            cudaStreamDestroy(stream);
    }
};

struct Job {
    uint32_t tag;  // store: chunk index; load: slot index
    uint32_t slot;
    void *host_ptr;
    void *dev_ptr;
    uint64_t bytes, hash;
    kvc_status status;
    bool existed;
    cudaEvent_t copied;  // DEVICE_STAGED store: the event behind the slot's device-to-host copy
};

// A queue of jobs with all its memory taken up front: a job holds a staging slot, so there are never
// more jobs than slots, and neither the calling thread nor an I/O thread (where an allocation
// failure could not be reported) allocates while the pipeline runs.
struct JobQueue {
    std::vector<Job> buf;
    size_t head = 0, count = 0;
    bool empty() const { return count == 0; }
    void push(const Job &j)
    {
        buf[(head + count) % buf.size()] = j;
        ++count;
    }
    Job pop()
    {
        const Job j = buf[head];
        head = (head + 1) % buf.size();
        --count;
        return j;
    }
};

// Work queue for the I/O threads and completion queue back to the calling thread.
struct Queues {
    std::mutex mu;
    std::condition_variable work_cv, done_cv;
    JobQueue work, done;
    bool closing = false;
};

void io_worker(Queues *q, kvc_ring *ring, kvc_store *store, bool storing)
{
    for (;;) {
        Job j;
        {
            std::unique_lock<std::mutex> lk(q->mu);
            q->work_cv.wait(lk, [&] { return q->closing || !q->work.empty(); });
            if (q->closing)
                return;  // jobs still queued are dropped; the caller returns their slots
            j = q->work.pop();
        }
        if (storing) {
            // the slot's copy was only enqueued: wait for its "filled" event (or, for a staged
            // slot, for the copy into its host half), then write the file
            if (j.copied)
                j.status = cudaEventSynchronize(j.copied) == cudaSuccess ? KVC_OK : KVC_ERR_CUDA;
            else
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
            q->done.push(j);
        }
        q->done_cv.notify_one();
    }
}

struct Workers {
    Queues q;
    std::vector<std::thread> threads;
    // Stops the threads after the job each one is running; returns the jobs that never started.
    JobQueue stop()
    {
        JobQueue dropped;
        {
            std::lock_guard<std::mutex> lk(q.mu);
            q.closing = true;
            std::swap(dropped, q.work);  // (moves the buffers: nothing is allocated)
        }
        q.work_cv.notify_all();
        for (std::thread &t : threads)
            if (t.joinable())
                t.join();
        return dropped;
    }
    ~Workers() { (void)stop(); }
};

double now_s()
{
    return std::chrono::duration<double>(std::chrono::steady_clock::now().time_since_epoch()).count();
}

constexpr double kDeadlineSeconds = 600.0;  // every wait in here is bounded

bool start_workers(Workers &w, uint32_t io_threads, kvc_ring *ring, kvc_store *store, bool storing)
{
    const uint32_t n = io_threads ? io_threads : 4;
    try {
        const size_t cap = (size_t)kvc_staging_ring_num_slots(ring) + 1;
        w.q.work.buf.resize(cap);
        w.q.done.buf.resize(cap);
        for (uint32_t i = 0; i < n; ++i)
            w.threads.emplace_back(io_worker, &w.q, ring, store, storing);
    } catch (...) {
        return false;
    }
    return true;
}

void submit(Workers &w, const Job &j)
{
    {
        std::lock_guard<std::mutex> lk(w.q.mu);
        w.q.work.push(j);
    }
    w.q.work_cv.notify_one();
}

// Moves finished jobs out of the completion queue; with block != 0 waits up to 200 ms for one.
void collect(Workers &w, bool block, std::vector<Job> *out)
{
    std::unique_lock<std::mutex> lk(w.q.mu);
    if (block && w.q.done.empty())
        w.q.done_cv.wait_for(lk, std::chrono::milliseconds(200));
    while (!w.q.done.empty())
        out->push_back(w.q.done.pop());
}

// One slot for (cls, key): FIFO order for a plain ring, the slot policy for a pool.
kvc_status take_slot(kvc_ring *ring, bool pool, kvc_slot_class cls, uint64_t key, uint32_t *slot,
                     void **dptr, void **hptr, int *joined)
{
    *joined = 0;
    if (pool)
        return kvc_staging_ring_acquire_for(ring, cls, key, 0, slot, dptr, hptr, joined);
    return kvc_staging_ring_acquire(ring, 0, slot, dptr, hptr);
}

// ------------------------------------------------------------------------------------ store

kvc_status run_store(kvc_layout *lay, kvc_ring *ring, kvc_store *store, const int32_t *ids, uint32_t n_blocks,
                     const uint64_t *hashes, uint32_t n_hashes, uint32_t io_threads, int use_copy_engine,
                     void *stream, kvc_pipeline_stats *out)
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
    const bool pool = kvc_staging_ring_pool_mode(ring) != 0;
    StagedCopies staged;  // destroyed after the workers below: their copies are waited for first
    rc = staged.start(ring);
    if (rc != KVC_OK)
        return rc;
    Workers w;
    if (!start_workers(w, io_threads, ring, store, true))
        return KVC_ERR_NOMEM;

    uint32_t issued = 0, finished = 0;
    kvc_status first_err = KVC_OK;
    std::vector<Job> done;
    done.reserve((size_t)kvc_staging_ring_num_slots(ring) + 1);
    auto reap = [&](bool block) {
        done.clear();
        collect(w, block && finished < issued, &done);
        for (const Job &j : done) {
            ++finished;
            kvc_staging_ring_release_host(ring, j.slot);  // written, or failed: the slot goes back
            if (j.status != KVC_OK) {
                if (first_err == KVC_OK)
                    first_err = j.status;
                continue;
            }
            st.bytes += j.bytes;
            j.existed ? ++st.already_present : ++st.published;
        }
    };

    const double deadline = now_s() + kDeadlineSeconds;
    for (uint32_t c = 0; c < n_chunks && first_err == KVC_OK; ++c) {
        const kvc_chunk_desc &d = descs[c];
        uint32_t slot = 0;
        void *dptr = nullptr, *hptr = nullptr;
        int joined = 0;
        for (;;) {
            reap(false);
            if (first_err != KVC_OK)
                break;
            kvc_status s = take_slot(ring, pool, KVC_CLASS_STORE, hashes[c], &slot, &dptr, &hptr, &joined);
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
                reap(true);  // a slot comes back when one of the jobs in flight completes
            else
                std::this_thread::sleep_for(std::chrono::microseconds(50));  // waiting for a kernel
        }
        if (first_err != KVC_OK)
            break;
        if (joined) {
            // the chunk already sits in the staging memory (another store, a load, or the cache):
            // whoever holds it publishes or has published it; nothing to copy
            kvc_staging_ring_release_host(ring, slot);
            ++st.already_present;
            ++st.chunks;
            continue;
        }
        if (!hptr) {  // the pipelines need slots the host can read and write
            kvc_staging_ring_abandon(ring, slot);
            first_err = KVC_ERR_INVALID_ARG;
            break;
        }
        kvc_status s = use_copy_engine
                           ? kvc_pack_copy_engine(lay, ids + d.first, d.n_blocks, hptr, d.bytes, stream)
                           : kvc_pack(lay, ids + d.first, d.n_blocks, 0, dptr, d.bytes, stream);
        if (s != KVC_OK) {
            kvc_staging_ring_abandon(ring, slot);  // nothing was enqueued into it
            first_err = s;
            break;
        }
        s = kvc_staging_ring_commit(ring, slot, stream);
        if (s != KVC_OK) {
            // the copy is enqueued but the slot cannot be tracked: wait for the copy, then let go
            kvc_staging_ring_commit_host(ring, slot);
            kvc_staging_ring_release(ring, slot, stream);
            first_err = s;
            break;
        }
        Job j = {c, slot, hptr, dptr, d.bytes, hashes[c], KVC_OK, false, nullptr};
        if (staged.on && !use_copy_engine) {
            // device half -> host half once the pack has run; the file is written from the host half
            s = kvc_staging_ring_wait_filled(ring, slot, staged.stream);
            if (s == KVC_OK)
                s = staged.copy(slot, hptr, dptr, d.bytes, cudaMemcpyDeviceToHost);
            if (s != KVC_OK) {
                kvc_staging_ring_sync_filled(ring, slot);
                kvc_staging_ring_release_host(ring, slot);
                first_err = s;
                break;
            }
            j.copied = staged.done[slot];
        }
        submit(w, j);
        ++issued;
        ++st.chunks;
    }
    // Drain.  After an error nothing new starts: jobs not yet picked up are dropped, and their
    // slots go back once the copy that was enqueued into them has run.
    if (first_err != KVC_OK) {
        JobQueue dropped = w.stop();
        reap(false);
        while (!dropped.empty()) {
            const Job j = dropped.pop();
            kvc_staging_ring_sync_filled(ring, j.slot);
            if (j.copied)
                cudaEventSynchronize(j.copied);
            kvc_staging_ring_release_host(ring, j.slot);
            ++finished;
        }
    }
    while (finished < issued && now_s() < deadline)
        reap(true);
    if (finished < issued) {
        // out of time with writes still running: wait for the threads (each finishes its current
        // file), then return what is left
        JobQueue dropped = w.stop();
        reap(false);
        while (!dropped.empty()) {
            const Job j = dropped.pop();
            kvc_staging_ring_sync_filled(ring, j.slot);
            if (j.copied)
                cudaEventSynchronize(j.copied);
            kvc_staging_ring_release_host(ring, j.slot);
            ++finished;
        }
        if (first_err == KVC_OK)
            first_err = KVC_ERR_TIMEOUT;
    }
    st.seconds = now_s() - t0;
    if (out)
        *out = st;
    return first_err;
}

// ------------------------------------------------------------------------------------ load

struct Waiter {
    uint32_t req, chunk;
};

struct SlotWork {
    void *host_ptr = nullptr, *dev_ptr = nullptr;
    uint64_t bytes = 0;
    bool reading = false;  // a read job of this call is in flight for the slot
    std::vector<Waiter> waiters;
};

struct ReqState {
    std::vector<kvc_chunk_desc> descs;
    uint32_t present = 0;  // chunks of the contiguous present prefix
    uint32_t done = 0;     // chunks unpacked (demand) or staged (preload)
};

kvc_status run_load(kvc_layout *lay, kvc_ring *ring, kvc_store *store, kvc_load_request *reqs, uint32_t n_reqs,
                    uint32_t io_threads, int use_copy_engine, void *stream, kvc_load_many_stats *out)
{
    if (!lay || !ring || !store || (!reqs && n_reqs))
        return KVC_ERR_INVALID_ARG;
    kvc_load_many_stats st = {};
    const double t0 = now_s();
    const bool pool = kvc_staging_ring_pool_mode(ring) != 0;
    const uint64_t slot_bytes = kvc_staging_ring_slot_bytes(ring);
    const uint32_t n_slots = kvc_staging_ring_num_slots(ring);
    std::vector<ReqState> rs;
    std::vector<Waiter> pending;  // demand chunks first, then preloads; each class in request order
    std::vector<char> issued;     // per entry of `pending`: has a slot (or has been given up)
    std::map<uint64_t, std::vector<uint32_t>> by_hash;  // entries of `pending` that want the same chunk
    std::vector<SlotWork> slots;
    try {
        rs.resize(n_reqs);
        slots.resize(n_slots);
        for (uint32_t r = 0; r < n_reqs; ++r) {
            kvc_load_request &q = reqs[r];
            q.loaded_chunks = 0;
            q.ready_seconds = 0;
            if (q.cls != KVC_CLASS_DEMAND_LOAD && q.cls != KVC_CLASS_PRELOAD)
                return KVC_ERR_INVALID_ARG;
            if ((!q.ids && q.n_blocks && q.cls == KVC_CLASS_DEMAND_LOAD) || (!q.hashes && q.n_hashes))
                return KVC_ERR_INVALID_ARG;
            if (q.cls == KVC_CLASS_PRELOAD && !pool)
                return KVC_ERR_INVALID_ARG;  // a preload needs somewhere to wait: pool mode only
            uint32_t n_chunks = 0;
            kvc_status rc = kvc_map_request(lay, q.n_blocks, 0, nullptr, 0, &n_chunks);
            if (rc != KVC_OK)
                return rc;
            if (q.n_hashes < n_chunks)
                return KVC_ERR_INVALID_ARG;
            rs[r].descs.resize(n_chunks ? n_chunks : 1);
            rc = kvc_map_request(lay, q.n_blocks, 0, rs[r].descs.data(), n_chunks, &n_chunks);
            if (rc != KVC_OK)
                return rc;
            // only the contiguous prefix of chunks that are present (and of the right size) counts
            uint32_t have = 0;
            for (; have < n_chunks; ++have) {
                if (rs[r].descs[have].bytes > slot_bytes)
                    return KVC_ERR_INVALID_ARG;
                uint64_t sz = 0;
                if (kvc_store_lookup(store, q.hashes[have], &sz) != KVC_OK || sz != rs[r].descs[have].bytes)
                    break;
            }
            rs[r].present = have;
        }
        for (int cls = 0; cls < 2; ++cls)
            for (uint32_t r = 0; r < n_reqs; ++r)
                if ((reqs[r].cls == KVC_CLASS_PRELOAD) == (cls == 1))
                    for (uint32_t c = 0; c < rs[r].present; ++c) {
                        by_hash[reqs[r].hashes[c]].push_back((uint32_t)pending.size());
                        pending.push_back({r, c});
                    }
        issued.assign(pending.size(), 0);
    } catch (const std::bad_alloc &) {
        return KVC_ERR_NOMEM;
    }
    std::vector<std::pair<Waiter, uint32_t>> ready;  // (who, slot) whose bytes are in the slot
    std::vector<Job> done;
    std::vector<kvc_chunk_op> ops;
    try {
        // everything the loop below appends to, at its largest possible size
        ready.reserve(pending.size());
        ops.reserve(pending.size());
        done.reserve((size_t)n_slots + 1);
        size_t most = 1;  // the most requests that can wait for one chunk
        for (const auto &kv : by_hash)
            most = kv.second.size() > most ? kv.second.size() : most;
        for (SlotWork &sw : slots)
            sw.waiters.reserve(most);
    } catch (const std::bad_alloc &) {
        return KVC_ERR_NOMEM;
    }
    StagedCopies staged;
    {
        const kvc_status rc = staged.start(ring);
        if (rc != KVC_OK)
            return rc;
    }
    Workers w;
    if (!start_workers(w, io_threads, ring, store, false))
        return KVC_ERR_NOMEM;

    kvc_status first_err = KVC_OK;
    size_t next = 0;           // next entry of `pending` to issue
    uint32_t reading = 0;      // read jobs in flight
    const double deadline = now_s() + kDeadlineSeconds;
    double preload_refused_since = -1;
    auto note_error = [&](kvc_status s) {
        if (s != KVC_OK && first_err == KVC_OK)
            first_err = s;
    };
    auto finish_one = [&](const Waiter &wt) {
        ReqState &q = rs[wt.req];
        ++q.done;
        reqs[wt.req].loaded_chunks = q.done;
        if (q.done == q.present)
            reqs[wt.req].ready_seconds = now_s() - t0;
        ++st.chunks;
    };

    while (next < pending.size() || reading || !ready.empty()) {
        if (now_s() > deadline) {
            note_error(KVC_ERR_TIMEOUT);
            break;
        }
        // 1. reads that completed: the chunk is staged, everyone waiting for it becomes ready
        collect(w, false, &done);
        for (const Job &j : done) {
            --reading;
            SlotWork &sw = slots[j.slot];
            sw.reading = false;
            kvc_staging_ring_commit_host(ring, j.slot);
            if (j.status != KVC_OK) {
                note_error(j.status);
                for (size_t i = 0; i < sw.waiters.size(); ++i)
                    kvc_staging_ring_release_host(ring, j.slot);
                sw.waiters.clear();
                continue;
            }
            st.bytes_read += j.bytes;
            if (staged.on && !use_copy_engine) {
                // host half -> device half; the unpack stream waits for this copy only
                kvc_status s = staged.copy(j.slot, sw.dev_ptr, sw.host_ptr, j.bytes, cudaMemcpyHostToDevice);
                if (s == KVC_OK && cudaStreamWaitEvent((cudaStream_t)stream, staged.done[j.slot], 0) != cudaSuccess)
                    s = KVC_ERR_CUDA;
                if (s != KVC_OK) {
                    note_error(s);
                    for (size_t i = 0; i < sw.waiters.size(); ++i)
                        kvc_staging_ring_release_host(ring, j.slot);
                    sw.waiters.clear();
                    continue;
                }
            }
            for (const Waiter &wt : sw.waiters)
                ready.push_back({wt, j.slot});
            sw.waiters.clear();
        }
        done.clear();
        if (first_err != KVC_OK)
            break;
        // 2. everything that is ready, of whichever request, in ONE unpack launch
        if (!ready.empty()) {
            ops.clear();
            for (const auto &pr : ready) {
                const Waiter &wt = pr.first;
                if (reqs[wt.req].cls != KVC_CLASS_DEMAND_LOAD)
                    continue;
                const kvc_chunk_desc &d = rs[wt.req].descs[wt.chunk];
                if (use_copy_engine) {
                    note_error(kvc_unpack_copy_engine(lay, slots[pr.second].host_ptr, d.bytes,
                                                      reqs[wt.req].ids + d.first, d.n_blocks, stream));
                } else {
                    kvc_chunk_op op;
                    op.slot = slots[pr.second].dev_ptr;
                    op.ids = reqs[wt.req].ids + d.first;
                    op.n_blocks = d.n_blocks;
                    op.reserved = 0;
                    try {
                        ops.push_back(op);
                    } catch (const std::bad_alloc &) {
                        note_error(KVC_ERR_NOMEM);
                    }
                }
            }
            if (!ops.empty() && first_err == KVC_OK) {
                kvc_status s = kvc_unpack_batch(lay, ops.data(), (uint32_t)ops.size(), 0, stream);
                note_error(s);
                if (s == KVC_OK)
                    ++st.unpack_launches;
            }
            for (const auto &pr : ready) {
                const bool demand = reqs[pr.first.req].cls == KVC_CLASS_DEMAND_LOAD;
                // a demand reference ends when the unpack enqueued above has run; a preload's own
                // reference ends now -- its chunk stays in the slot, unclaimed, for the request
                if (demand && first_err == KVC_OK)
                    note_error(kvc_staging_ring_release(ring, pr.second, stream));
                else
                    kvc_staging_ring_release_host(ring, pr.second);
                if (first_err == KVC_OK)
                    finish_one(pr.first);
            }
            ready.clear();
            if (first_err != KVC_OK)
                break;
        }
        // 3. start what can start, most urgent first.  When a chunk gets a slot, every other
        //    request of this call that wants the same chunk joins it in the same breath, however
        //    far down the list it is: one read and one slot per distinct chunk (Sec. 6.5).
        bool blocked = false;
        while (next < pending.size() && !blocked && first_err == KVC_OK) {
            if (issued[next]) {
                ++next;
                continue;
            }
            const size_t lead = next;
            const uint64_t hash = reqs[pending[lead].req].hashes[pending[lead].chunk];
            const std::vector<uint32_t> *same = nullptr;
            if (pool) {
                auto it = by_hash.find(hash);
                if (it != by_hash.end())
                    same = &it->second;
            }
            const size_t n_same = same ? same->size() : 1;
            for (size_t si = 0; si < n_same + 1 && first_err == KVC_OK && !blocked; ++si) {
                // the leader first, then everybody else who wants this chunk
                const size_t idx = si == 0 ? lead : (same ? (size_t)(*same)[si - 1] : lead);
                if (issued[idx] || (si > 0 && !same))
                    continue;
                const Waiter wt = pending[idx];
                const kvc_load_request &q = reqs[wt.req];
                const kvc_chunk_desc &d = rs[wt.req].descs[wt.chunk];
                uint32_t slot = 0;
                void *dptr = nullptr, *hptr = nullptr;
                int joined = 0;
                kvc_status s = take_slot(ring, pool, (kvc_slot_class)q.cls, hash, &slot, &dptr, &hptr, &joined);
                if (s == KVC_ERR_WOULD_BLOCK) {
                    ++st.ring_stalls;
                    if (q.cls == KVC_CLASS_PRELOAD && reading == 0) {
                        // Nothing of this call is being read and the policy still refuses.  Slots
                        // whose unpack kernels are finishing come back within milliseconds; after
                        // that the reserve (or other users of the pool) leave no room -- preloads
                        // are best effort.
                        if (preload_refused_since < 0) {
                            preload_refused_since = now_s();
                        } else if (now_s() - preload_refused_since > 0.02) {
                            for (size_t k = next; k < pending.size(); ++k)
                                st.preloads_refused += !issued[k];
                            next = pending.size();
                        }
                    }
                    blocked = true;
                    break;
                }
                if (s != KVC_OK) {
                    note_error(s);
                    break;
                }
                preload_refused_since = -1;
                issued[idx] = 1;
                SlotWork &sw = slots[slot];
                sw.dev_ptr = dptr;  // the same for every holder of the slot
                sw.host_ptr = hptr;
                if (joined) {
                    ++st.joins;
                    int filled = 0;
                    kvc_staging_ring_slot_filled(ring, slot, &filled);
                    if (filled) {
                        ready.push_back({wt, slot});
                    } else if (sw.reading) {
                        sw.waiters.push_back(wt);
                    } else {
                        // being filled by somebody outside this call: its completion is not ours to see
                        kvc_staging_ring_release_host(ring, slot);
                        note_error(KVC_ERR_STATE);
                    }
                    continue;
                }
                if (!hptr) {
                    kvc_staging_ring_abandon(ring, slot);
                    note_error(KVC_ERR_INVALID_ARG);
                    break;
                }
                sw.bytes = d.bytes;
                sw.reading = true;
                sw.waiters.clear();
                sw.waiters.push_back(wt);
                Job j = {slot, slot, hptr, dptr, d.bytes, hash, KVC_OK, false, nullptr};
                submit(w, j);
                ++reading;
                ++st.reads;
            }
        }
        if (first_err != KVC_OK)
            break;
        // 4. nothing to do until a read completes or a slot's event fires
        if (ready.empty()) {
            if (reading) {
                collect(w, true, &done);  // handled by step 1 of the next pass
            } else if (blocked) {
                std::this_thread::sleep_for(std::chrono::microseconds(50));  // waiting for a kernel
            }
        }
    }
    if (first_err != KVC_OK) {
        // Error exit: nothing new starts.  Reads that never started give their slots back at once,
        // reads in progress are waited for, and every reference this call still holds is dropped.
        JobQueue dropped = w.stop();
        collect(w, false, &done);
        while (!dropped.empty())
            done.push_back(dropped.pop());
        for (const Job &j : done) {
            SlotWork &sw = slots[j.slot];
            kvc_staging_ring_commit_host(ring, j.slot);
            for (size_t i = 0; i < sw.waiters.size(); ++i)
                kvc_staging_ring_release_host(ring, j.slot);
            sw.waiters.clear();
            sw.reading = false;
        }
        for (const auto &pr : ready)
            kvc_staging_ring_release_host(ring, pr.second);
        ready.clear();
    }
    if (pool) {
        kvc_slot_pool_counters c;
        if (kvc_staging_ring_policy_counters(ring, &c) == KVC_OK)
            st.claims = (uint32_t)c.claims;
    }
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
    // (the bookkeeping containers are sized up front; should an allocation still fail inside, the
    // exception must not cross the C boundary)
    try {
        return run_store(lay, ring, store, ids, n_blocks, hashes, n_hashes, io_threads, use_copy_engine,
                         stream, stats);
    } catch (...) {
        return KVC_ERR_NOMEM;
    }
}

kvc_status kvc_pipeline_load(kvc_layout *lay, kvc_ring *ring, kvc_store *store, const int32_t *ids,
                             uint32_t n_blocks, const uint64_t *hashes, uint32_t n_hashes,
                             uint32_t io_threads, int use_copy_engine, void *stream,
                             kvc_pipeline_stats *stats)
{
    if (!ids && n_blocks)
        return KVC_ERR_INVALID_ARG;
    kvc_load_request q = {};
    q.ids = ids;
    q.n_blocks = n_blocks;
    q.hashes = hashes;
    q.n_hashes = n_hashes;
    q.cls = KVC_CLASS_DEMAND_LOAD;
    kvc_load_many_stats ms = {};
    kvc_status rc;
    try {
        rc = run_load(lay, ring, store, &q, 1, io_threads, use_copy_engine, stream, &ms);
    } catch (...) {
        rc = KVC_ERR_NOMEM;
    }
    if (stats) {
        kvc_pipeline_stats st = {};
        st.bytes = ms.bytes_read;
        st.seconds = ms.seconds;
        st.chunks = ms.chunks;
        st.ring_stalls = ms.ring_stalls;
        *stats = st;
    }
    return rc;
}

kvc_status kvc_pipeline_load_many(kvc_layout *lay, kvc_ring *ring, kvc_store *store, kvc_load_request *reqs,
                                  uint32_t n_reqs, uint32_t io_threads, void *stream,
                                  kvc_load_many_stats *stats)
{
    if (ring && !kvc_staging_ring_pool_mode(ring))
        return KVC_ERR_STATE;
    try {
        return run_load(lay, ring, store, reqs, n_reqs, io_threads, 0, stream, stats);
    } catch (...) {
        return KVC_ERR_NOMEM;
    }
}

}  // extern "C"
