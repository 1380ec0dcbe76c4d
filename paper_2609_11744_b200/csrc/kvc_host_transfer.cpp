// Offload a request to HOST memory and load it back, chunk by chunk through the bounded staging
// ring: the GPU <-> CPU leg of an external KV cache (Sec. 5.1: transfers between paged GPU blocks
// and host buffers at a chosen granularity; Sec. 6.4: every transfer goes through one bounded pool
// of staging slots that are reused only after the event behind their last copy has completed).
//
//   offload : kvc_pack -> slot (kernel stream) -> cudaMemcpyAsync slot -> host (copy stream)
//   load    : cudaMemcpyAsync host -> slot (copy stream) -> kvc_unpack (kernel stream)
//
// The kernels stay in device memory at HBM speed and occupy SMs for microseconds per chunk; the
// copy engines cross the host link.  With a ring of mapped pinned slots the kernels cross the link
// themselves and the copy is host-to-host.  Built from the public entry points of this library
// plus the CUDA runtime for the copies; every exit hands every slot back to the ring.
#include <new>
#include <vector>

#include <cuda_runtime.h>

#include "kvc.h"

namespace {

struct Plan {
    std::vector<kvc_chunk_desc> descs;
    uint32_t n_chunks = 0;
    uint64_t total = 0;
};

kvc_status make_plan(kvc_layout *lay, kvc_ring *ring, const int32_t *ids, uint32_t n_blocks, const void *host,
                     uint64_t host_bytes, int64_t slot_timeout_us, Plan *p)
{
    if (!lay || !ring || (!ids && n_blocks) || (!host && n_blocks) || slot_timeout_us <= 0)
        return KVC_ERR_INVALID_ARG;
    if (kvc_staging_ring_pool_mode(ring))
        return KVC_ERR_STATE;  // slots of a pool are keyed by chunk hash; these calls have none
    kvc_status rc = kvc_map_request(lay, n_blocks, 0, nullptr, 0, &p->n_chunks);
    if (rc != KVC_OK)
        return rc;
    try {
        p->descs.resize(p->n_chunks ? p->n_chunks : 1);
    } catch (const std::bad_alloc &) {
        return KVC_ERR_NOMEM;
    }
    rc = kvc_map_request(lay, n_blocks, 0, p->descs.data(), p->n_chunks, &p->n_chunks);
    if (rc != KVC_OK)
        return rc;
    const uint64_t slot_bytes = kvc_staging_ring_slot_bytes(ring);
    for (uint32_t c = 0; c < p->n_chunks; ++c) {
        if (p->descs[c].bytes > slot_bytes)
            return KVC_ERR_INVALID_ARG;
        p->total += p->descs[c].bytes;
    }
    if (host_bytes < p->total)
        return KVC_ERR_INVALID_ARG;
    return KVC_OK;
}

// The whole block table is checked before anything is enqueued, so that a bad id near the end of a
// long request cannot leave half of it transferred.  `seen` != nullptr also rejects repeated ids.
kvc_status check_ids(kvc_layout *lay, const int32_t *ids, uint32_t n, std::vector<bool> *seen)
{
    const uint32_t nb = kvc_layout_num_blocks(lay);
    if (seen) {
        try {
            seen->assign(nb, false);
        } catch (const std::bad_alloc &) {
            return KVC_ERR_NOMEM;
        }
    }
    for (uint32_t i = 0; i < n; ++i) {
        if (ids[i] < 0 || (uint32_t)ids[i] >= nb)
            return KVC_ERR_OUT_OF_RANGE;
        if (seen) {
            if ((*seen)[(uint32_t)ids[i]])
                return KVC_ERR_CONFLICT;
            (*seen)[(uint32_t)ids[i]] = true;
        }
    }
    return KVC_OK;
}

void fill_stats(kvc_ring *ring, uint64_t stalls0, const Plan &p, uint32_t chunks, uint64_t bytes,
                kvc_host_transfer_stats *out)
{
    if (!out)
        return;
    uint64_t stalls = stalls0;
    kvc_staging_ring_stats(ring, nullptr, nullptr, &stalls);
    out->bytes = bytes;
    out->chunks = chunks;
    out->total_chunks = p.n_chunks;
    out->ring_stalls = stalls - stalls0;
}

}  // namespace

extern "C" {

kvc_status kvc_offload_to_host(kvc_layout *lay, kvc_ring *ring, const int32_t *ids, uint32_t n_blocks,
                               void *host_dst, uint64_t host_bytes, void *kernel_stream, void *copy_stream,
                               int64_t slot_timeout_us, kvc_host_transfer_stats *stats)
{
    if (stats)
        *stats = kvc_host_transfer_stats();
    Plan p;
    kvc_status rc = make_plan(lay, ring, ids, n_blocks, host_dst, host_bytes, slot_timeout_us, &p);
    if (rc != KVC_OK)
        return rc;
    if ((rc = check_ids(lay, ids, n_blocks, nullptr)) != KVC_OK)
        return rc;
    uint64_t stalls0 = 0;
    kvc_staging_ring_stats(ring, nullptr, nullptr, &stalls0);
    const bool mapped = kvc_staging_ring_kind(ring) == KVC_RING_HOST_MAPPED;
    unsigned char *out = static_cast<unsigned char *>(host_dst);
    uint64_t off = 0;
    uint32_t c = 0;
    for (; c < p.n_chunks; ++c) {
        const kvc_chunk_desc &d = p.descs[c];
        uint32_t slot = 0;
        void *dptr = nullptr, *hptr = nullptr;
        if ((rc = kvc_staging_ring_acquire(ring, slot_timeout_us, &slot, &dptr, &hptr)) != KVC_OK)
            break;
        if ((rc = kvc_pack(lay, ids + d.first, d.n_blocks, 0, dptr, d.bytes, kernel_stream)) != KVC_OK) {
            kvc_staging_ring_abandon(ring, slot);  // nothing was enqueued into it
            break;
        }
        if ((rc = kvc_staging_ring_commit(ring, slot, kernel_stream)) != KVC_OK) {
            // the kernel is enqueued but its event is not: mark the slot filled by hand and let it
            // go behind the kernel's own stream
            kvc_staging_ring_commit_host(ring, slot);
            kvc_staging_ring_release(ring, slot, kernel_stream);
            break;
        }
        rc = kvc_staging_ring_wait_filled(ring, slot, copy_stream);
        if (rc == KVC_OK &&
            cudaMemcpyAsync(out + off, mapped ? hptr : dptr, d.bytes, cudaMemcpyDefault,
                            (cudaStream_t)copy_stream) != cudaSuccess) {
            (void)cudaGetLastError();
            rc = KVC_ERR_CUDA;
        }
        // success or not, the slot goes back once everything enqueued on it so far has run
        const kvc_status rel = kvc_staging_ring_release(ring, slot, rc == KVC_OK ? copy_stream : kernel_stream);
        if (rc == KVC_OK)
            rc = rel;
        if (rc != KVC_OK)
            break;
        off += d.bytes;
    }
    fill_stats(ring, stalls0, p, c, off, stats);
    return rc;
}

kvc_status kvc_load_from_host(kvc_layout *lay, kvc_ring *ring, const void *host_src, uint64_t host_bytes,
                              const int32_t *ids, uint32_t n_blocks, void *kernel_stream, void *copy_stream,
                              int64_t slot_timeout_us, kvc_host_transfer_stats *stats)
{
    if (stats)
        *stats = kvc_host_transfer_stats();
    Plan p;
    kvc_status rc = make_plan(lay, ring, ids, n_blocks, host_src, host_bytes, slot_timeout_us, &p);
    if (rc != KVC_OK)
        return rc;
    {
        std::vector<bool> seen;  // a block named twice would be written by two chunks' kernels
        if ((rc = check_ids(lay, ids, n_blocks, &seen)) != KVC_OK)
            return rc;
    }
    uint64_t stalls0 = 0;
    kvc_staging_ring_stats(ring, nullptr, nullptr, &stalls0);
    const bool mapped = kvc_staging_ring_kind(ring) == KVC_RING_HOST_MAPPED;
    const unsigned char *in = static_cast<const unsigned char *>(host_src);
    uint64_t off = 0;
    uint32_t c = 0;
    for (; c < p.n_chunks; ++c) {
        const kvc_chunk_desc &d = p.descs[c];
        uint32_t slot = 0;
        void *dptr = nullptr, *hptr = nullptr;
        if ((rc = kvc_staging_ring_acquire(ring, slot_timeout_us, &slot, &dptr, &hptr)) != KVC_OK)
            break;
        if (cudaMemcpyAsync(mapped ? hptr : dptr, in + off, d.bytes, cudaMemcpyDefault,
                            (cudaStream_t)copy_stream) != cudaSuccess) {
            (void)cudaGetLastError();
            kvc_staging_ring_abandon(ring, slot);  // nothing was enqueued into it
            rc = KVC_ERR_CUDA;
            break;
        }
        if ((rc = kvc_staging_ring_commit(ring, slot, copy_stream)) != KVC_OK) {
            kvc_staging_ring_commit_host(ring, slot);
            kvc_staging_ring_release(ring, slot, copy_stream);
            break;
        }
        rc = kvc_staging_ring_wait_filled(ring, slot, kernel_stream);
        bool unpack_enqueued = false;
        if (rc == KVC_OK) {
            rc = kvc_unpack(lay, dptr, d.bytes, ids + d.first, d.n_blocks, 0, kernel_stream);
            unpack_enqueued = rc == KVC_OK;
        }
        const kvc_status rel = kvc_staging_ring_release(ring, slot, unpack_enqueued ? kernel_stream : copy_stream);
        if (rc == KVC_OK)
            rc = rel;
        if (rc != KVC_OK)
            break;
        off += d.bytes;
    }
    fill_stats(ring, stalls0, p, c, off, stats);
    return rc;
}

}  // extern "C"
