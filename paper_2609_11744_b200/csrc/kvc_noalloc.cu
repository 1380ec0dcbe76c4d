// kvc_pack_batch_static: the batched pack for callers that must not allocate.
//
// Some callers cannot reach cudaMalloc when they need to move KV blocks: a serving engine
// that handed all spare device memory to its KV pool at start-up and treats any later
// allocation as a bug, a latency-critical scheduler thread for which the implicit device
// synchronisation of an allocation is unacceptable, or code running inside a memory-pool
// or sandbox layer that forbids raw allocations.  kvc_pack_batch keeps its per-call id table
// (and the handle's status words and plane-pointer table) in memory it allocates on demand.
// This entry point keeps all three in one fixed array that is part of the library image, so
// nothing is allocated or freed, by it or by anything it calls.
//
// The array lives in every device that loads the library until the process exits.  All calls
// share it and it keeps the previous call's contents: the tables are overwritten as far as a
// call needs them, the two status counters start at zero when the library is loaded and are
// cleared by kvc_poll_static_status, and two calls whose GPU work overlaps in time (different
// streams) race on it.
//
// The tables reach the device inside kernel parameters: a tiny kernel stores its own parameter
// block into the array (the plane pointers), or expands the compact chunk records and ids it
// carries into table entries.  A launch copies its parameters before it returns, so the host-side
// staging buffer can be refilled at once, the call never waits for the stream (an asynchronous
// copy from pageable memory would: the runtime documents that it first synchronises the stream
// and returns only when the bytes sit in a driver staging buffer), and no pinned buffer -- which
// would have to be allocated -- is needed.
#include <string.h>

#include <mutex>

#include "kvc_internal.h"

namespace {

constexpr uint32_t kStatusBytes = 256;
constexpr uint32_t kPlaneTableBytes = KVC_STATIC_MAX_PLANES * sizeof(uint64_t);
constexpr uint32_t kTableOffset = kStatusBytes + kPlaneTableBytes;
constexpr uint32_t kScratchBytes = kTableOffset + KVC_STATIC_MAX_BLOCKS * sizeof(KvcEnt);
static_assert(kTableOffset % 256 == 0, "id table must stay 256-byte aligned");

// Device-side scratch.  In host code this name is only a handle for the runtime's symbol
// lookup, never an address a kernel may use: the per-device address comes from
// cudaGetSymbolAddress below.
static __device__ __align__(256) unsigned char kvc_static_scratch[kScratchBytes];

// One parameter block: up to kUploadVecs 16-byte words for scratch[dst_off ...).  Kernel
// parameters may be up to 32,764 bytes on this architecture.
constexpr uint32_t kUploadVecs = 2032;
struct UploadParams {
    uint32_t dst_off;  // byte offset into the scratch array, multiple of 16
    uint32_t n_vecs;
    uint32_t pad[2];
    uint4 data[kUploadVecs];
};
static_assert(sizeof(UploadParams) <= 32764, "parameter block too large");

__global__ void __launch_bounds__(256) kvc_static_upload_kernel(const __grid_constant__ UploadParams p)
{
    uint4 *dst = reinterpret_cast<uint4 *>(kvc_static_scratch + p.dst_off);
    for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < p.n_vecs; i += gridDim.x * blockDim.x)
        dst[i] = p.data[i];
}

// The id table is not shipped entry by entry (32 bytes per block) but in the compact form the
// caller gave it -- one record per chunk and 4 bytes per block id -- and expanded on the device:
// one thread block per chunk writes that chunk's entries.  A parameter block of 32 KiB carries
// about 5000 blocks in 256-token chunks, so a typical call needs one or two of these launches.
struct ChunkRec {
    uint64_t slot;        // chunk base in the staging memory
    uint64_t ent_step;    // bytes between consecutive blocks of a plane inside the chunk
    uint64_t plane_step;  // bytes between consecutive planes of a block inside the chunk
    uint32_t first_ent;   // index of the chunk's first table entry
    uint32_t n_blocks;
    uint32_t ids_off;     // where the chunk's ids start in the id area of this parameter block
    uint32_t pad;
};
static_assert(sizeof(ChunkRec) == 40, "parameter block layout");
constexpr uint32_t kExpandPayload = 32512;  // bytes: ChunkRec[n_chunks], then int32 ids
struct alignas(16) ExpandParams {
    uint32_t n_chunks;
    uint32_t ids_at;  // byte offset of the id area inside payload (8-byte aligned)
    uint32_t pad[2];
    unsigned char payload[kExpandPayload];
};
static_assert(sizeof(ExpandParams) <= 32764, "parameter block too large");

__global__ void __launch_bounds__(128) kvc_static_expand_kernel(const __grid_constant__ ExpandParams p)
{
    const ChunkRec c = reinterpret_cast<const ChunkRec *>(p.payload)[blockIdx.x];
    const int32_t *ids = reinterpret_cast<const int32_t *>(p.payload + p.ids_at) + c.ids_off;
    KvcEnt *table = reinterpret_cast<KvcEnt *>(kvc_static_scratch + kTableOffset);
    for (uint32_t j = threadIdx.x; j < c.n_blocks; j += blockDim.x) {
        KvcEnt e;
        e.slot_addr = c.slot + (uint64_t)j * c.ent_step;
        e.id_or_ptr = (uint64_t)(uint32_t)ids[j];
        e.plane_step = c.plane_step;
        e.nb_c = c.n_blocks;
        e.first_ent = c.first_ent;
        table[c.first_ent + j] = e;
    }
}

constexpr int kMaxDevices = 64;
struct DeviceSetup {
    bool ready;
    unsigned char *scratch;  // device address of kvc_static_scratch on this device
    int sm_count, vec_blocks_per_sm, max_smem_optin;
};
// All host-side state of this file is guarded by one mutex; the call is far off any hot path.
std::mutex g_mu;
DeviceSetup g_setup[kMaxDevices];
UploadParams g_params;        // host-side staging of one parameter block
ExpandParams g_expand;        // ... and of one compact table block
uint32_t g_host_status[2];    // landing place of kvc_poll_static_status

// Once per device, with that device current.  Caller holds g_mu.
kvc_status setup_device(DeviceSetup **out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) {
        (void)cudaGetLastError();
        return KVC_ERR_CUDA;
    }
    if (dev < 0 || dev >= kMaxDevices)
        return KVC_ERR_INVALID_ARG;
    DeviceSetup &d = g_setup[dev];
    if (!d.ready) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, kvc_static_scratch) != cudaSuccess || p == nullptr) {
            (void)cudaGetLastError();
            return KVC_ERR_CUDA;
        }
        if (kvc_kernel_limits(&d.sm_count, &d.vec_blocks_per_sm, &d.max_smem_optin) != cudaSuccess) {
            (void)cudaGetLastError();
            return KVC_ERR_CUDA;
        }
        if (d.vec_blocks_per_sm < 1)
            d.vec_blocks_per_sm = 1;
        d.scratch = static_cast<unsigned char *>(p);
        d.ready = true;
    }
    *out = &d;
    return KVC_OK;
}

// scratch[dst_off, dst_off + bytes) = src, through kernel parameters.  bytes % 16 == 0.
kvc_status upload(uint32_t dst_off, const void *src, uint64_t bytes, cudaStream_t st)
{
    const unsigned char *p = static_cast<const unsigned char *>(src);
    while (bytes) {
        const uint32_t n = (uint32_t)(bytes < kUploadVecs * 16ull ? bytes : kUploadVecs * 16ull);
        g_params.dst_off = dst_off;
        g_params.n_vecs = n / 16;
        memcpy(g_params.data, p, n);
        kvc_static_upload_kernel<<<(g_params.n_vecs + 255) / 256, 256, 0, st>>>(g_params);
        if (cudaGetLastError() != cudaSuccess)
            return KVC_ERR_CUDA;
        p += n;
        dst_off += n;
        bytes -= n;
    }
    return KVC_OK;
}

}  // namespace

extern "C" kvc_status kvc_pack_batch_static(kvc_layout *lay, const kvc_chunk_op *ops, uint32_t n_ops,
                                            void *stream)
{
    if (!lay || (!ops && n_ops))
        return KVC_ERR_INVALID_ARG;
    uint64_t n_ent = 0;
    const void *probe = nullptr;
    for (uint32_t i = 0; i < n_ops; ++i) {
        if (ops[i].reserved != 0)
            return KVC_ERR_INVALID_ARG;
        if (ops[i].n_blocks == 0)
            continue;
        if (!ops[i].slot || !ops[i].ids)
            return KVC_ERR_INVALID_ARG;
        if (((uintptr_t)ops[i].slot & 15u) != 0)
            return KVC_ERR_ALIGNMENT;
        if (!probe || ((uintptr_t)ops[i].slot % 32) != 0)
            probe = ops[i].slot;
        n_ent += ops[i].n_blocks;
    }
    if (n_ent == 0)
        return KVC_OK;
    if (n_ent > KVC_STATIC_MAX_BLOCKS || lay->plane_ptrs.size() > KVC_STATIC_MAX_PLANES)
        return KVC_ERR_TOO_LARGE;
    // ids are host-resident: check them all before anything is enqueued (pack may repeat ids)
    for (uint32_t i = 0; i < n_ops; ++i)
        for (uint32_t j = 0; j < ops[i].n_blocks; ++j)
            if (ops[i].ids[j] < 0 || (uint32_t)ops[i].ids[j] >= lay->d.num_blocks)
                return KVC_ERR_OUT_OF_RANGE;

    std::lock_guard<std::mutex> lock(g_mu);
    DeviceSetup *dev = nullptr;
    kvc_status s = setup_device(&dev);
    if (s != KVC_OK)
        return s;
    if (lay->dev_ready) {
        // a handle belongs to the device of its first launch: its pool pointers mean nothing elsewhere
        if (&g_setup[lay->device] != dev)
            return KVC_ERR_INVALID_ARG;
    } else {
        // the planner reads the device limits from the handle; fill them without allocating
        lay->sm_count = dev->sm_count;
        lay->vec_blocks_per_sm = dev->vec_blocks_per_sm;
        lay->max_smem_optin = dev->max_smem_optin;
    }
    KvcLaunch a;
    memset(&a, 0, sizeof(a));
    KvcPlan plan;
    s = kvc_make_plan(lay, n_ent, probe, &a, &plan);
    if (s != KVC_OK)
        return s;

    cudaStream_t st = (cudaStream_t)stream;
    if (!lay->plane_ptrs.empty()) {
        // 8-byte pointers, 16-byte words: an odd count carries one word of padding
        static uint64_t planes[KVC_STATIC_MAX_PLANES + 1];
        const size_t n = lay->plane_ptrs.size();
        for (size_t i = 0; i < n; ++i)
            planes[i] = (uint64_t)(uintptr_t)lay->plane_ptrs[i];
        planes[n] = 0;
        s = upload(kStatusBytes, planes, ((n + 1) / 2) * 16, st);
        if (s != KVC_OK)
            return s;
    }
    // the id table, in compact form: as many whole chunks per parameter block as fit
    {
        uint64_t k = 0;     // table entries described so far
        uint32_t i = 0;     // next op
        while (i < n_ops) {
            // how many ops fit: 40 bytes per chunk record + 4 bytes per id (+ alignment slack)
            uint32_t n_c = 0, n_ids = 0, j = i;
            for (; j < n_ops; ++j) {
                if (ops[j].n_blocks == 0)
                    continue;
                const uint64_t need = (uint64_t)(n_c + 1) * sizeof(ChunkRec) + 8 +
                                      (uint64_t)(n_ids + ops[j].n_blocks) * sizeof(int32_t);
                if (need > kExpandPayload)
                    break;
                ++n_c;
                n_ids += ops[j].n_blocks;
            }
            if (n_c == 0) {
                if (j >= n_ops)
                    break;  // only empty ops were left
                // a single chunk with more ids than one parameter block holds: ship its entries
                // ready-made, 32 bytes each, through the plain upload path
                static KvcEnt ents[kUploadVecs / 2];
                uint64_t ent_step, plane_step;
                kvc_chunk_steps(lay, ops[j].n_blocks, &ent_step, &plane_step);
                const uint32_t first = (uint32_t)k;
                uint32_t filled = 0, base = first;
                for (uint32_t b = 0; b < ops[j].n_blocks; ++b) {
                    KvcEnt &e = ents[filled++];
                    e.slot_addr = (uint64_t)(uintptr_t)ops[j].slot + (uint64_t)b * ent_step;
                    e.id_or_ptr = (uint64_t)(uint32_t)ops[j].ids[b];
                    e.plane_step = plane_step;
                    e.nb_c = ops[j].n_blocks;
                    e.first_ent = first;
                    if (filled == kUploadVecs / 2 || b + 1 == ops[j].n_blocks) {
                        s = upload(kTableOffset + base * (uint32_t)sizeof(KvcEnt), ents,
                                   (uint64_t)filled * sizeof(KvcEnt), st);
                        if (s != KVC_OK)
                            return s;
                        base += filled;
                        filled = 0;
                    }
                }
                k += ops[j].n_blocks;
                i = j + 1;
                continue;
            }
            g_expand.n_chunks = n_c;
            g_expand.ids_at = (uint32_t)((n_c * sizeof(ChunkRec) + 7u) & ~7u);
            ChunkRec *recs = reinterpret_cast<ChunkRec *>(g_expand.payload);
            int32_t *ids_area = reinterpret_cast<int32_t *>(g_expand.payload + g_expand.ids_at);
            uint32_t c = 0, ids_off = 0;
            for (; i < j; ++i) {
                if (ops[i].n_blocks == 0)
                    continue;
                ChunkRec &r = recs[c++];
                r.slot = (uint64_t)(uintptr_t)ops[i].slot;
                kvc_chunk_steps(lay, ops[i].n_blocks, &r.ent_step, &r.plane_step);
                r.first_ent = (uint32_t)k;
                r.n_blocks = ops[i].n_blocks;
                r.ids_off = ids_off;
                r.pad = 0;
                memcpy(ids_area + ids_off, ops[i].ids, (size_t)ops[i].n_blocks * sizeof(int32_t));
                ids_off += ops[i].n_blocks;
                k += ops[i].n_blocks;
            }
            kvc_static_expand_kernel<<<n_c, 128, 0, st>>>(g_expand);
            if (cudaGetLastError() != cudaSuccess)
                return KVC_ERR_CUDA;
        }
    }
    unsigned char *scratch = dev->scratch;
    a.table = reinterpret_cast<const KvcEnt *>(scratch + kTableOffset);
    a.status = reinterpret_cast<uint32_t *>(scratch);
    a.g.plane_table = lay->plane_ptrs.empty()
                          ? nullptr
                          : reinterpret_cast<const unsigned char *const *>(scratch + kStatusBytes);
    // The copy kernel reads the tables through the read-only data path, so it must not become
    // resident while the upload kernels are still writing them: plain stream order, no
    // programmatic overlap with the preceding kernel.
    a.pdl = 0;
    // (kvc_launch_copy directly: the timing diagnostic of the handle creates events, this path must not)
    if (kvc_launch_copy(KVC_DIR_PACK, plan.variant, a, plan.grid, plan.smem, st) != cudaSuccess)
        return KVC_ERR_CUDA;
    ++lay->launches;
    return KVC_OK;
}

extern "C" kvc_status kvc_poll_static_status(void *stream, uint32_t *n_skipped, uint32_t *n_wait_expired)
{
    if (n_skipped)
        *n_skipped = 0;
    if (n_wait_expired)
        *n_wait_expired = 0;
    std::lock_guard<std::mutex> lock(g_mu);
    DeviceSetup *dev = nullptr;
    kvc_status s = setup_device(&dev);
    if (s != KVC_OK)
        return s;
    cudaStream_t st = (cudaStream_t)stream;
    // device -> pageable host: the runtime returns only when the bytes have arrived
    if (cudaMemcpyAsync(g_host_status, dev->scratch, sizeof(g_host_status), cudaMemcpyDeviceToHost,
                        st) != cudaSuccess ||
        cudaMemsetAsync(dev->scratch, 0, sizeof(g_host_status), st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess) {
        (void)cudaGetLastError();
        return KVC_ERR_CUDA;
    }
    if (n_skipped)
        *n_skipped = g_host_status[0];
    if (n_wait_expired)
        *n_wait_expired = g_host_status[1];
    return KVC_OK;
}
