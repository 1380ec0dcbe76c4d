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
// share it and it keeps the previous call's contents: the status words are cleared at the start
// of every call, the tables are overwritten as far as the call needs them, and two calls whose
// GPU work overlaps in time (different streams, or different host threads) race on it.
#include <string.h>

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

constexpr int kMaxDevices = 64;
struct DeviceSetup {
    bool ready;
    unsigned char *scratch;  // device address of kvc_static_scratch on this device
    int sm_count, vec_blocks_per_sm, max_smem_optin;
};
DeviceSetup g_setup[kMaxDevices];

// Host-side staging of the id table (plain static storage; pageable, so the runtime has copied
// it out before cudaMemcpyAsync returns and the next call may overwrite it).
KvcEnt g_host_table[KVC_STATIC_MAX_BLOCKS];

// Once per device, with that device current.
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

    DeviceSetup *dev = nullptr;
    kvc_status s = setup_device(&dev);
    if (s != KVC_OK)
        return s;
    if (!lay->dev_ready) {
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

    uint64_t k = 0;
    for (uint32_t i = 0; i < n_ops; ++i) {
        uint64_t ent_step, plane_step;
        kvc_chunk_steps(lay, ops[i].n_blocks, &ent_step, &plane_step);
        const uint32_t first = (uint32_t)k;
        for (uint32_t j = 0; j < ops[i].n_blocks; ++j, ++k) {
            KvcEnt &e = g_host_table[k];
            e.slot_addr = (uint64_t)(uintptr_t)ops[i].slot + (uint64_t)j * ent_step;
            e.id_or_ptr = (uint64_t)(uint32_t)ops[i].ids[j];
            e.plane_step = plane_step;
            e.nb_c = ops[i].n_blocks;
            e.first_ent = first;
        }
    }
    cudaStream_t st = (cudaStream_t)stream;
    unsigned char *scratch = dev->scratch;
    // status words must start at zero; the tables are rewritten as far as this call reads them
    if (cudaMemsetAsync(scratch, 0, kStatusBytes, st) != cudaSuccess)
        return KVC_ERR_CUDA;
    if (!lay->plane_ptrs.empty() &&
        cudaMemcpyAsync(scratch + kStatusBytes, lay->plane_ptrs.data(),
                        lay->plane_ptrs.size() * sizeof(void *), cudaMemcpyHostToDevice, st) != cudaSuccess)
        return KVC_ERR_CUDA;
    if (cudaMemcpyAsync(scratch + kTableOffset, g_host_table, n_ent * sizeof(KvcEnt),
                        cudaMemcpyHostToDevice, st) != cudaSuccess)
        return KVC_ERR_CUDA;
    a.table = reinterpret_cast<const KvcEnt *>(scratch + kTableOffset);
    a.status = reinterpret_cast<uint32_t *>(scratch);
    a.g.plane_table = lay->plane_ptrs.empty()
                          ? nullptr
                          : reinterpret_cast<const unsigned char *const *>(scratch + kStatusBytes);
    if (kvc_launch_copy(KVC_DIR_PACK, plan.variant, a, plan.grid, plan.smem, st) != cudaSuccess)
        return KVC_ERR_CUDA;
    ++lay->launches;
    return KVC_OK;
}
