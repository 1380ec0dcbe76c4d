// Host side of libkvc: layout descriptor (Sec. 2.1), block-table -> chunk mapper (Sec. 6.4,
// shared prefixes Sec. 6.5), argument validation and the launch front ends of pack / unpack.
#include <string.h>

#include <algorithm>
#include <map>
#include <new>
#include <utility>

#include "kvc_internal.h"

namespace {

inline bool mult16(uint64_t v) { return (v & 15u) == 0; }

kvc_status ensure_device(kvc_layout *lay)
{
    if (lay->dev_ready) {
        // a handle belongs to the device that was current at its first launch
        int dev = -1;
        if (cudaGetDevice(&dev) != cudaSuccess)
            return KVC_ERR_CUDA;
        return dev == lay->device ? KVC_OK : KVC_ERR_INVALID_ARG;
    }
    if (cudaGetDevice(&lay->device) != cudaSuccess)
        return KVC_ERR_CUDA;
    if (kvc_kernel_limits(&lay->sm_count, &lay->vec_blocks_per_sm, &lay->max_smem_optin) !=
        cudaSuccess) {
        (void)cudaGetLastError();
        return KVC_ERR_CUDA;
    }
    if (lay->vec_blocks_per_sm < 1)
        lay->vec_blocks_per_sm = 1;
    if (cudaMalloc(&lay->d_status, 2 * sizeof(uint32_t)) != cudaSuccess)
        return KVC_ERR_NOMEM;
    if (cudaMemset(lay->d_status, 0, 2 * sizeof(uint32_t)) != cudaSuccess)
        return KVC_ERR_CUDA;
    if (cudaHostAlloc(&lay->h_status, 2 * sizeof(uint32_t), cudaHostAllocDefault) != cudaSuccess)
        return KVC_ERR_NOMEM;
    if (cudaStreamCreateWithFlags(&lay->upload_stream, cudaStreamNonBlocking) != cudaSuccess ||
        cudaEventCreateWithFlags(&lay->upload_done, cudaEventDisableTiming) != cudaSuccess)
        return KVC_ERR_CUDA;
    if (!lay->plane_ptrs.empty()) {
        size_t bytes = lay->plane_ptrs.size() * sizeof(void *);
        if (cudaMalloc(&lay->d_plane_table, bytes) != cudaSuccess)
            return KVC_ERR_NOMEM;
        if (cudaMemcpy(lay->d_plane_table, lay->plane_ptrs.data(), bytes, cudaMemcpyHostToDevice) !=
            cudaSuccess)
            return KVC_ERR_CUDA;
    }
    lay->dev_ready = true;
    return KVC_OK;
}

}  // namespace

// Fills the geometry and the launch shape that do not depend on the ids.
kvc_status kvc_make_plan(kvc_layout *lay, uint64_t n_ent, const void *slot_probe, KvcLaunch *a,
                         KvcPlan *plan)
{
    const kvc_tuning &t = lay->tuning;
    KvcGeom &g = a->g;
    g.base = static_cast<const unsigned char *>(lay->d.base);
    g.layer_stride = lay->d.layer_stride;
    g.plane_stride = lay->d.plane_stride;
    g.plane_table = lay->d_plane_table;
    g.block_stride = lay->block_stride;
    g.slab_bytes = (uint32_t)lay->slab_bytes;
    g.planes_total = lay->planes_total;
    g.planes_per_layer = lay->d.kv_planes;
    g.num_blocks = lay->d.num_blocks;

    int variant = t.variant ? (int)t.variant : KVC_VARIANT_BULK;
    bool host_slot = false;
    if (variant == KVC_VARIANT_BULK) {
        // Bulk copies are used for device memory only; a slot in mapped host memory is
        // written with ordinary vector stores.
        bool device_slot = t.slot_memory == 1;
        if (t.slot_memory == 0) {
            cudaPointerAttributes attr;
            if (cudaPointerGetAttributes(&attr, slot_probe) != cudaSuccess) {
                (void)cudaGetLastError();
                return KVC_ERR_CUDA;
            }
            device_slot = attr.type == cudaMemoryTypeDevice;
        }
        if (!device_slot) {
            variant = KVC_VARIANT_VEC;
            host_slot = true;
        }
    }
    // Two launch shapes.  Streaming (the default): many short-lived blocks, each taking a few
    // consecutive work items, handed out by the hardware scheduler as SMs free up -- measured
    // 2-4 % faster than a persistent grid because it balances itself and throttles the bytes in
    // flight, and several such launches on different streams share the SMs well (per-chunk
    // launches rotated over 4 streams reach the batched rate; with persistent grids they lose
    // 10 %).  Persistent: a fixed, small number of blocks that stride over all items, used when
    // the caller caps the blocks (to leave SMs to a compute stream) or the slot is host memory.
    const bool persistent = t.max_ctas != 0 || host_slot;
    uint32_t tile = t.tile_bytes;
    if (tile == 0)
        tile = (variant == KVC_VARIANT_BULK || !persistent) ? 32768u : 16384u;
    const bool small_vec_blocks = variant != KVC_VARIANT_BULK && t.vec_threads && t.vec_threads < KVC_VEC_THREADS;
    if (small_vec_blocks)  // blocks of fewer than 256 threads exist for the one-warp-per-tile kernels only
        tile = std::min<uint32_t>(tile, KVC_VEC_WARP_TEAM_MAX_TILE);
    tile = (uint32_t)std::min<uint64_t>(tile, lay->slab_bytes);
    uint32_t stages = 0, lag = 0, smem = 0, group_shift = 0;
    if (variant == KVC_VARIANT_BULK) {
        const uint32_t per_sm = t.ctas_per_sm ? t.ctas_per_sm
                                              : (persistent ? 1u : KVC_BULK_STREAMING_BLOCKS_PER_SM);
        // every resident block also costs 1 KiB of system-reserved shared memory
        // (the larger header of the multi-slab kernel is assumed for either kernel)
        const uint32_t room = ((uint32_t)lay->max_smem_optin + 1024u) / per_sm - 1024u -
                              KVC_GROUP_SMEM_HEADER(KVC_BULK_MAX_STAGES);
        if (tile > room / 2)
            tile = (room / 2) & ~15u;
        // Several slabs per work item: the largest power of two of whole slabs that fits the tile,
        // by default at most 16 slabs and (below 4 KiB slabs) at most 16 KiB.  Measured on B200 with
        // 2 GiB requests and slabs of 256 B to 4 KiB: items of 16 slabs in two stages per block
        // reach 6.3-6.7 TB/s, because the small footprint lets ~10-24 one-warp blocks share an SM
        // and their table lookups overlap; 32 KiB items (three blocks per SM) fall to 2.6-6.0 TB/s
        // below 2 KiB slabs, and so do more than two stages.
        const uint32_t def_cap = lay->slab_bytes >= 4096u ? 32768u : 16384u;
        const uint32_t tile_cap = std::min<uint32_t>(t.tile_bytes ? t.tile_bytes : def_cap, (room / 2) & ~15u);
        const uint32_t want_group = t.group & ~KVC_GROUP_FORCE_KERNEL;
        uint32_t group = 1;
        if (want_group != 1 && lay->slab_bytes <= tile_cap) {
            const uint32_t cap = std::min<uint32_t>(want_group ? want_group : KVC_GROUP_DEFAULT_SLABS,
                                                    (uint32_t)(tile_cap / lay->slab_bytes));
            while (group * 2 <= cap) {
                group *= 2;
                ++group_shift;
            }
        }
        const bool grouped = (group > 1 || (t.group & KVC_GROUP_FORCE_KERNEL)) && lay->slab_bytes <= tile_cap;
        if (grouped) {
            variant = KVC_VARIANT_BULK_GROUP;
            tile = group * (uint32_t)lay->slab_bytes;
        }
        const uint32_t def_stages = persistent ? KVC_BULK_DEFAULT_STAGES : KVC_BULK_STREAMING_STAGES;
        stages = t.stages ? t.stages : def_stages;
        stages = std::min<uint32_t>(std::min<uint32_t>(stages, room / tile), KVC_BULK_MAX_STAGES);
        if (stages < 2)
            return KVC_ERR_INVALID_ARG;
        // a stage is reloaded only when at most `pending` newer stores still read shared memory,
        // so loads can run at most stages-2 items ahead of the stores
        lag = stages - 2;
        const uint32_t want_lag = t.lag ? t.lag
                                        : (grouped ? std::max<uint32_t>(1u, stages / 2 - 1) : KVC_BULK_DEFAULT_LAG);
        if (want_lag < lag)
            lag = want_lag;
        smem = (grouped ? KVC_GROUP_SMEM_HEADER(stages) : KVC_BULK_SMEM_HEADER) + stages * tile;
    } else {
        // 32-byte vectors need every address the kernel forms to be 32-byte aligned
        bool a32 = (lay->slab_bytes % 32 == 0) && (tile % 32 == 0) && (lay->block_stride % 32 == 0) &&
                   ((uintptr_t)slot_probe % 32 == 0);
        if (lay->plane_ptrs.empty()) {
            a32 = a32 && ((uintptr_t)lay->d.base % 32 == 0) && (lay->d.layer_stride % 32 == 0) &&
                  (lay->d.plane_stride % 32 == 0);
        } else {
            for (const void *p : lay->plane_ptrs)
                a32 = a32 && ((uintptr_t)p % 32 == 0);
        }
        variant = a32 ? (int)KVC_VARIANT_VEC32 : (int)KVC_VARIANT_VEC;
        // small slabs: several per work item, one warp per item
        const uint32_t want_group = t.group & ~KVC_GROUP_FORCE_KERNEL;
        if (want_group != 1 && lay->slab_bytes <= KVC_VEC_GROUP_MAX_SLAB && t.tile_bytes == 0) {
            const uint32_t cap = std::min<uint32_t>(want_group ? want_group : KVC_GROUP_MAX_SLABS,
                                                    (uint32_t)(KVC_VEC_GROUP_ITEM_BYTES / lay->slab_bytes));
            uint32_t group = 1;
            while (group * 2 <= cap) {
                group *= 2;
                ++group_shift;
            }
            variant = a32 ? (int)KVC_VARIANT_VEC32_GROUP : (int)KVC_VARIANT_VEC_GROUP;
            tile = group * (uint32_t)lay->slab_bytes;
            a->vec_magic = (1ull << 32) / (lay->slab_bytes / (a32 ? 32u : 16u)) + 1ull;
        }
    }
    g.tile_bytes = tile;
    const bool vec_grouped = variant == KVC_VARIANT_VEC_GROUP || variant == KVC_VARIANT_VEC32_GROUP;
    const bool grouped = variant == KVC_VARIANT_BULK_GROUP || vec_grouped;
    g.parts = grouped ? 1u : (uint32_t)((lay->slab_bytes + tile - 1) / tile);
    const uint64_t n_slabs = n_ent * lay->planes_total;
    const uint64_t n_items = grouped ? (n_slabs + (1u << group_shift) - 1) >> group_shift : n_slabs * g.parts;
    if (n_items == 0 || n_items > 0xFFFFFFFFull || n_slabs > 0xFFFFFFFFull)
        return KVC_ERR_INVALID_ARG;
    a->n_slabs = n_slabs;
    a->vec_threads = small_vec_blocks ? t.vec_threads : 0;
    a->group_shift = group_shift;
    // stores that may still be reading shared memory when a stage is reloaded: the stage's last
    // store is stages-lag groups back, so everything newer than that may stay outstanding
    a->pending = stages >= 2 + lag ? std::min<uint32_t>(stages - 1 - lag, 7u) : 1u;
    a->n_items = n_items;
    a->n_ent = (uint32_t)n_ent;
    a->order = t.order ? t.order : KVC_ORDER_CHUNK_MAJOR;
    a->block_major_chunks = lay->d.chunk_order == KVC_CHUNK_BLOCK_MAJOR;
    a->stages = stages;
    a->lag = lag;
    // bit 0: loads, bit 1: stores
    a->l2_evict_first = t.l2_hint == 2 ? 3u : t.l2_hint == 3 ? 1u : t.l2_hint == 4 ? 2u : 0u;
    // 0 = plain launch, 1 = programmatic dependent launch, 2 = the same without waiting for the
    // previous kernel (only where the launch reads nothing a kernel could have written: the
    // batched calls read a table that an asynchronous copy delivers, which is ordered by an event)
    a->pdl = t.pdl == 1 ? 0u : (t.pdl == 3 ? 2u : 1u);
    a->status = lay->d_status;
    uint64_t grid;
    if (t.max_ctas) {
        grid = t.max_ctas;
    } else if (host_slot) {
        // a slot in host memory is bound by the host link: 16 blocks saturate it (measured), more
        // would only hold SMs while they wait for the link
        grid = KVC_HOST_SLOT_DEFAULT_CTAS;
    } else {
        // streaming: about 64 KiB (bulk) or 32 KiB (vector) of items per block
        uint32_t per_block = t.items_per_cta;
        if (vec_grouped) {
            // one item per warp at a time: a block of 8 warps takes 8 * items_per_cta items
            // (default 16 per warp, about 1 MiB per block: measured 3-5 % faster than 4)
            const uint32_t warps = (a->vec_threads ? a->vec_threads : KVC_VEC_THREADS) / 32u;
            per_block = warps * (per_block ? per_block : 16u);
        } else if (per_block == 0) {
            const bool bulk = variant == KVC_VARIANT_BULK || variant == KVC_VARIANT_BULK_GROUP;
            const uint32_t bytes = bulk ? 65536u : 32768u;
            per_block = std::max<uint32_t>(bulk ? 2u : 1u, bytes / tile);
        }
        grid = (n_items + per_block - 1) / per_block;
    }
    grid = std::min<uint64_t>(std::min<uint64_t>(grid, n_items), 0x7FFFFFFFull);
    plan->variant = variant;
    plan->grid = (uint32_t)grid;
    plan->smem = smem;
    plan->stages = stages;
    plan->lag = lag;
    return KVC_OK;
}

kvc_status kvc_launch_timed(kvc_layout *lay, int dir, int variant, const KvcLaunch &a, uint32_t grid,
                            uint32_t smem, cudaStream_t st)
{
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    // on a failure the events taken for this launch are destroyed, not leaked
    auto fail = [&](kvc_status s) {
        (void)cudaGetLastError();
        if (e0)
            cudaEventDestroy(e0);
        if (e1)
            cudaEventDestroy(e1);
        return s;
    };
    if (lay->time_kernels) {
        cudaEvent_t *ev[2] = {&e0, &e1};
        for (cudaEvent_t *e : ev) {
            if (!lay->spare_events.empty()) {
                *e = lay->spare_events.back();
                lay->spare_events.pop_back();
            } else if (cudaEventCreate(e) != cudaSuccess) {
                *e = nullptr;
                return fail(KVC_ERR_CUDA);
            }
        }
        try {
            lay->timed.reserve(lay->timed.size() + 1);
        } catch (const std::bad_alloc &) {
            return fail(KVC_ERR_NOMEM);
        }
        if (cudaEventRecord(e0, st) != cudaSuccess)
            return fail(KVC_ERR_CUDA);
    }
    if (kvc_launch_copy(dir, variant, a, grid, smem, st) != cudaSuccess)
        return fail(KVC_ERR_CUDA);
    if (lay->time_kernels) {
        if (cudaEventRecord(e1, st) != cudaSuccess)
            return fail(KVC_ERR_CUDA);
        lay->timed.emplace_back(e0, e1);  // room was reserved above
    }
    ++lay->launches;
    return KVC_OK;
}

namespace {

// Range check, and for unpack a duplicate check across the whole call, on host-resident ids.
kvc_status check_host_ids(kvc_layout *lay, const int32_t *ids, uint32_t n, bool reject_dup)
{
    const uint32_t nb = lay->d.num_blocks;
    for (uint32_t j = 0; j < n; ++j)
        if (ids[j] < 0 || (uint32_t)ids[j] >= nb)
            return KVC_ERR_OUT_OF_RANGE;
    if (reject_dup) {
        for (uint32_t j = 0; j < n; ++j) {
            uint32_t &s = lay->seen[(uint32_t)ids[j]];
            if (s == lay->seen_stamp)
                return KVC_ERR_CONFLICT;
            s = lay->seen_stamp;
        }
    }
    return KVC_OK;
}

void begin_dup_scope(kvc_layout *lay)
{
    if (lay->seen.size() != lay->d.num_blocks)
        lay->seen.assign(lay->d.num_blocks, 0);
    if (++lay->seen_stamp == 0) {  // stamp wrapped: clear and restart
        std::fill(lay->seen.begin(), lay->seen.end(), 0u);
        lay->seen_stamp = 1;
    }
}

kvc_status copy_one(kvc_layout *lay, int dir, const int32_t *ids, uint32_t n_blocks,
                    int ids_on_device, void *slot, uint64_t slot_bytes, void *stream)
{
    if (!lay || (!ids && n_blocks) || (!slot && n_blocks))
        return KVC_ERR_INVALID_ARG;
    if (n_blocks == 0)
        return KVC_OK;
    const uint64_t need = kvc_layout_chunk_bytes(lay, n_blocks);
    if (slot_bytes < need)
        return KVC_ERR_INVALID_ARG;
    if (!mult16((uintptr_t)slot))
        return KVC_ERR_ALIGNMENT;
    if (!ids_on_device) {
        if (dir == KVC_DIR_UNPACK) {  // only unpack looks for repeated ids
            try {
                begin_dup_scope(lay);
            } catch (const std::bad_alloc &) {
                return KVC_ERR_NOMEM;
            }
        }
        kvc_status s = check_host_ids(lay, ids, n_blocks, dir == KVC_DIR_UNPACK);
        if (s != KVC_OK)
            return s;
        if (n_blocks > KVC_PARAM_IDS) {
            // too many ids for the kernel parameters: go through the table path
            kvc_chunk_op op;
            op.slot = slot;
            op.ids = ids;
            op.n_blocks = n_blocks;
            op.reserved = 0;
            return dir == KVC_DIR_PACK ? kvc_pack_batch(lay, &op, 1, 0, stream)
                                       : kvc_unpack_batch(lay, &op, 1, 0, stream);
        }
    }
    kvc_status s = ensure_device(lay);
    if (s != KVC_OK)
        return s;
    KvcLaunch a;
    memset(&a, 0, sizeof(a));
    KvcPlan plan;
    s = kvc_make_plan(lay, n_blocks, slot, &a, &plan);
    if (s != KVC_OK)
        return s;
    a.slot = (uint64_t)(uintptr_t)slot;
    kvc_chunk_steps(lay, n_blocks, &a.ent_step, &a.plane_step);
    if (ids_on_device)
        a.dev_ids = ids;
    else
        memcpy(a.ids, ids, n_blocks * sizeof(int32_t));
    return kvc_launch_timed(lay, dir, plan.variant, a, plan.grid, plan.smem, (cudaStream_t)stream);
}

// Picks the next table arena, waiting (on the host) for the kernel that last read it.
kvc_status take_arena(kvc_layout *lay, uint64_t n_ent, KvcArena **out)
{
    KvcArena &ar = lay->arenas[lay->next_arena];
    lay->next_arena = (lay->next_arena + 1) % KVC_NUM_ARENAS;
    if (ar.busy) {
        if (cudaEventSynchronize(ar.done) != cudaSuccess)
            return KVC_ERR_CUDA;
        ar.busy = false;
    }
    if (!ar.done && cudaEventCreateWithFlags(&ar.done, cudaEventDisableTiming) != cudaSuccess)
        return KVC_ERR_CUDA;
    if (ar.cap < n_ent) {
        if (ar.host)
            cudaFreeHost(ar.host);
        if (ar.dev)
            cudaFree(ar.dev);
        ar.host = nullptr;
        ar.dev = nullptr;
        ar.cap = 0;
        uint64_t cap = std::max<uint64_t>(n_ent, 4096);
        if (cudaHostAlloc(&ar.host, cap * sizeof(KvcEnt), cudaHostAllocDefault) != cudaSuccess) {
            (void)cudaGetLastError();
            ar.host = nullptr;
            return KVC_ERR_NOMEM;
        }
        if (cudaMalloc(&ar.dev, cap * sizeof(KvcEnt)) != cudaSuccess) {
            (void)cudaGetLastError();
            cudaFreeHost(ar.host);
            ar.host = nullptr;
            ar.dev = nullptr;
            return KVC_ERR_NOMEM;
        }
        ar.cap = cap;
    }
    *out = &ar;
    return KVC_OK;
}

kvc_status copy_batch(kvc_layout *lay, int dir, const kvc_chunk_op *ops, uint32_t n_ops,
                      int ids_on_device, void *stream)
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
        if (!mult16((uintptr_t)ops[i].slot))
            return KVC_ERR_ALIGNMENT;
        if (!probe || ((uintptr_t)ops[i].slot % 32) != 0)
            probe = ops[i].slot;  // the least aligned slot decides the vector width
        n_ent += ops[i].n_blocks;
    }
    if (n_ent == 0)
        return KVC_OK;
    if (!ids_on_device) {
        if (dir == KVC_DIR_UNPACK) {
            try {
                begin_dup_scope(lay);
            } catch (const std::bad_alloc &) {
                return KVC_ERR_NOMEM;
            }
        }
        for (uint32_t i = 0; i < n_ops; ++i) {
            kvc_status s = check_host_ids(lay, ops[i].ids, ops[i].n_blocks, dir == KVC_DIR_UNPACK);
            if (s != KVC_OK)
                return s;
        }
    }
    kvc_status s = ensure_device(lay);
    if (s != KVC_OK)
        return s;
    KvcLaunch a;
    memset(&a, 0, sizeof(a));
    KvcPlan plan;
    s = kvc_make_plan(lay, n_ent, probe, &a, &plan);
    if (s != KVC_OK)
        return s;
    KvcArena *ar = nullptr;
    s = take_arena(lay, n_ent, &ar);
    if (s != KVC_OK)
        return s;
    uint64_t k = 0;
    for (uint32_t i = 0; i < n_ops; ++i) {
        if (ops[i].n_blocks >= KVC_ENT_ID_IS_PTR)
            return KVC_ERR_INVALID_ARG;
        uint64_t ent_step, plane_step;
        kvc_chunk_steps(lay, ops[i].n_blocks, &ent_step, &plane_step);
        const uint32_t first = (uint32_t)k;
        for (uint32_t j = 0; j < ops[i].n_blocks; ++j, ++k) {
            KvcEnt &e = ar->host[k];
            e.slot_addr = (uint64_t)(uintptr_t)ops[i].slot + (uint64_t)j * ent_step;
            e.plane_step = plane_step;
            e.first_ent = first;
            if (ids_on_device) {
                e.id_or_ptr = (uint64_t)(uintptr_t)(ops[i].ids + j);
                e.nb_c = ops[i].n_blocks | KVC_ENT_ID_IS_PTR;
            } else {
                e.id_or_ptr = (uint64_t)(uint32_t)ops[i].ids[j];
                e.nb_c = ops[i].n_blocks;
            }
        }
    }
    // The table travels on the handle's own stream so that the copy overlaps whatever still runs
    // on the caller's stream; the kernel waits for it through an event.
    cudaStream_t st = (cudaStream_t)stream;
    if (cudaMemcpyAsync(ar->dev, ar->host, n_ent * sizeof(KvcEnt), cudaMemcpyHostToDevice,
                        lay->upload_stream) != cudaSuccess ||
        cudaEventRecord(lay->upload_done, lay->upload_stream) != cudaSuccess ||
        cudaStreamWaitEvent(st, lay->upload_done, 0) != cudaSuccess)
        return KVC_ERR_CUDA;
    a.table = ar->dev;
    s = kvc_launch_timed(lay, dir, plan.variant, a, plan.grid, plan.smem, st);
    if (s != KVC_OK)
        return s;
    if (cudaEventRecord(ar->done, st) != cudaSuccess)
        return KVC_ERR_CUDA;
    ar->busy = true;
    return KVC_OK;
}

}  // namespace

extern "C" {

const char *kvc_status_str(kvc_status s)
{
    switch (s) {
    case KVC_OK: return "ok";
    case KVC_ERR_INVALID_ARG: return "invalid argument";
    case KVC_ERR_OUT_OF_RANGE: return "block id out of range";
    case KVC_ERR_ALIGNMENT: return "pointer, stride or slab size not a multiple of 16 bytes";
    case KVC_ERR_CONFLICT: return "destination block named twice";
    case KVC_ERR_NOMEM: return "out of memory";
    case KVC_ERR_CUDA: return "CUDA runtime call failed";
    case KVC_ERR_WOULD_BLOCK: return "no free staging slot";
    case KVC_ERR_TIMEOUT: return "timed out waiting for a staging slot";
    case KVC_ERR_STATE: return "call does not fit the slot's state";
    case KVC_ERR_TOO_LARGE: return "more blocks or planes than this fixed-capacity entry point takes per call";
    case KVC_ERR_EXISTS: return "entry already published";
    case KVC_ERR_NOT_FOUND: return "no such entry";
    case KVC_ERR_IO: return "file-system call failed or entry has the wrong size";
    }
    return "unknown status";
}

kvc_status kvc_layout_desc_init_dense(kvc_layout_desc *d, const void *base, uint32_t num_layers,
                                      uint32_t kv_planes, uint32_t num_blocks, uint32_t block_size,
                                      uint32_t num_kv_heads, uint32_t head_dim, uint32_t elem_bytes,
                                      uint32_t chunk_tokens, uint32_t chunk_order)
{
    if (!d)
        return KVC_ERR_INVALID_ARG;
    memset(d, 0, sizeof(*d));
    d->num_layers = num_layers;
    d->kv_planes = kv_planes;
    d->num_blocks = num_blocks;
    d->block_size = block_size;
    d->num_kv_heads = num_kv_heads;
    d->head_dim = head_dim;
    d->elem_bytes = elem_bytes;
    d->chunk_tokens = chunk_tokens;
    d->chunk_order = chunk_order;
    d->base = base;
    // slab = B*H*D*e, plane = NB*slab, layer = P*plane; every factor is < 2^32
    unsigned __int128 slab = (unsigned __int128)block_size * num_kv_heads;
    slab = slab * head_dim * elem_bytes;
    const unsigned __int128 plane = slab * num_blocks;
    const unsigned __int128 layer = plane * kv_planes;
    const unsigned __int128 lim = ~(uint64_t)0;
    if (slab > lim || plane > lim || layer > lim || layer * num_layers > lim)
        return KVC_ERR_INVALID_ARG;
    d->block_stride = (uint64_t)slab;
    d->plane_stride = (uint64_t)plane;
    d->layer_stride = (uint64_t)layer;
    return KVC_OK;
}

kvc_status kvc_layout_create(const kvc_layout_desc *d, kvc_layout **out)
{
    if (!d || !out)
        return KVC_ERR_INVALID_ARG;
    *out = nullptr;
    if (!d->num_layers || !d->kv_planes || !d->num_blocks || !d->block_size || !d->num_kv_heads ||
        !d->head_dim || !d->chunk_tokens)
        return KVC_ERR_INVALID_ARG;
    if (d->elem_bytes != 1 && d->elem_bytes != 2 && d->elem_bytes != 4)
        return KVC_ERR_INVALID_ARG;
    if (d->chunk_tokens % d->block_size)
        return KVC_ERR_INVALID_ARG;
    if ((d->chunk_order != KVC_CHUNK_LAYER_MAJOR && d->chunk_order != KVC_CHUNK_BLOCK_MAJOR) ||
        d->reserved != 0)
        return KVC_ERR_INVALID_ARG;
    if (!d->plane_ptrs && !d->base)
        return KVC_ERR_INVALID_ARG;
    const uint64_t row = (uint64_t)d->num_kv_heads * d->head_dim * d->elem_bytes;
    const uint64_t slab = row * d->block_size;
    const uint64_t planes = (uint64_t)d->num_layers * d->kv_planes;
    if (slab > 0x7FFFFFFFull || planes > 0xFFFFFFull)
        return KVC_ERR_INVALID_ARG;
    const uint64_t bstride = d->block_stride ? d->block_stride : slab;
    if (bstride < slab)
        return KVC_ERR_INVALID_ARG;
    if (!mult16(slab) || !mult16(bstride))
        return KVC_ERR_ALIGNMENT;
    if (d->plane_ptrs) {
        for (uint64_t i = 0; i < planes; ++i) {
            if (!d->plane_ptrs[i])
                return KVC_ERR_INVALID_ARG;
            if (!mult16((uintptr_t)d->plane_ptrs[i]))
                return KVC_ERR_ALIGNMENT;
        }
    } else {
        if (!mult16((uintptr_t)d->base) || !mult16(d->layer_stride) || !mult16(d->plane_stride))
            return KVC_ERR_ALIGNMENT;
        // Two ways to keep planes from overlapping: every plane is its own range
        // ([L][P][NB][..], plane stride >= one plane), or the planes of a layer interleave inside
        // the block axis ([L][NB][P][..], block stride >= planes * plane stride >= planes * slab).
        const uint64_t plane_span = (uint64_t)(d->num_blocks - 1) * bstride + slab;
        const bool disjoint = d->kv_planes == 1 || d->plane_stride >= plane_span;
        const bool interleaved = d->plane_stride >= slab && bstride >= d->kv_planes * d->plane_stride;
        if (!disjoint && !interleaved)
            return KVC_ERR_INVALID_ARG;
        const uint64_t layer_span =
            disjoint ? (uint64_t)(d->kv_planes - 1) * d->plane_stride + plane_span
                     : (uint64_t)(d->num_blocks - 1) * bstride + (uint64_t)d->kv_planes * d->plane_stride;
        if (d->num_layers > 1 && d->layer_stride < layer_span)
            return KVC_ERR_INVALID_ARG;
    }
    kvc_layout *lay = new (std::nothrow) kvc_layout();
    if (!lay)
        return KVC_ERR_NOMEM;
    lay->d = *d;
    try {
        if (d->plane_ptrs)
            lay->plane_ptrs.assign(d->plane_ptrs, d->plane_ptrs + planes);
    } catch (const std::bad_alloc &) {
        delete lay;
        return KVC_ERR_NOMEM;
    }
    lay->d.plane_ptrs = nullptr;  // the caller's array is not kept
    lay->slab_bytes = slab;
    lay->row_bytes = row;
    lay->block_stride = bstride;
    lay->bpc = d->chunk_tokens / d->block_size;
    lay->planes_total = (uint32_t)planes;
    memset(&lay->tuning, 0, sizeof(lay->tuning));
    lay->dev_ready = false;
    lay->device = -1;
    lay->sm_count = lay->vec_blocks_per_sm = lay->max_smem_optin = 0;
    lay->d_plane_table = nullptr;
    lay->d_status = nullptr;
    lay->h_status = nullptr;
    lay->next_arena = 0;
    lay->upload_stream = nullptr;
    lay->upload_done = nullptr;
    lay->launches = 0;
    lay->seen_stamp = 0;
    lay->time_kernels = false;
    *out = lay;
    return KVC_OK;
}

kvc_status kvc_layout_destroy(kvc_layout *lay)
{
    if (!lay)
        return KVC_ERR_INVALID_ARG;
    kvc_status rc = KVC_OK;
    for (KvcArena &ar : lay->arenas) {
        if (ar.busy && cudaEventSynchronize(ar.done) != cudaSuccess)
            rc = KVC_ERR_CUDA;
        if (ar.done)
            cudaEventDestroy(ar.done);
        if (ar.host)
            cudaFreeHost(ar.host);
        if (ar.dev)
            cudaFree(ar.dev);
    }
    for (auto &pr : lay->timed) {
        cudaEventDestroy(pr.first);
        cudaEventDestroy(pr.second);
    }
    for (cudaEvent_t e : lay->spare_events)
        cudaEventDestroy(e);
    if (lay->upload_done)
        cudaEventDestroy(lay->upload_done);
    if (lay->upload_stream)
        cudaStreamDestroy(lay->upload_stream);
    if (lay->d_plane_table)
        cudaFree((void *)lay->d_plane_table);
    if (lay->d_status)
        cudaFree(lay->d_status);
    if (lay->h_status)
        cudaFreeHost(lay->h_status);
    delete lay;
    return rc;
}

uint64_t kvc_layout_slab_bytes(const kvc_layout *lay) { return lay ? lay->slab_bytes : 0; }

uint64_t kvc_layout_bytes_per_token(const kvc_layout *lay)
{
    return lay ? (uint64_t)lay->planes_total * lay->row_bytes : 0;
}

uint32_t kvc_layout_blocks_per_chunk(const kvc_layout *lay) { return lay ? lay->bpc : 0; }

uint64_t kvc_layout_chunk_bytes(const kvc_layout *lay, uint32_t n_blocks)
{
    return lay ? (uint64_t)lay->planes_total * n_blocks * lay->slab_bytes : 0;
}

uint32_t kvc_layout_num_chunks(const kvc_layout *lay, uint32_t n_blocks)
{
    return lay ? (uint32_t)(((uint64_t)n_blocks + lay->bpc - 1) / lay->bpc) : 0;
}

kvc_status kvc_layout_set_tuning(kvc_layout *lay, const kvc_tuning *t)
{
    if (!lay || !t)
        return KVC_ERR_INVALID_ARG;
    if (t->variant > KVC_VARIANT_BULK || t->order > KVC_ORDER_CHUNK_MAJOR)
        return KVC_ERR_INVALID_ARG;
    if (t->tile_bytes % 16)
        return KVC_ERR_INVALID_ARG;
    if (t->stages == 1 || t->stages > KVC_BULK_MAX_STAGES)
        return KVC_ERR_INVALID_ARG;
    if (t->ctas_per_sm > 4 || t->l2_hint > 4 || t->lag > KVC_BULK_MAX_STAGES || t->pdl > 3 || t->items_per_cta > (1u << 20))
        return KVC_ERR_INVALID_ARG;
    if ((t->group & ~KVC_GROUP_FORCE_KERNEL) > KVC_GROUP_MAX_SLABS || t->slot_memory > 2)
        return KVC_ERR_INVALID_ARG;
    if (t->vec_threads % 32 || t->vec_threads > KVC_VEC_THREADS)
        return KVC_ERR_INVALID_ARG;
    lay->tuning = *t;
    return KVC_OK;
}

kvc_status kvc_tuning_preset(kvc_preset which, kvc_tuning *out)
{
    if (!out || (which != KVC_PRESET_DEFAULT && which != KVC_PRESET_BESIDE_COMPUTE))
        return KVC_ERR_INVALID_ARG;
    memset(out, 0, sizeof(*out));
    if (which == KVC_PRESET_BESIDE_COMPUTE) {
        out->max_ctas = 16;
        out->tile_bytes = 8192;
        out->stages = 2;
    }
    return KVC_OK;
}

kvc_status kvc_map_request(const kvc_layout *lay, uint32_t n_blocks, uint32_t flags,
                           kvc_chunk_desc *out, uint32_t cap, uint32_t *n_out)
{
    if (!lay || !n_out || (!out && cap) || (flags & ~KVC_MAP_FULL_CHUNKS_ONLY))
        return KVC_ERR_INVALID_ARG;
    uint32_t n = 0;
    for (uint64_t first = 0; first < n_blocks; first += lay->bpc) {
        uint32_t nb = (uint32_t)std::min<uint64_t>(lay->bpc, n_blocks - first);
        if (nb < lay->bpc && (flags & KVC_MAP_FULL_CHUNKS_ONLY))
            break;
        if (n < cap) {
            out[n].request = 0;
            out[n].chunk = n;
            out[n].first = (uint32_t)first;
            out[n].n_blocks = nb;
            out[n].bytes = kvc_layout_chunk_bytes(lay, nb);
        }
        ++n;
    }
    *n_out = n;
    return KVC_OK;
}

kvc_status kvc_map_requests_shared(const kvc_layout *lay, const int32_t *const *tables,
                                   const uint32_t *lens, uint32_t n_requests, uint32_t flags,
                                   kvc_chunk_desc *out, uint32_t cap, uint32_t *n_out,
                                   uint64_t *unique_blocks)
{
    if (!lay || !n_out || (!out && cap) || (n_requests && (!tables || !lens)) ||
        (flags & ~KVC_MAP_FULL_CHUNKS_ONLY))
        return KVC_ERR_INVALID_ARG;
    for (uint32_t r = 0; r < n_requests; ++r)
        if (lens[r] && !tables[r])
            return KVC_ERR_INVALID_ARG;
    try {
        // A trie over block tables: node = (parent node, block id).  Two table positions are the
        // same staged block exactly when they reach the same node.  Longer requests go first, so
        // a chunk that is a truncation of another request's chunk arrives after it and finds its
        // last node already covered.
        // child(parent node, block id) -> node, in an open-addressing table (total table length is
        // known up front, so it never grows)
        uint64_t total_len = 0;
        for (uint32_t r = 0; r < n_requests; ++r)
            total_len += lens[r];
        uint64_t tcap = 16;
        while (tcap < 2 * total_len + 2)
            tcap *= 2;
        const uint64_t kEmpty = ~0ull;
        std::vector<uint64_t> keys(tcap, kEmpty);
        std::vector<uint32_t> vals(tcap, 0);
        auto child_of = [&](uint32_t node, int32_t id, uint32_t next_id, bool *created) {
            const uint64_t key = ((uint64_t)node << 32) | (uint32_t)id;
            uint64_t h = key * 0x9E3779B97F4A7C15ull;
            h ^= h >> 29;
            for (uint64_t i = h & (tcap - 1);; i = (i + 1) & (tcap - 1)) {
                if (keys[i] == key) {
                    *created = false;
                    return vals[i];
                }
                if (keys[i] == kEmpty) {
                    keys[i] = key;
                    vals[i] = next_id;
                    *created = true;
                    return next_id;
                }
            }
        };
        std::vector<char> covered(1, 0);  // node 0 = root
        covered.reserve(total_len + 1);
        std::vector<uint32_t> order(n_requests);
        for (uint32_t r = 0; r < n_requests; ++r)
            order[r] = r;
        std::stable_sort(order.begin(), order.end(),
                         [&](uint32_t x, uint32_t y) { return lens[x] > lens[y]; });
        std::vector<kvc_chunk_desc> kept;
        std::vector<uint32_t> kept_end;            // trie node where each kept chunk ends
        const uint32_t kNobody = ~0u;
        std::vector<uint32_t> owner(total_len + 1, kNobody);  // chunk end node -> lowest request ending a chunk there
        std::vector<uint32_t> path;
        uint64_t uniq = 0;
        for (uint32_t r : order) {
            const uint32_t n = lens[r];
            path.resize(n);
            uint32_t node = 0;
            for (uint32_t i = 0; i < n; ++i) {
                bool created = false;
                node = child_of(node, tables[r][i], (uint32_t)covered.size(), &created);
                if (created)
                    covered.push_back(0);
                path[i] = node;
            }
            uint32_t c = 0;
            for (uint64_t first = 0; first < n; first += lay->bpc, ++c) {
                uint32_t nb = (uint32_t)std::min<uint64_t>(lay->bpc, n - first);
                if (nb < lay->bpc && (flags & KVC_MAP_FULL_CHUNKS_ONLY))
                    break;
                const uint32_t end = path[first + nb - 1];
                if (owner[end] == kNobody || r < owner[end])
                    owner[end] = r;
                if (covered[end])
                    continue;
                for (uint32_t i = 0; i < nb; ++i) {
                    if (!covered[path[first + i]]) {
                        covered[path[first + i]] = 1;
                        ++uniq;
                    }
                }
                kvc_chunk_desc cd;
                cd.request = r;
                cd.chunk = c;
                cd.first = (uint32_t)first;
                cd.n_blocks = nb;
                cd.bytes = kvc_layout_chunk_bytes(lay, nb);
                kept.push_back(cd);
                kept_end.push_back(end);
            }
        }
        // identical chunks of several requests are attributed to the lowest request index
        for (size_t i = 0; i < kept.size(); ++i)
            kept[i].request = owner[kept_end[i]];
        std::sort(kept.begin(), kept.end(), [](const kvc_chunk_desc &x, const kvc_chunk_desc &y) {
            return x.request != y.request ? x.request < y.request : x.chunk < y.chunk;
        });
        for (size_t i = 0; i < kept.size() && i < cap; ++i)
            out[i] = kept[i];
        *n_out = (uint32_t)kept.size();
        if (unique_blocks)
            *unique_blocks = uniq;
    } catch (const std::bad_alloc &) {
        return KVC_ERR_NOMEM;
    }
    return KVC_OK;
}

kvc_status kvc_pack(kvc_layout *lay, const int32_t *ids, uint32_t n_blocks, int ids_on_device,
                    void *dst_slot, uint64_t slot_bytes, void *stream)
{
    return copy_one(lay, KVC_DIR_PACK, ids, n_blocks, ids_on_device, dst_slot, slot_bytes, stream);
}

kvc_status kvc_unpack(kvc_layout *lay, const void *src_slot, uint64_t slot_bytes,
                      const int32_t *ids, uint32_t n_blocks, int ids_on_device, void *stream)
{
    return copy_one(lay, KVC_DIR_UNPACK, ids, n_blocks, ids_on_device, const_cast<void *>(src_slot),
                    slot_bytes, stream);
}

kvc_status kvc_pack_batch(kvc_layout *lay, const kvc_chunk_op *ops, uint32_t n_ops,
                          int ids_on_device, void *stream)
{
    return copy_batch(lay, KVC_DIR_PACK, ops, n_ops, ids_on_device, stream);
}

kvc_status kvc_unpack_batch(kvc_layout *lay, const kvc_chunk_op *ops, uint32_t n_ops,
                            int ids_on_device, void *stream)
{
    return copy_batch(lay, KVC_DIR_UNPACK, ops, n_ops, ids_on_device, stream);
}

kvc_status kvc_poll_device_status(kvc_layout *lay, void *stream, uint32_t *n_skipped,
                                  uint32_t *n_wait_expired)
{
    if (!lay)
        return KVC_ERR_INVALID_ARG;
    if (n_skipped)
        *n_skipped = 0;
    if (n_wait_expired)
        *n_wait_expired = 0;
    if (!lay->dev_ready)
        return KVC_OK;  // nothing was ever launched
    cudaStream_t st = (cudaStream_t)stream;
    if (cudaMemcpyAsync(lay->h_status, lay->d_status, 2 * sizeof(uint32_t), cudaMemcpyDeviceToHost,
                        st) != cudaSuccess ||
        cudaMemsetAsync(lay->d_status, 0, 2 * sizeof(uint32_t), st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess)
        return KVC_ERR_CUDA;
    if (n_skipped)
        *n_skipped = lay->h_status[0];
    if (n_wait_expired)
        *n_wait_expired = lay->h_status[1];
    return KVC_OK;
}

uint64_t kvc_layout_launch_count(const kvc_layout *lay) { return lay ? lay->launches : 0; }
uint32_t kvc_layout_num_blocks(const kvc_layout *lay) { return lay ? lay->d.num_blocks : 0; }

kvc_status kvc_layout_set_kernel_timing(kvc_layout *lay, int on)
{
    if (!lay)
        return KVC_ERR_INVALID_ARG;
    lay->time_kernels = on != 0;
    return KVC_OK;
}

kvc_status kvc_layout_kernel_time(kvc_layout *lay, uint32_t *launches, double *total_ms, double *min_ms,
                                  double *max_ms)
{
    if (!lay)
        return KVC_ERR_INVALID_ARG;
    double total = 0, lo = 0, hi = 0;
    uint32_t n = 0;
    kvc_status rc = KVC_OK;
    for (auto &pr : lay->timed) {
        float ms = 0;
        if (cudaEventSynchronize(pr.second) != cudaSuccess ||
            cudaEventElapsedTime(&ms, pr.first, pr.second) != cudaSuccess) {
            (void)cudaGetLastError();
            rc = KVC_ERR_CUDA;
        } else {
            total += ms;
            lo = n == 0 || ms < lo ? ms : lo;
            hi = n == 0 || ms > hi ? ms : hi;
            ++n;
        }
        try {
            lay->spare_events.push_back(pr.first);
            lay->spare_events.push_back(pr.second);
        } catch (const std::bad_alloc &) {
            cudaEventDestroy(pr.first);
            cudaEventDestroy(pr.second);
        }
    }
    lay->timed.clear();
    if (launches)
        *launches = n;
    if (total_ms)
        *total_ms = total;
    if (min_ms)
        *min_ms = lo;
    if (max_ms)
        *max_ms = hi;
    return rc;
}

}  // extern "C"
