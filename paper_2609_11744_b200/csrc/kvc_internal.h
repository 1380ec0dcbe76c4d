// Internal declarations shared by the host side and the kernels of libkvc.
#ifndef KVC_INTERNAL_H
#define KVC_INTERNAL_H

#include <cuda_runtime.h>
#include <stdint.h>

#include <utility>
#include <vector>

#include "kvc.h"

#define KVC_PARAM_IDS 128u      // block ids that travel inside the kernel parameters
#define KVC_VEC_THREADS 256u    // threads per block of the vector kernels
#define KVC_VEC_UNROLL 4u       // vectors in flight per thread
#define KVC_VEC_WARP_TEAM_MAX_TILE 4096u  // tiles up to this size are copied by one warp each
// Slabs up to this size go through the multi-slab vector kernel, one warp per work item; an item
// is about KVC_VEC_GROUP_ITEM_BYTES (several small slabs, or one slab of 8-16 KiB).
#define KVC_VEC_GROUP_MAX_SLAB 16384u
#define KVC_VEC_GROUP_ITEM_BYTES 8192u
#define KVC_HOST_SLOT_DEFAULT_CTAS 16u
#define KVC_BULK_THREADS 32u    // one warp drives the bulk-copy pipeline
#define KVC_BULK_MAX_STAGES 16u
// Measured on B200 (80k-token prefix, 32 KiB slabs): HBM throughput peaks when each SM keeps one
// to two 32 KiB loads in flight (about 5-9 MB over the GPU); deeper prefetch lowers it by 3-4 %.
#define KVC_BULK_DEFAULT_STAGES 4u
#define KVC_BULK_DEFAULT_LAG 1u
// Streaming launch shape (measured on B200 against the persistent one in the same process, all
// workloads): two resident blocks per SM, each with two 32 KiB stages (load, then store, no
// prefetch) and about 64 KiB of work, in chunk-major order: 6.68-6.78 TB/s pack, 6.77-6.88 TB/s
// unpack where the persistent grid reaches 6.54-6.60 TB/s.
#define KVC_BULK_STREAMING_BLOCKS_PER_SM 2u
#define KVC_BULK_STREAMING_STAGES 2u
#define KVC_BULK_SMEM_HEADER 1024u  // mbarriers + per-stage bookkeeping ahead of the data stages
// Multi-slab kernel: a work item is a run of up to 32 consecutive slabs (a power of two), at most
// one tile in total.  Its shared-memory header holds the mbarriers (128 bytes) and, per stage, the
// address and length of up to 32 stores (384 bytes), rounded up to 128 bytes.
#define KVC_GROUP_MAX_SLABS 32u
#define KVC_GROUP_DEFAULT_SLABS 16u
#define KVC_GROUP_STAGE_INFO_BYTES 384u
#define KVC_GROUP_SMEM_HEADER(stages) ((128u + (stages) * KVC_GROUP_STAGE_INFO_BYTES + 127u) & ~127u)
#define KVC_WAIT_LIMIT (1u << 22)   // polls of an mbarrier before a kernel gives up

// Where the planes of the paged pool live (kernel-side copy of the layout).
struct KvcGeom {
    const unsigned char *base;              // monolithic pool (plane_table == nullptr)
    uint64_t layer_stride, plane_stride;
    const unsigned char *const *plane_table;  // device array of LP plane bases, or nullptr
    uint64_t block_stride;
    uint32_t slab_bytes;                    // S
    uint32_t planes_total;                  // LP = L*P
    uint32_t planes_per_layer;              // P
    uint32_t num_blocks;                    // NB
    uint32_t tile_bytes;                    // bytes of a slab moved by one work item
    uint32_t parts;                         // ceil(S / tile_bytes)
};

// One block of one chunk in a batched launch.  Entries are ordered by chunk, then by block.
struct KvcEnt {
    uint64_t slot_addr;   // chunk base + j*ent_step : where block j of the chunk starts in plane 0
    uint64_t id_or_ptr;   // the pool block id, or the device address of it
    uint64_t plane_step;  // bytes between consecutive planes of this block inside the chunk
    uint32_t nb_c;        // blocks in this chunk; bit 31 set: id_or_ptr is an address
    uint32_t first_ent;   // index of the chunk's first entry
};
#define KVC_ENT_ID_IS_PTR 0x80000000u
static_assert(sizeof(KvcEnt) == 32, "KvcEnt is loaded as two 16-byte vectors");

// Kernel parameters.
struct KvcLaunch {
    KvcGeom g;
    const KvcEnt *table;      // batched launch: n_ent entries in device memory; else nullptr
    uint64_t slot;            // single-chunk launch: chunk base
    uint64_t ent_step;        // single-chunk launch: bytes between consecutive blocks of a plane
    uint64_t plane_step;      // single-chunk launch: bytes between consecutive planes of a block
    const int32_t *dev_ids;   // single-chunk launch with device-resident ids; else nullptr
    uint32_t *status;         // [0] blocks skipped (bad device id), [1] waits that gave up
    uint64_t n_items;         // n_ent * LP * parts
    uint32_t n_ent;
    uint32_t order;           // kvc_order (never AUTO here)
    uint32_t block_major_chunks;  // chunk layout is [n][L][P].. (else [L][P][n]..)
    uint32_t stages;          // bulk kernels
    uint32_t lag;             // bulk kernels: loads issued ahead of the store they feed
    uint32_t l2_evict_first;  // single-slab bulk kernel: evict-first L2 policy on loads (bit 0), stores (bit 1)
    uint32_t pdl;             // launch with programmatic stream serialisation
    uint32_t group_shift;     // multi-slab kernel: log2 of the slabs per work item
    uint32_t pending;         // bulk kernels: stores that may still read shared memory at a stage reuse
    uint64_t n_slabs;         // multi-slab kernels: n_ent * LP
    uint32_t vec_threads;     // vector kernels with one warp per item: threads per block (0 = 256)
    uint64_t vec_magic;       // multi-slab vector kernel: 2^32 / (vectors per slab) + 1, for v / vps
    int32_t ids[KVC_PARAM_IDS];
};

enum { KVC_DIR_PACK = 0, KVC_DIR_UNPACK = 1 };
// Internal refinements: 32-byte vectors when everything is 32-byte aligned; the bulk kernel whose
// work items span several slabs.
enum { KVC_VARIANT_VEC32 = 100, KVC_VARIANT_BULK_GROUP = 101, KVC_VARIANT_VEC_GROUP = 102,
       KVC_VARIANT_VEC32_GROUP = 103 };

// Implemented in kvc_kernels.cu.
cudaError_t kvc_launch_copy(int dir, int variant, const KvcLaunch &a, uint32_t grid,
                            uint32_t smem_bytes, cudaStream_t stream);
cudaError_t kvc_kernel_limits(int *sm_count, int *vec_blocks_per_sm, int *max_smem_optin);

// A pinned-host + device pair that carries one batched launch's entry table.
struct KvcArena {
    KvcEnt *host = nullptr;
    KvcEnt *dev = nullptr;
    uint64_t cap = 0;           // entries
    cudaEvent_t done = nullptr; // recorded after the kernel that reads `dev`
    bool busy = false;
};

#define KVC_NUM_ARENAS 8

struct kvc_layout {
    kvc_layout_desc d;
    std::vector<const void *> plane_ptrs;  // host copy (empty for monolithic pools)
    uint64_t slab_bytes, row_bytes, block_stride;
    uint32_t bpc, planes_total;
    kvc_tuning tuning;
    // device state, created by the first launch
    bool dev_ready;
    int device;
    int sm_count, vec_blocks_per_sm, max_smem_optin;
    const unsigned char **d_plane_table;
    uint32_t *d_status;
    uint32_t *h_status;  // pinned
    KvcArena arenas[KVC_NUM_ARENAS];
    uint32_t next_arena;
    cudaStream_t upload_stream;  // entry tables travel on their own stream
    cudaEvent_t upload_done;
    uint64_t launches;
    std::vector<uint32_t> seen;  // scratch for duplicate detection: stamp per pool block
    uint32_t seen_stamp;
    // kernel timing (diagnostic): event pairs around launches not yet collected, and spare events
    bool time_kernels;
    std::vector<std::pair<cudaEvent_t, cudaEvent_t>> timed;
    std::vector<cudaEvent_t> spare_events;
};

// Launches the copy kernel; with kernel timing on, between two events on the same stream.
kvc_status kvc_launch_timed(kvc_layout *lay, int dir, int variant, const KvcLaunch &a, uint32_t grid,
                            uint32_t smem, cudaStream_t st);


// Where block j, plane lp of a chunk of nb blocks starts, relative to the chunk base:
// j * ent_step + lp * plane_step.  Layer-major chunks [L][P][nb][..]: (S, nb*S);
// block-major chunks [nb][L][P][..]: (L*P*S, S).
inline void kvc_chunk_steps(const kvc_layout *lay, uint32_t nb, uint64_t *ent_step, uint64_t *plane_step)
{
    if (lay->d.chunk_order == KVC_CHUNK_BLOCK_MAJOR) {
        *ent_step = (uint64_t)lay->planes_total * lay->slab_bytes;
        *plane_step = lay->slab_bytes;
    } else {
        *ent_step = lay->slab_bytes;
        *plane_step = (uint64_t)nb * lay->slab_bytes;
    }
}

// Launch shape chosen by the host for one call.
struct KvcPlan {
    int variant;
    uint32_t grid, smem, stages, lag;
};
// Implemented in kvc_layout.cu.  Reads the handle's tuning and the device limits cached in it.
kvc_status kvc_make_plan(kvc_layout *lay, uint64_t n_ent, const void *slot_probe, KvcLaunch *a,
                         KvcPlan *plan);

#endif
