/*
 * kvc -- paged KV-cache pack / unpack and a bounded staging ring for external
 * KV-cache offload, for NVIDIA B200 (sm_100a).
 *
 * The operations follow the problem statement of "Building py-kvcache":
 *   - Sec. 2.1: the KV cache of a serving engine is a pool of fixed-size token
 *     blocks; bytes per token = layers x 2 x KV heads x head dim x element size.
 *   - Sec. 6.4: an external cache stores "storage blocks" (here: chunks) that
 *     group several GPU blocks of one request, in request order; an operation
 *     on a whole prefix is cut into one job per chunk; every job moves through
 *     one slot of a fixed, bounded staging pool, and a slot is reused only after
 *     the CUDA event guarding its last copy has completed.
 *   - Sec. 6.4 (loads): all block mappings that are ready, from any number of
 *     requests, are fused into a single launch.
 *   - Sec. 6.5: requests with an identical prefix stage the shared chunks once.
 *
 * Memory model.  The paged pool is [layer][K|V][block][token][kv_head][head_dim]:
 * every (layer, K|V) "plane" is an array of `num_blocks` blocks, each a run of
 *     slab_bytes = block_size * num_kv_heads * head_dim * elem_bytes
 * contiguous bytes, `block_stride` bytes apart.  A chunk of n blocks is the
 * same layout with the block axis gathered: [layer][K|V][n][token][head][dim],
 * exactly  layers * planes * n * slab_bytes  bytes, no padding (a short last
 * chunk is stored compactly).
 *
 *   pack  : chunk[l][p][j][...] = pool[l][p][ids[j]][...]     (save / offload)
 *   unpack: pool[l][p][ids[j]][...] = chunk[l][p][j][...]     (load / preload)
 *
 * Elements are opaque bytes.  All functions return a status and never abort.
 * The library never owns the KV pool.  Handles are not thread-safe: use one
 * layout handle and one ring per host thread.  Streams are `cudaStream_t`
 * values passed as `void*` so that this header needs no CUDA include.
 *
 * Every copy runs in the library's CUDA kernels; there is no host fallback.
 */
#ifndef KVC_H
#define KVC_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    KVC_OK = 0,
    KVC_ERR_INVALID_ARG = 1,  /* NULL handle/pointer, zero size, slot too small, bad enum */
    KVC_ERR_OUT_OF_RANGE = 2, /* a host-resident block id is < 0 or >= num_blocks */
    KVC_ERR_ALIGNMENT = 3,    /* a pointer, stride or slab size is not a multiple of 16 bytes */
    KVC_ERR_CONFLICT = 4,     /* unpack: the same destination block named twice (host ids) */
    KVC_ERR_NOMEM = 5,        /* host or device allocation failed */
    KVC_ERR_CUDA = 6,         /* a CUDA runtime call failed (no device, launch error, ...) */
    KVC_ERR_WOULD_BLOCK = 7,  /* ring: no free slot and timeout_us == 0 */
    KVC_ERR_TIMEOUT = 8,      /* ring: no free slot before the deadline */
    KVC_ERR_STATE = 9,        /* ring: call does not fit the slot's state */
    KVC_ERR_TOO_LARGE = 10,   /* more work than a fixed-capacity entry point can take in one call */
    KVC_ERR_EXISTS = 11,      /* store: the entry is already published (first writer wins) */
    KVC_ERR_NOT_FOUND = 12,   /* store: no entry for this hash */
    KVC_ERR_IO = 13           /* store: a file-system call failed, or an entry has the wrong size */
} kvc_status;

const char *kvc_status_str(kvc_status s);

/* ------------------------------------------------------------------ layout (Sec. 2.1) */

typedef struct kvc_layout kvc_layout;

/* Byte order inside a chunk of n blocks.  The paper fixes only the file naming (Sec. 6.3), not
 * the order inside a storage block.  LAYER_MAJOR [layer][K|V][n][token][head][dim] is the paged
 * layout with the block axis gathered.  BLOCK_MAJOR [n][layer][K|V][token][head][dim] keeps all
 * layers of one block together, so a shorter chunk is a prefix of a longer one. */
typedef enum { KVC_CHUNK_LAYER_MAJOR = 0, KVC_CHUNK_BLOCK_MAJOR = 1 } kvc_chunk_order;

typedef struct {
    uint32_t num_layers;
    uint32_t kv_planes;    /* planes per layer: 2 (K and V), or 1 for a fused cache */
    uint32_t num_blocks;   /* blocks in every plane of the pool */
    uint32_t block_size;   /* tokens per block */
    uint32_t num_kv_heads;
    uint32_t head_dim;
    uint32_t elem_bytes;   /* 1, 2 or 4 */
    uint32_t chunk_tokens; /* tokens per chunk; a positive multiple of block_size */
    /* Either plane_ptrs != NULL: HOST array of num_layers*kv_planes DEVICE pointers,
     * entry l*kv_planes+p is the base of plane (l,p) (the array is copied);
     * or plane_ptrs == NULL: plane (l,p) starts at base + l*layer_stride + p*plane_stride.
     * Planes must not overlap: either plane_stride >= the span of one plane (pool order
     * [layer][K|V][block]..), or block_stride >= kv_planes*plane_stride >= kv_planes*slab_bytes
     * (pool order [layer][block][K|V].., K and V of a block adjacent). */
    const void *const *plane_ptrs;
    const void *base;      /* device pointer */
    uint64_t layer_stride; /* bytes */
    uint64_t plane_stride; /* bytes */
    uint64_t block_stride; /* bytes between consecutive blocks of a plane; 0 means slab_bytes */
    uint32_t chunk_order;  /* kvc_chunk_order: byte order inside a chunk */
    uint32_t reserved;     /* must be 0 */
} kvc_layout_desc;

/* Fills *desc for a pool that is one dense allocation [layer][K|V][block][token][head][dim]
 * starting at `base` (Sec. 2.1 layout, no padding anywhere): plane_ptrs = NULL, plane stride =
 * num_blocks * slab bytes, layer stride = kv_planes * plane stride, block stride = slab bytes.
 * Pure arithmetic, no validation beyond NULL (kvc_layout_create validates).  INVALID_ARG if desc
 * is NULL or a product overflows 64 bits. */
kvc_status kvc_layout_desc_init_dense(kvc_layout_desc *desc, const void *base, uint32_t num_layers,
                                      uint32_t kv_planes, uint32_t num_blocks, uint32_t block_size,
                                      uint32_t num_kv_heads, uint32_t head_dim, uint32_t elem_bytes,
                                      uint32_t chunk_tokens, uint32_t chunk_order);

/* Validates and copies the descriptor.  Makes no CUDA call: the small device-side
 * state a launch needs (plane-pointer table, status words, id-table arenas) is
 * allocated by the first pack/unpack call on the handle, which therefore must not
 * happen during stream capture.  From then on the handle belongs to the device that was
 * current at that call (INVALID_ARG if another device is current later); use one handle per GPU.
 * Errors: INVALID_ARG (NULL, zero dimension, chunk_tokens not a multiple of
 * block_size, elem_bytes not 1/2/4, block_stride < slab_bytes), ALIGNMENT (slab
 * bytes, a base pointer or a stride not a multiple of 16), NOMEM. */
kvc_status kvc_layout_create(const kvc_layout_desc *desc, kvc_layout **out);
/* Frees the handle and its device state (synchronises with work that still uses it). */
kvc_status kvc_layout_destroy(kvc_layout *layout);

uint64_t kvc_layout_slab_bytes(const kvc_layout *layout);
uint64_t kvc_layout_bytes_per_token(const kvc_layout *layout);      /* Sec. 2.1 formula */
uint32_t kvc_layout_blocks_per_chunk(const kvc_layout *layout);     /* chunk_tokens / block_size */
uint64_t kvc_layout_chunk_bytes(const kvc_layout *layout, uint32_t n_blocks); /* L*P*n*slab */
uint32_t kvc_layout_num_chunks(const kvc_layout *layout, uint32_t n_blocks);  /* ceil(n / bpc) */
uint32_t kvc_layout_num_blocks(const kvc_layout *layout);           /* blocks in the pool (NB) */

/* How the copy kernels run (no counterpart in the paper: launch-shape knobs of this
 * implementation, used by its benchmarks and tests).  Zero in every field means "library default"
 * (AUTO: the bulk-copy kernel for slots in device memory, the vector kernel with 16 persistent
 * blocks for slots in mapped host memory; chunk-major order). */
typedef enum {
    KVC_VARIANT_AUTO = 0,
    KVC_VARIANT_VEC = 1,  /* 16- or 32-byte vector loads/stores through registers */
    KVC_VARIANT_BULK = 2  /* bulk async copies global->shared->global, one warp per thread block;
                             small slabs are moved several per work item (see kvc_tuning.group) */
} kvc_variant;
typedef enum {
    KVC_ORDER_AUTO = 0,
    KVC_ORDER_PLANE_MAJOR = 1, /* walk all blocks of one (layer,K|V) plane, then the next plane */
    KVC_ORDER_BLOCK_MAJOR = 2, /* walk all planes of one block, then the next block */
    KVC_ORDER_CHUNK_MAJOR = 3  /* walk the chunks one after another, each in the order its bytes
                                  lie in the slot: the staging side is accessed sequentially */
} kvc_order;
typedef struct {
    uint32_t variant;    /* kvc_variant */
    uint32_t order;      /* kvc_order */
    uint32_t max_ctas;   /* 0 = default launch shape: many short-lived blocks of a few work items
                            each, scheduled by the hardware.  N > 0: exactly N persistent blocks
                            that stride over all items; a small N leaves SMs to a concurrent
                            compute stream */
    uint32_t tile_bytes; /* bytes of one slab moved per work item (0 = default); multiple of 16 */
    uint32_t stages;     /* BULK: shared-memory stages per thread block (0 = default) */
    uint32_t ctas_per_sm; /* BULK: thread blocks the shared memory of one SM is divided among,
                            1..4 (0 = default); bounds stages * tile_bytes per block */
    uint32_t l2_hint;    /* BULK (single-slab kernel): 0 = default (= 1), 1 = no L2 priority hint,
                            2 = evict-first on loads and stores, 3 = on loads only, 4 = on stores only */
    uint32_t lag;        /* BULK: loads issued ahead of the store they feed, 1..stages-2 (0 = default) */
    uint32_t items_per_cta; /* default launch shape: work items per block (0 = about 64 KiB for
                            BULK, 32 KiB for VEC) */
    uint32_t pdl;        /* 0 = default (= 2), 1 = plain launches, 2 = programmatic dependent launch:
                            a kernel's blocks may be scheduled while the previous kernel of the
                            stream drains; they wait for its completion before reading memory.
                            3 = the same WITHOUT that wait, for a sequence of calls on one stream
                            whose kernels are independent of one another (packing the chunks of a
                            request into different slots; unpacking chunks into different blocks):
                            a kernel then runs beside the last blocks of the previous one instead
                            of after them.  The caller vouches for the independence: a pack right
                            after an unpack of the same blocks would read stale bytes.  Work of other
                            kinds queued earlier on the stream (copies, waits for events) is
                            complete either way, and an event recorded after a call still covers
                            that call and everything before it */
    uint32_t group;      /* BULK: slabs per work item.  0 = default: when a slab is at most half a
                            tile, as many whole slabs as fit one tile (a power of two, at most 16;
                            the default tile is 16 KiB for slabs under 4 KiB)
                            -- consecutive slabs of a chunk are contiguous in the slot, so one item
                            is several copies on the pool side and one on the slot side;
                            1 = one slab (or one tile of a slab) per item; N > 1 = at most N (<= 32).
                            VEC: slabs of at most 16 KiB go one warp per item, and as many whole
                            slabs as fit 8 KiB per item.
                            Adding KVC_GROUP_FORCE_KERNEL runs the multi-slab kernel even when that
                            leaves one slab per item (for same-process comparisons) */
    uint32_t slot_memory; /* where the staging slots of this handle's calls live: 0 = ask the CUDA
                            runtime on every call (one pointer-attribute query, a fraction of a
                            microsecond), 1 = device memory, 2 = mapped pinned host memory.  A
                            caller that issues many small per-chunk calls into slots it allocated
                            itself can save the query; a wrong answer picks a kernel tuned for the
                            other kind of memory */
    uint32_t vec_threads; /* VEC: threads per block, a multiple of 32 up to 256 (0 = 256).  Fewer than
                            256 makes every warp copy its own tile of at most 4 KiB.  max_ctas still
                            counts blocks.  An experiment knob: spreading the warps of the
                            mapped-host path over many small blocks was measured to disturb a
                            concurrent GEMM more, not less (the 16 full blocks of the default
                            occupy the fewest SMs) */
} kvc_tuning;
#define KVC_GROUP_FORCE_KERNEL 0x100u
/* Errors: INVALID_ARG (unknown enum, tile_bytes not a multiple of 16, stages*tile too large). */
kvc_status kvc_layout_set_tuning(kvc_layout *layout, const kvc_tuning *tuning);
/* Ready-made tunings (no counterpart in the paper; Sec. 5.1 is where the question comes from: a
 * copy kernel takes SM time away from the model).
 *   KVC_PRESET_DEFAULT         all zeros: highest copy throughput, for slots in device memory.
 *   KVC_PRESET_BESIDE_COMPUTE  for streaming chunks to or from the host while a compute stream is
 *       busy: 16 persistent one-warp blocks with two 8 KiB stages each (17 KB of shared memory and
 *       about 1000 registers per block), small enough to sit on an SM BESIDE a resident GEMM block
 *       instead of waiting for one to retire and then keeping the next one out.  Measured on B200
 *       next to a bf16 8192^3 matmul loop: the host link stays saturated (56.7 / 55.0 GB/s) and the
 *       GEMM loop slows down by about 2 % (0-2.6 % over four runs), against 7-8 % with the default
 *       66 KB blocks and about 1 % with the copy engines, which hold a lower link rate.  Its own
 *       ceiling is a few hundred GB/s: not for device-to-device staging at HBM speed.
 * Fills *out; pass it to kvc_layout_set_tuning.  INVALID_ARG for an unknown preset or NULL. */
typedef enum { KVC_PRESET_DEFAULT = 0, KVC_PRESET_BESIDE_COMPUTE = 1 } kvc_preset;
kvc_status kvc_tuning_preset(kvc_preset which, kvc_tuning *out);

/* ------------------------------------------------------------------ mapper (Sec. 6.4, 6.5) */

typedef struct {
    uint32_t request;  /* index of the request the chunk belongs to */
    uint32_t chunk;    /* chunk index inside that request */
    uint32_t first;    /* first block-table entry covered */
    uint32_t n_blocks; /* entries covered: blocks_per_chunk, or fewer in the last chunk */
    uint64_t bytes;    /* kvc_layout_chunk_bytes(n_blocks) */
} kvc_chunk_desc;

#define KVC_MAP_FULL_CHUNKS_ONLY 1u /* drop a short last chunk (only whole storage blocks are cached) */

/* Cuts one request of n_blocks table entries into chunks: chunk c covers entries
 * [c*bpc, min((c+1)*bpc, n_blocks)).  Writes up to `cap` descriptors to `out` (may be NULL
 * with cap 0 to query) and the total count to *n_out.  Host only.
 * Errors: INVALID_ARG. */
kvc_status kvc_map_request(const kvc_layout *layout, uint32_t n_blocks, uint32_t flags,
                           kvc_chunk_desc *out, uint32_t cap, uint32_t *n_out);

/* Same for many requests at once, staging every shared chunk once (Sec. 6.5): a chunk is
 * dropped when another request's chunk with the same index already carries all of its blocks
 * at the same table positions with an identical table before them.  tables[r] is a HOST array
 * of lens[r] block ids.  Output is in (request, chunk) order.  *unique_blocks (may be NULL)
 * receives the number of blocks covered by the kept chunks.  Host only. */
kvc_status kvc_map_requests_shared(const kvc_layout *layout, const int32_t *const *tables,
                                   const uint32_t *lens, uint32_t n_requests, uint32_t flags,
                                   kvc_chunk_desc *out, uint32_t cap, uint32_t *n_out,
                                   uint64_t *unique_blocks);

/* ------------------------------------------------------------------ pack / unpack (Sec. 6.4) */

/* One chunk.  `ids` is the chunk's slice of the request's block table, n_blocks entries,
 * in HOST memory (ids_on_device == 0; may be reused as soon as the call returns) or in DEVICE
 * memory (ids_on_device != 0; must stay valid until the kernel has run).  `slot` is DEVICE
 * memory (or mapped pinned host memory), 16-byte aligned, slot_bytes >= chunk_bytes(n_blocks);
 * bytes of the slot past the chunk are not touched, nor are pool blocks not named in ids.
 * Asynchronous: the kernel is enqueued on `stream` and the call returns.
 * Host ids are validated before anything is launched (OUT_OF_RANGE; unpack: CONFLICT on a
 * repeated id).  Device ids are range-checked in the kernel: a bad id skips its block and
 * is counted (see kvc_poll_device_status); repeated device ids in unpack are undefined.
 * n_blocks == 0 is a no-op returning KVC_OK.
 * With device ids, or with at most 128 host ids (they travel in the kernel parameters), a call
 * enqueues exactly one kernel and nothing else, so once the handle has made its first launch such
 * calls can be captured into a CUDA graph.  Longer host id lists, and the batched calls, also
 * upload an id table on a second stream and are not meant for capture.
 * Errors: INVALID_ARG, OUT_OF_RANGE, CONFLICT, ALIGNMENT, NOMEM, CUDA. */
kvc_status kvc_pack(kvc_layout *layout, const int32_t *ids, uint32_t n_blocks, int ids_on_device,
                    void *dst_slot, uint64_t slot_bytes, void *stream);
kvc_status kvc_unpack(kvc_layout *layout, const void *src_slot, uint64_t slot_bytes,
                      const int32_t *ids, uint32_t n_blocks, int ids_on_device, void *stream);

/* Many chunks, possibly of many requests, in ONE launch (the fused launch of Sec. 6.4).
 * ops is a HOST array; every op is one chunk as above with slot_bytes implied
 * (= chunk_bytes(n_blocks)).  With host ids, unpack also rejects an id repeated across ops. */
typedef struct {
    void *slot;         /* device (or mapped host) memory of chunk_bytes(n_blocks) bytes */
    const int32_t *ids; /* n_blocks ids, host or device as the call says */
    uint32_t n_blocks;
    uint32_t reserved;  /* must be 0 */
} kvc_chunk_op;
kvc_status kvc_pack_batch(kvc_layout *layout, const kvc_chunk_op *ops, uint32_t n_ops,
                          int ids_on_device, void *stream);
kvc_status kvc_unpack_batch(kvc_layout *layout, const kvc_chunk_op *ops, uint32_t n_ops,
                            int ids_on_device, void *stream);

/* No counterpart in the paper: the kernels' own health report.
 * Waits for `stream`, then reports and clears the handle's device-side counters:
 * *n_skipped = blocks skipped because a device-resident id was out of range,
 * *n_wait_expired = bounded waits inside a kernel that gave up (should be 0).
 * Either pointer may be NULL. */
kvc_status kvc_poll_device_status(kvc_layout *layout, void *stream, uint32_t *n_skipped,
                                  uint32_t *n_wait_expired);

/* Batched pack for callers that must not allocate (the paper has no counterpart: this is a
 * deployment aid).  Serving engines that gave every spare byte of device memory to their KV pool,
 * scheduler threads that cannot afford the device-wide stall an allocation may cause, and code
 * running under an allocator policy that forbids raw cudaMalloc can all still offload KV blocks
 * through this call: it allocates and frees nothing, on the device or on the host, and neither
 * does anything it calls.  Same result as kvc_pack_batch with ids_on_device == 0 (ids must be in
 * HOST memory; they are fully validated before anything is enqueued).
 * The id table, the plane-pointer table and two status counters live in a fixed array inside the
 * library image (about 264 KiB of device memory on every GPU that loads the library, held until
 * the process exits).  Limits: at most KVC_STATIC_MAX_BLOCKS blocks per call, summed over the
 * ops, and at most KVC_STATIC_MAX_PLANES planes for layouts given as plane pointers; beyond
 * either the call returns KVC_ERR_TOO_LARGE and enqueues nothing.
 * The tables travel to the device inside the parameters of small kernels enqueued on `stream`
 * ahead of the copy kernel -- chunk records and 4-byte ids, expanded into table entries on the
 * device: one launch per ~32 KiB of those, typically one or two -- so the call does not wait
 * for the stream and the host arrays may be reused as soon as it returns.
 * The first call on a device looks up the array's device address and the device's limits; make
 * that first call outside any stream capture.  Every call shares the one array, which keeps the
 * previous call's contents: calls whose GPU work can overlap -- different streams -- race on it,
 * so keep them on one stream (back-to-back calls on one stream need no synchronisation between
 * them).  Host-side the call is serialised by a lock.  The handle's own device status counters are
 * not touched; this path has its own pair, read with kvc_poll_static_status.
 * If the handle has launched before, the device it belongs to must be current (INVALID_ARG).
 * Errors: INVALID_ARG, ALIGNMENT, OUT_OF_RANGE, TOO_LARGE, CUDA. */
#define KVC_STATIC_MAX_BLOCKS 8192u
#define KVC_STATIC_MAX_PLANES 1024u
kvc_status kvc_pack_batch_static(kvc_layout *layout, const kvc_chunk_op *ops, uint32_t n_ops,
                                 void *stream);
/* kvc_poll_device_status for the kvc_pack_batch_static path of the current device (no counterpart
 * in the paper).  Waits for `stream`, reports and clears the two counters kept in the fixed array:
 * blocks skipped for a bad id (always 0 here, ids are validated on the host) and bounded in-kernel
 * waits that gave up (should be 0; non-zero means a pack did not complete).  Allocates nothing. */
kvc_status kvc_poll_static_status(void *stream, uint32_t *n_skipped, uint32_t *n_wait_expired);

/* Copy-engine variants (the paper's own mechanism, Sec. 6.2 / 6.4: a DMA-based batched block
 * copy between the KV tensors and pinned staging slots; Sec. 5.1 contrasts it with kernel copies).
 * Same result as kvc_pack / kvc_unpack for one chunk, but issued as strided asynchronous memory
 * copies on `stream` -- one per block where the planes are equally spaced, else one per layer or
 * per plane -- so no kernel runs and no SM is used.  `dst` / `src` may be DEVICE memory or PINNED
 * HOST memory; with host memory the chunk crosses the host link directly and no staging slot is
 * needed.  ids are HOST memory and are validated first (unpack rejects repeated ids).
 * They allocate nothing and do not count as kernel launches.
 * Errors: INVALID_ARG, ALIGNMENT, OUT_OF_RANGE, CONFLICT, CUDA. */
kvc_status kvc_pack_copy_engine(kvc_layout *layout, const int32_t *ids, uint32_t n_blocks, void *dst,
                                uint64_t dst_bytes, void *stream);
kvc_status kvc_unpack_copy_engine(kvc_layout *layout, const void *src, uint64_t src_bytes,
                                  const int32_t *ids, uint32_t n_blocks, void *stream);

/* Number of kernel launches issued through this handle so far (no counterpart in the paper;
 * the benchmark reports it so that a run that launched nothing cannot pass for a GPU run). */
uint64_t kvc_layout_launch_count(const kvc_layout *layout);

/* Kernel timing (diagnostic, no counterpart in the paper).  With on != 0 every copy kernel
 * launched through the handle (not kvc_pack_batch_static) is bracketed by two CUDA events on its
 * stream, so that the kernel's own duration can be told from the call's host work and table upload.
 * The events sit between consecutive kernels of a stream and so keep programmatic dependent launch
 * from overlapping them: leave it off outside measurements.  kvc_layout_kernel_time waits for the
 * launches timed since its last call and reports their number, summed, shortest and longest
 * duration in milliseconds (any pointer may be NULL).  Errors: INVALID_ARG, NOMEM, CUDA. */
kvc_status kvc_layout_set_kernel_timing(kvc_layout *layout, int on);
kvc_status kvc_layout_kernel_time(kvc_layout *layout, uint32_t *launches, double *total_ms,
                                  double *min_ms, double *max_ms);

/* ------------------------------------------------------------------ staging ring (Sec. 6.4) */

typedef struct kvc_ring kvc_ring;
typedef enum {
    KVC_RING_DEVICE = 0,      /* slots in device memory; the caller drains them with async copies */
    KVC_RING_HOST_MAPPED = 1, /* slots in mapped pinned host memory; kernels write them directly */
    KVC_RING_DEVICE_STAGED = 2 /* every slot is a pair: a device half that the kernels touch and a
                                 pinned host half of the same size that file I/O touches; one
                                 asynchronous copy moves a slot between the two (the store / load
                                 pipelines do it; other callers get both addresses from acquire).
                                 Kernels then run at HBM speed, with small blocks if a model is
                                 running (KVC_PRESET_BESIDE_COMPUTE), and the copy engines cross the
                                 link -- the combination that measured best beside a compute stream
                                 and with both directions busy.  The host half is always allocated
                                 by the library */
} kvc_ring_kind;

/* A ring of n_slots fixed slots of slot_bytes each (a multiple of 4096; use
 * chunk_bytes(blocks_per_chunk) rounded up).  mem == NULL: the library allocates
 * n_slots*slot_bytes (cudaMalloc, or cudaHostAlloc mapped) and frees it on destroy;
 * otherwise the caller's buffer of mem_bytes >= n_slots*slot_bytes is used and not freed.
 * Slot life cycle, strictly in slot order 0,1,..,n-1,0,.. (FIFO):
 *   acquire -> [producer work on stream A] -> commit(A) -> wait_filled(C) ->
 *   [consumer work on stream C] -> release(C) -> free again once the release event completes.
 * Errors: INVALID_ARG, ALIGNMENT, NOMEM, CUDA. */
kvc_status kvc_staging_ring_create(uint64_t slot_bytes, uint32_t n_slots, kvc_ring_kind kind,
                                   void *mem, uint64_t mem_bytes, kvc_ring **out);
/* Waits for outstanding slot events, frees library-owned memory and the handle. */
kvc_status kvc_staging_ring_destroy(kvc_ring *ring);
/* Next slot in FIFO order.  It is handed out only if it was never used or the event recorded
 * by its last release has completed (polled on the host; no device-wide synchronisation).
 * timeout_us == 0: try once (WOULD_BLOCK); > 0: poll until the deadline (TIMEOUT);
 * < 0: INVALID_ARG (unbounded waits are not offered).
 * *dev_ptr is the address kernels and async copies use; *host_ptr the host address of the same
 * bytes (HOST_MAPPED rings), the slot's separate pinned host half (DEVICE_STAGED rings), or NULL.
 * Either may be NULL. */
kvc_status kvc_staging_ring_acquire(kvc_ring *ring, int64_t timeout_us, uint32_t *slot,
                                    void **dev_ptr, void **host_ptr);
/* Records the slot's "filled" event on the producer stream.  STATE unless acquired. */
kvc_status kvc_staging_ring_commit(kvc_ring *ring, uint32_t slot, void *producer_stream);
/* Makes consumer_stream wait for the slot's "filled" event.  STATE unless committed. */
kvc_status kvc_staging_ring_wait_filled(kvc_ring *ring, uint32_t slot, void *consumer_stream);
/* Records the slot's "drained" event on the consumer stream; the slot becomes free when that
 * event completes.  STATE unless committed. */
kvc_status kvc_staging_ring_release(kvc_ring *ring, uint32_t slot, void *consumer_stream);
/* Host-side producers and consumers (file reads and writes on mapped pinned slots):
 * commit_host marks an acquired slot filled by the host (no event; wait_filled then adds no
 * dependency), sync_filled blocks the calling host thread until the slot's "filled" event has
 * completed (may be called from a worker thread, for distinct slots concurrently with other ring
 * calls), release_host frees a filled slot at once because its consumer was the host and is done.
 * STATE unless the slot is acquired (commit_host) or filled (the other two). */
kvc_status kvc_staging_ring_commit_host(kvc_ring *ring, uint32_t slot);
kvc_status kvc_staging_ring_sync_filled(kvc_ring *ring, uint32_t slot);
kvc_status kvc_staging_ring_release_host(kvc_ring *ring, uint32_t slot);
/* in_flight = slots that are not free right now (the events of released slots are queried);
 * stalls = acquire polls that found the next slot still busy.  Any pointer may be NULL. */
kvc_status kvc_staging_ring_stats(const kvc_ring *ring, uint32_t *in_flight, uint64_t *acquires,
                                  uint64_t *stalls);
/* Slot transitions with host timestamps, for timelines of a transfer (the paper traces its
 * pipeline the same way, Sec. 4.1).  `buf` is a HOST array of `cap` entries owned by the caller and
 * must outlive the ring or be detached with buf = NULL; entries past `cap` are dropped but still
 * counted.  A stall is logged once per acquire call that had to wait or was refused. */
typedef enum { KVC_TRACE_ACQUIRE = 0, KVC_TRACE_COMMIT = 1, KVC_TRACE_RELEASE = 2, KVC_TRACE_STALL = 3 } kvc_ring_trace_kind;
typedef struct {
    uint64_t t_ns; /* steady-clock nanoseconds */
    uint32_t slot;
    uint32_t what; /* kvc_ring_trace_kind */
} kvc_ring_trace_entry;
kvc_status kvc_staging_ring_set_trace(kvc_ring *ring, kvc_ring_trace_entry *buf, uint32_t cap);
uint32_t kvc_staging_ring_trace_count(const kvc_ring *ring);
uint64_t kvc_staging_ring_slot_bytes(const kvc_ring *ring);
uint32_t kvc_staging_ring_num_slots(const kvc_ring *ring);
int kvc_staging_ring_pool_mode(const kvc_ring *ring); /* 1 after kvc_staging_ring_set_policy */
kvc_ring_kind kvc_staging_ring_kind(const kvc_ring *ring);

/* ------------------------------------------------------------------ chunk files (Sec. 6.3) */

/* The step behind the ring: one file per chunk in a hash-addressed directory tree that several
 * engine instances can share (Sec. 6.3).  Host only; every pointer is HOST memory.
 * Path of an entry: <root>/<model_tag>/<hh>/<hh>/<16 hex digits of the hash>.kv, the two
 * directory levels taken from the top two bytes of the hash.
 * Publication is first-writer-wins: the data goes to a uniquely named temporary file in the
 * target directory, a hard link creates the final name atomically (KVC_ERR_EXISTS if another
 * writer was first; the existing entry is kept), the temporary name is removed.  Readers open
 * final names only, so an entry is either absent or complete.
 * direct_io != 0: files are opened with O_DIRECT when the buffer is 4096-byte aligned and the
 * size a multiple of 4096 (ring slots are); where the file system refuses the flag the call
 * falls back to buffered I/O and counts it (kvc_store_direct_io_refused).
 * A store handle may be used from several threads at once. */
typedef struct kvc_store kvc_store;
kvc_status kvc_store_open(const char *root, const char *model_tag, int direct_io, kvc_store **out);
kvc_status kvc_store_close(kvc_store *store);
/* Writes the entry's path (NUL-terminated) into buf.  INVALID_ARG if cap is too small. */
kvc_status kvc_store_path(const kvc_store *store, uint64_t hash, char *buf, uint32_t cap);
/* KVC_OK and the file size, or KVC_ERR_NOT_FOUND (size 0). */
kvc_status kvc_store_lookup(const kvc_store *store, uint64_t hash, uint64_t *bytes);
/* Errors: INVALID_ARG, EXISTS, IO. */
kvc_status kvc_store_publish(kvc_store *store, uint64_t hash, const void *host_buf, uint64_t bytes);
/* Reads exactly `bytes`; INVALID_ARG if the entry has another size.  Errors: NOT_FOUND, IO. */
kvc_status kvc_store_read(kvc_store *store, uint64_t hash, void *host_buf, uint64_t bytes);
int kvc_store_direct_io_refused(const kvc_store *store);
/* Entries read and published through this handle so far, and their bytes (completed calls only):
 * with these a caller can check that a chunk shared by several requests was read once. */
typedef struct {
    uint64_t reads, read_bytes, publishes, publish_bytes;
} kvc_store_counters;
kvc_status kvc_store_get_counters(const kvc_store *store, kvc_store_counters *out);
/* Test seam (no counterpart in the paper): every file the store opens goes through `fn`
 * (path, open(2) flags, mode; returns a descriptor or -1 with errno set).  NULL restores open(2).
 * Process-wide.  Lets a host test play a file system that refuses O_DIRECT. */
typedef int (*kvc_open_fn)(const char *path, int flags, unsigned mode);
kvc_status kvc_store_set_open_fn(kvc_open_fn fn);

/* Prefix-hash chaining (Sec. 2.1): the hash of a block covers its tokens and the hash of the
 * block before it, so two requests share an entry only if they agree from the first token on.
 * 64-bit FNV-1a over the 8 bytes of `prev` (little endian) followed by the tokens' bytes;
 * prev = 0 starts a chain.  kvc_fnv1a64 is the plain hash of a byte string. */
uint64_t kvc_chain_hash(uint64_t prev, const int32_t *tokens, uint32_t n_tokens);
uint64_t kvc_fnv1a64(const void *data, uint64_t n);

/* ------------------------------------------------------------------ store / load pipelines (Sec. 6.4) */

typedef struct {
    uint64_t bytes;           /* chunk bytes written to / read from files */
    double seconds;           /* wall time of the call */
    uint32_t chunks;          /* chunks processed (load: length of the prefix that was present) */
    uint32_t published;       /* store: files this call created */
    uint32_t already_present; /* store: chunks another writer had published already */
    uint32_t ring_stalls;     /* polls that found no free slot */
} kvc_pipeline_stats;

/* Offload one request to chunk files: for every chunk (kvc_map_request order) acquire a ring slot,
 * pack the chunk's blocks into it on `stream`, and let one of `io_threads` (0 = 4) host threads
 * publish the slot as the file named by hashes[c] once its copy has completed; the slot returns
 * to the ring when the file is written.  `ring` must be a KVC_RING_HOST_MAPPED ring whose slots
 * hold a full chunk; the request may be far larger than the ring.  use_copy_engine != 0 packs
 * with the DMA engines (kvc_pack_copy_engine) instead of a kernel.  ids and hashes are HOST
 * arrays; n_hashes >= number of chunks.  Returns when every file is published.
 * kvc_pipeline_load is the reverse: it looks up the chunks in order, stops at the first one that
 * is missing or has the wrong size (only a contiguous prefix is usable, Sec. 2.1), reads the rest
 * into ring slots with the host threads and unpacks each slot into ids on `stream` as it arrives.
 * It returns when all files are read and all unpacks are ENQUEUED: synchronise `stream` before
 * using the blocks.  stats->chunks * blocks_per_chunk (capped by n_blocks) blocks were loaded.
 * Neither call is re-entrant on the same ring.
 * Errors: INVALID_ARG (no host-visible slots, slot too small, too few hashes), TIMEOUT, and
 * whatever pack / unpack / the store report. */
kvc_status kvc_pipeline_store(kvc_layout *layout, kvc_ring *ring, kvc_store *store, const int32_t *ids,
                              uint32_t n_blocks, const uint64_t *hashes, uint32_t n_hashes,
                              uint32_t io_threads, int use_copy_engine, void *stream,
                              kvc_pipeline_stats *stats);
kvc_status kvc_pipeline_load(kvc_layout *layout, kvc_ring *ring, kvc_store *store, const int32_t *ids,
                             uint32_t n_blocks, const uint64_t *hashes, uint32_t n_hashes,
                             uint32_t io_threads, int use_copy_engine, void *stream,
                             kvc_pipeline_stats *stats);
/* Both calls work on a FIFO ring and on a ring in pool mode (below); in pool mode the chunk hash
 * is the slot key, so a chunk that is already in the staging memory is neither packed nor read
 * again.  On any error exit every slot the call took is handed back: a slot whose copy was never
 * enqueued at once, the others after the copy or file operation in progress on them has ended;
 * queued file operations that had not started are dropped. */

/* ------------------------------------------------------------------ to and from HOST memory (Sec. 5.1, 6.4) */

/* A whole request between the paged pool and a HOST buffer, chunk by chunk through the ring: the
 * GPU <-> CPU transfer of Sec. 5.1 at the granularity of the layout's chunk_tokens, through the
 * bounded staging memory of Sec. 6.4, so the request may be far larger than the ring.
 *   kvc_offload_to_host: for every chunk (kvc_map_request order) acquire a slot, kvc_pack the
 *     chunk's blocks into it on `kernel_stream`, copy the slot to the host buffer on `copy_stream`
 *     (which waits for the slot's "filled" event only), release the slot behind that copy.
 *   kvc_load_from_host: the reverse -- host buffer -> slot on `copy_stream`, kvc_unpack into ids on
 *     `kernel_stream`, release behind the kernel.
 * The chunks lie back to back in the host buffer in request order (chunk c starts at the sum of
 * the earlier chunks' bytes; the last may be short); host_bytes must cover them all.  The host
 * buffer should be pinned: from pageable memory the runtime's copies stop being asynchronous.
 * `ring`: a FIFO ring (KVC_ERR_STATE in pool mode) of any kind whose slots hold a full chunk; with
 * KVC_RING_HOST_MAPPED the kernels cross the host link themselves and the copy is host to host.
 * The two streams may be the same; different streams let one chunk's kernel run beside another
 * chunk's copy.  The transfer is bound by the host link either way, so while a model is running
 * give the handle the KVC_PRESET_BESIDE_COMPUTE tuning: same link rate, a quarter of the cost to
 * the model.  ids is a HOST array and is validated as a whole before anything is enqueued
 * (OUT_OF_RANGE; load: CONFLICT on a repeated id anywhere in the request).
 * The calls block only while the ring is full (each wait for a slot is bounded by slot_timeout_us
 * > 0: TIMEOUT) and return when the last chunk is ENQUEUED: synchronise `copy_stream` (offload) or
 * `kernel_stream` (load) before using the result.  On an error exit nothing further is enqueued,
 * every slot taken is handed back, and stats->chunks says how many chunks were enqueued in full.
 * Not re-entrant on the same ring.
 * Errors: INVALID_ARG, STATE, OUT_OF_RANGE, CONFLICT, TIMEOUT, NOMEM, CUDA. */
typedef struct {
    uint64_t bytes;        /* chunk bytes enqueued for transfer */
    uint64_t ring_stalls;  /* polls that found the next slot still busy */
    uint32_t chunks;       /* chunks enqueued in full */
    uint32_t total_chunks; /* chunks of the request */
} kvc_host_transfer_stats;
kvc_status kvc_offload_to_host(kvc_layout *layout, kvc_ring *ring, const int32_t *ids, uint32_t n_blocks,
                               void *host_dst, uint64_t host_bytes, void *kernel_stream, void *copy_stream,
                               int64_t slot_timeout_us, kvc_host_transfer_stats *stats);
kvc_status kvc_load_from_host(kvc_layout *layout, kvc_ring *ring, const void *host_src, uint64_t host_bytes,
                              const int32_t *ids, uint32_t n_blocks, void *kernel_stream, void *copy_stream,
                              int64_t slot_timeout_us, kvc_host_transfer_stats *stats);

/* Several requests served at once from one staging pool (Sec. 6.4: every mapping that became ready
 * during one pass of the loop, from whichever request, goes into ONE fused unpack launch; Sec. 6.5:
 * demand loads before preloads, a chunk already in the pool -- being read, read, or cached -- is
 * joined, not read again; a finished preload waits in its slot until the demand load for the same
 * hash claims it).  `ring` must be in pool mode with host-visible slots.
 * Per request: ids (HOST, n_blocks destination blocks; unused for a preload), one hash per chunk,
 * and the class, KVC_CLASS_DEMAND_LOAD (chunks are unpacked into ids on `stream`) or
 * KVC_CLASS_PRELOAD (chunks are only brought into the pool, as far as the policy lets them).
 * For every request the contiguous prefix of chunks present in the store is processed;
 * loaded_chunks and ready_seconds (seconds from the start of the call until the request's last
 * unpack was enqueued, or its last chunk staged) are written back.  Destination blocks of different
 * requests must be distinct.  Returns when all reads are done and all unpacks ENQUEUED:
 * synchronise `stream` before using the blocks.  Not re-entrant on the same ring.
 * Errors: INVALID_ARG, STATE (ring not in pool mode, or a chunk is being filled by another user
 * of the pool), TIMEOUT, and whatever unpack / the store report. */
typedef struct {
    const int32_t *ids;
    uint32_t n_blocks;
    const uint64_t *hashes;
    uint32_t n_hashes;
    uint32_t cls;           /* kvc_slot_class: KVC_CLASS_DEMAND_LOAD or KVC_CLASS_PRELOAD */
    uint32_t loaded_chunks; /* out */
    double ready_seconds;   /* out */
} kvc_load_request;
typedef struct {
    uint64_t bytes_read;       /* bytes read from files by this call */
    double seconds;            /* wall time of the call */
    uint32_t chunks;           /* (request, chunk) pairs completed */
    uint32_t reads;            /* files read */
    uint32_t joins;            /* chunks served from a slot that already held them */
    uint32_t claims;           /* preloads claimed by demand loads (pool total so far) */
    uint32_t unpack_launches;  /* fused unpack launches */
    uint32_t ring_stalls;      /* acquisition attempts that found nothing available */
    uint32_t preloads_refused; /* preload chunks given up because the policy left no room */
} kvc_load_many_stats;
kvc_status kvc_pipeline_load_many(kvc_layout *layout, kvc_ring *ring, kvc_store *store,
                                  kvc_load_request *requests, uint32_t n_requests, uint32_t io_threads,
                                  void *stream, kvc_load_many_stats *stats);

/* ------------------------------------------------------------------ slot policy (Sec. 6.5) */

/* Who gets a staging slot when demand loads, stores and speculative preloads share one pool.
 * Host bookkeeping only (no CUDA call); slot indices name regions of the caller's staging memory.
 * Rules (Sec. 6.4, 6.5): `foreground_reserve` slots (the I/O depth) are kept for demand loads and
 * stores -- a preload gets a slot only while more than that many are free and fewer than
 * `max_speculative` preloads are in flight (0 = no limit); requests for a key (chunk hash) that
 * already holds a slot join it (reference count) instead of reading again, and a demand request
 * joining a preload claims it; with no free slot, foreground work takes over the least recently
 * used retained slot, else a staged preload nobody claimed or still holds; an unclaimed preload in flight can be
 * cancelled; with retain_completed != 0 released staged slots stay as a cache until taken over.
 * Not thread-safe. */
typedef struct kvc_slot_pool kvc_slot_pool;
typedef enum { KVC_CLASS_DEMAND_LOAD = 0, KVC_CLASS_STORE = 1, KVC_CLASS_PRELOAD = 2 } kvc_slot_class;
typedef struct {
    uint32_t n_free, n_in_flight, n_staged, n_retained; /* slots by state, now */
    uint64_t acquires;            /* slots handed out for a new operation */
    uint64_t joins;               /* requests that joined a slot already holding their key */
    uint64_t claims;              /* preloads taken over by a demand request for the same key */
    uint64_t reclaims;            /* retained or unclaimed staged slots taken over by foreground work */
    uint64_t cancels;             /* preloads cancelled in flight */
    uint64_t preload_refusals;    /* preloads refused by the reserve or the in-flight limit */
    uint64_t foreground_refusals; /* foreground requests that found nothing to take */
} kvc_slot_pool_counters;
kvc_status kvc_slot_pool_create(uint32_t n_slots, uint32_t foreground_reserve, uint32_t max_speculative,
                                int retain_completed, kvc_slot_pool **out);
kvc_status kvc_slot_pool_destroy(kvc_slot_pool *pool);
/* A slot for `key`.  *joined = 1: the key already has a slot (in flight, staged or retained); the
 * caller shares it and must not start another read.  *joined = 0: a slot was taken for a new
 * operation (state "in flight").  WOULD_BLOCK: nothing available for this class right now. */
kvc_status kvc_slot_pool_acquire(kvc_slot_pool *pool, kvc_slot_class cls, uint64_t key, uint32_t *slot,
                                 int *joined);
/* The slot's I/O has completed: the chunk is staged.  STATE unless in flight. */
kvc_status kvc_slot_pool_mark_staged(kvc_slot_pool *pool, uint32_t slot);
/* Drops one reference.  At zero the slot is freed -- or, if staged, kept: as a cache entry when
 * retention is on, or as a finished preload waiting to be claimed. */
kvc_status kvc_slot_pool_release(kvc_slot_pool *pool, uint32_t slot);
/* Gives up an unclaimed preload that is still in flight and has a single holder (its read is
 * abandoned and requeued by the caller).  STATE for anything else, including a preload that other
 * preload candidates have joined. */
kvc_status kvc_slot_pool_cancel(kvc_slot_pool *pool, uint32_t slot);
kvc_status kvc_slot_pool_get_counters(const kvc_slot_pool *pool, kvc_slot_pool_counters *out);
/* One slot's bookkeeping: state (kvc_slot_state), references held, key, and whether it is a
 * preload no demand request has claimed.  Any pointer may be NULL. */
typedef enum { KVC_SLOT_FREE = 0, KVC_SLOT_IN_FLIGHT = 1, KVC_SLOT_STAGED = 2, KVC_SLOT_RETAINED = 3 } kvc_slot_state;
kvc_status kvc_slot_pool_slot_info(const kvc_slot_pool *pool, uint32_t slot, uint32_t *state, uint32_t *refs,
                                   uint64_t *key, int *speculative);

/* ------------------------------------------------------------------ staging pool mode (Sec. 6.4, 6.5) */

/* The paper's staging memory is ONE pool shared by demand loads, stores and preloads, and any free
 * slot goes to the most urgent job that is ready (Sec. 6.4, 6.5); a FIFO ring cannot do that: a
 * slow file read on slot k would hold up every later slot.  kvc_staging_ring_set_policy switches a
 * ring whose slots are all free to pool mode: slots are then handed out in any order under the
 * slot-policy rules above (foreground reserve, bound on preloads in flight, one shared
 * reference-counted slot per key, claims, take-over of retained and of unclaimed staged slots),
 * and the two events per slot keep their meaning -- a slot returns to the policy only after the
 * event recorded behind its last GPU consumer has completed.
 *   acquire_for  class + key (chunk hash).  *joined = 0: a slot for a new operation; fill it, then
 *                commit / commit_host.  *joined = 1: the key already holds this slot (being filled,
 *                filled, or cached); the caller holds one more reference and must not fill it --
 *                kvc_staging_ring_slot_filled tells whether the bytes are there yet.
 *                timeout_us as for kvc_staging_ring_acquire.  Errors: WOULD_BLOCK, TIMEOUT, STATE
 *                (ring not in pool mode), NOMEM, CUDA.
 *   commit, commit_host, wait_filled, sync_filled: as in FIFO mode.
 *   release      drops ONE reference once the GPU work enqueued so far on consumer_stream has run
 *                (the slot's "drained" event is re-recorded behind every consumer, chained to the
 *                previous record); release_host drops one reference at once.  When the last
 *                reference is gone the slot is free -- or kept as a cached chunk (retention on) or
 *                as a finished preload waiting to be claimed, until foreground work takes it over.
 *   cancel       gives up an unclaimed preload that is still being filled (sole holder only).
 *   abandon      returns a slot that was acquired (not joined by anyone else) and will not be
 *                filled after all, e.g. because its copy could not be enqueued; also valid in
 *                FIFO mode.  STATE otherwise.
 * In pool mode kvc_staging_ring_acquire returns STATE, and the in_flight figure of
 * kvc_staging_ring_stats counts cached chunks as well. */
kvc_status kvc_staging_ring_set_policy(kvc_ring *ring, uint32_t foreground_reserve, uint32_t max_speculative,
                                       int retain_completed);
kvc_status kvc_staging_ring_acquire_for(kvc_ring *ring, kvc_slot_class cls, uint64_t key, int64_t timeout_us,
                                        uint32_t *slot, void **dev_ptr, void **host_ptr, int *joined);
kvc_status kvc_staging_ring_slot_filled(kvc_ring *ring, uint32_t slot, int *filled);
kvc_status kvc_staging_ring_cancel(kvc_ring *ring, uint32_t slot);
kvc_status kvc_staging_ring_abandon(kvc_ring *ring, uint32_t slot);
/* The policy's counters (after handing back references whose GPU work has completed). */
kvc_status kvc_staging_ring_policy_counters(kvc_ring *ring, kvc_slot_pool_counters *out);

/* Event provider used by a ring (test seam, no counterpart in the paper; the paper's rule it
 * serves is Sec. 6.4's "a slot is reused only after its CUDA event has completed").
 * The default one wraps CUDA events.  Tests replace it to
 * drive the slot state machine on a machine without a GPU (events that complete on command);
 * it must be installed before the ring is created and applies to rings created afterwards.
 * Passing NULL restores the CUDA provider. */
typedef struct {
    void *ctx;
    int (*create)(void *ctx, void **event);               /* 0 on success */
    int (*destroy)(void *ctx, void *event);
    int (*record)(void *ctx, void *event, void *stream);
    int (*query)(void *ctx, void *event);                 /* 0 done, 1 not yet, <0 error */
    int (*stream_wait)(void *ctx, void *stream, void *event);
    int (*synchronize)(void *ctx, void *event);
} kvc_event_provider;
kvc_status kvc_staging_ring_set_event_provider(const kvc_event_provider *provider);

#ifdef __cplusplus
}
#endif
#endif /* KVC_H */
