// Copy kernels of libkvc for sm_100a: paged-KV pack (gather) and unpack (scatter).
//
// A launch moves n_ent blocks x LP planes x `parts` tiles.  Work item w names one
// tile of one slab (the contiguous bytes of one block in one (layer, K|V) plane):
//     pool side : plane(lp) + id*block_stride + part*tile
//     slot side : chunk + j*ent_step + lp*plane_step + part*tile
//                 (layer-major chunk: ent_step = S, plane_step = nb_c*S)
// pack copies pool -> slot, unpack slot -> pool.  Nothing is a contraction: the
// kernels are bound by HBM bandwidth, so they only keep many full-line requests
// in flight and touch every byte once.
//
// Two ways to move a tile:
//   VEC  : every thread keeps KVC_VEC_UNROLL 16- or 32-byte loads in flight, then
//          stores them; streaming cache hints.
//   BULK : a one-warp block drives a few shared-memory stages with bulk async
//          copies (global -> shared, completion on an mbarrier; shared -> global,
//          completion by bulk group).  Lanes decode up to 32 work items at a time
//          and hand them to the issuing lane by shuffle.  Almost no registers or
//          issue slots are used, which leaves the SM's math pipes to other work.
// A block handles items blockIdx.x, blockIdx.x + gridDim.x, ...: with a large grid
// every block takes a couple of items and retires (the default), with a small one
// the blocks persist and stride over everything.
// Every byte is read exactly once by exactly one SM, so blocks never share tiles: no thread-block
// clusters are launched and every copy is addressed to the issuing block's own shared memory.
#include <string.h>

#include <atomic>
#include <mutex>

#include "kvc_internal.h"

namespace {

struct Item {
    uint64_t pool;  // address on the paged-pool side
    uint64_t slot;  // address on the staging side
    uint32_t len;   // bytes; 0 = skip (block id out of range)
};

__device__ __forceinline__ uint64_t plane_base(const KvcGeom &g, uint32_t lp)
{
    if (g.plane_table != nullptr)
        return __ldg(reinterpret_cast<const unsigned long long *>(g.plane_table) + lp);
    uint32_t l = lp / g.planes_per_layer, p = lp - l * g.planes_per_layer;
    return (uint64_t)g.base + (uint64_t)l * g.layer_stride + (uint64_t)p * g.plane_stride;
}

// Work item -> addresses.  TABLE: entries come from device memory (batched launch);
// otherwise ids are in the kernel parameters or in a device id array (one chunk).
template <bool TABLE>
__device__ __forceinline__ Item decode(const KvcLaunch &a, uint32_t w, bool count_bad)
{
    const KvcGeom &g = a.g;
    uint32_t part = w % g.parts;
    uint32_t r = w / g.parts;
    uint32_t ent, lp;
    if (a.order == KVC_ORDER_PLANE_MAJOR) {
        lp = r / a.n_ent;
        ent = r - lp * a.n_ent;
    } else if (a.order == KVC_ORDER_BLOCK_MAJOR) {
        ent = r / g.planes_total;
        lp = r - ent * g.planes_total;
    } else {
        // chunk-major: slabs in the order they lie in staging memory, chunk after chunk.  Slab r
        // belongs to the chunk that owns entry r / LP (a chunk of nb blocks owns nb*LP slabs
        // starting at slab first_ent*LP); inside the chunk, q walks the chunk linearly.
        uint32_t first = 0, nb = a.n_ent;
        if (TABLE) {
            const uint4 probe = __ldg(reinterpret_cast<const uint4 *>(a.table + r / g.planes_total) + 1);
            nb = probe.z & ~KVC_ENT_ID_IS_PTR;
            first = probe.w;
        }
        const uint32_t q = r - first * g.planes_total;
        uint32_t j;
        if (a.block_major_chunks) {
            j = q / g.planes_total;
            lp = q - j * g.planes_total;
        } else {
            lp = q / nb;
            j = q - lp * nb;
        }
        ent = first + j;
    }
    uint64_t slot_j, plane_step;
    int64_t id;
    if (TABLE) {
        const uint4 *e = reinterpret_cast<const uint4 *>(a.table + ent);
        uint4 lo = __ldg(e), hi = __ldg(e + 1);
        slot_j = ((uint64_t)lo.y << 32) | lo.x;
        uint64_t idp = ((uint64_t)lo.w << 32) | lo.z;
        plane_step = ((uint64_t)hi.y << 32) | hi.x;
        id = (hi.z & KVC_ENT_ID_IS_PTR) ? (int64_t)__ldg(reinterpret_cast<const int32_t *>(idp))
                                        : (int64_t)(int32_t)lo.z;
    } else {
        slot_j = a.slot + (uint64_t)ent * a.ent_step;
        plane_step = a.plane_step;
        id = a.dev_ids ? (int64_t)__ldg(a.dev_ids + ent) : (int64_t)a.ids[ent];
    }
    Item it;
    uint32_t off = part * g.tile_bytes;
    it.len = min(g.tile_bytes, g.slab_bytes - off);
    if (id < 0 || id >= (int64_t)g.num_blocks) {
        // never touch memory for a bad id: count the block once and skip it
        if (count_bad && part == 0 && lp == 0)
            atomicAdd(a.status, 1u);
        it.len = 0;
        id = 0;
    }
    it.pool = plane_base(g, lp) + (uint64_t)id * g.block_stride + off;
    it.slot = slot_j + (uint64_t)lp * plane_step + off;
    return it;
}

// Programmatic dependent launch: when the launch carries the stream-serialisation attribute, the
// grid may be scheduled while the previous kernel of the stream is still draining.  Nothing in
// global memory may be read before grid_dependency_wait() returns (it waits for the previous
// grid to complete and its writes to be visible); after it, the next kernel is let in early.
// Without the attribute both instructions do nothing.
// With overlap != 0 the wait is skipped: the caller has declared that this launch does not touch
// what the previous kernel of the stream reads or writes, so its blocks may run beside that
// kernel's last blocks (work that preceded the previous kernel has completed either way, because
// that kernel could not start before it).
__device__ __forceinline__ void grid_dependency_wait(uint32_t overlap = 0)
{
    if (!overlap)
        asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

// ------------------------------------------------------------------------------------ VEC

// A VB-byte vector held in registers.  VB = 32 uses the 256-bit global accesses of sm_100,
// which also accept an L2 evict-first priority (the data is touched once); VB = 16 is the
// path for layouts that are only 16-byte aligned.  The loads are ordinary coherent loads, not
// the read-only (.nc) form: with programmatic dependent launch a grid can be resident while an
// earlier grid of the stream is still writing the same pool blocks, and the read-only path
// promises nothing about data that changes during the kernel's lifetime.
template <int VB>
struct Vec;

template <>
struct Vec<16> {
    uint32_t r[4];
    __device__ __forceinline__ void load(uint64_t addr)
    {
        asm volatile("ld.global.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                     : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                     : "l"(addr));
    }
    __device__ __forceinline__ void store(uint64_t addr) const
    {
        asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(addr), "r"(r[0]), "r"(r[1]),
                     "r"(r[2]), "r"(r[3])
                     : "memory");
    }
};

template <>
struct Vec<32> {
    uint32_t r[8];
    __device__ __forceinline__ void load(uint64_t addr)
    {
        asm volatile(
            "ld.global.L1::no_allocate.L2::evict_first.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
            : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]),
              "=r"(r[7])
            : "l"(addr));
    }
    __device__ __forceinline__ void store(uint64_t addr) const
    {
        asm volatile(
            "st.global.L1::no_allocate.L2::evict_first.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(
                addr),
            "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
            : "memory");
    }
};

// TEAM threads share one work item: the whole block for ordinary tiles, one warp for tiles of at
// most 4 KiB (small slabs), so that eight small items are in flight per block instead of one.
template <int DIR, bool TABLE, int VB, int TEAM>
__global__ void __launch_bounds__(KVC_VEC_THREADS)
kvc_vec_kernel(const __grid_constant__ KvcLaunch a)
{
    constexpr uint32_t SH = VB == 32 ? 5 : 4;
    const uint32_t TEAMS = blockDim.x / TEAM;  // blocks of fewer than 256 threads: warp teams only
    const uint32_t t = threadIdx.x % TEAM;
    const uint32_t n_items = (uint32_t)a.n_items;
    const uint64_t stride = (uint64_t)gridDim.x * TEAMS;
    uint64_t w = (uint64_t)blockIdx.x * TEAMS + threadIdx.x / TEAM;
    grid_dependency_wait(a.pdl == 2u);
    if (w >= n_items)
        return;
    Item cur = decode<TABLE>(a, (uint32_t)w, t == 0);
    while (true) {
        // decode the next item before the copy so its table read overlaps the data loads
        const uint64_t wn = w + stride;
        const bool more = wn < n_items;
        Item nxt = cur;
        if (more)
            nxt = decode<TABLE>(a, (uint32_t)wn, t == 0);
        const uint64_t src = DIR == KVC_DIR_PACK ? cur.pool : cur.slot;
        const uint64_t dst = DIR == KVC_DIR_PACK ? cur.slot : cur.pool;
        const uint32_t nvec = cur.len >> SH;
        for (uint32_t v0 = 0; v0 < nvec; v0 += TEAM * KVC_VEC_UNROLL) {
            Vec<VB> r[KVC_VEC_UNROLL];
#pragma unroll
            for (uint32_t u = 0; u < KVC_VEC_UNROLL; ++u) {
                uint32_t v = v0 + u * TEAM + t;
                if (v < nvec)
                    r[u].load(src + ((uint64_t)v << SH));
            }
#pragma unroll
            for (uint32_t u = 0; u < KVC_VEC_UNROLL; ++u) {
                uint32_t v = v0 + u * TEAM + t;
                if (v < nvec)
                    r[u].store(dst + ((uint64_t)v << SH));
            }
        }
        if (!more)
            break;
        cur = nxt;
        w = wn;
    }
}


// ------------------------------------------------------------------------------------ VEC, several slabs per item
//
// Small slabs (a tensor-parallel shard of the KV heads, 1-byte elements, small blocks): the cost
// that matters is per slab -- the table lookups of the decode -- and the remedy is many warps,
// each with many independent loads in flight.  A work item is a run of R = 2^group_shift
// consecutive slabs (in slot order) given to ONE warp: lane i decodes slab i, then the warp copies
// the R*S bytes as one stream of vectors, each lane fetching the addresses of the slab its vector
// falls in from the decoding lane by shuffle.  The next item is decoded before the current one is
// copied, so the lookups overlap the copies.
template <int DIR, bool TABLE, int VB>
__global__ void __launch_bounds__(KVC_VEC_THREADS)
kvc_vec_group_kernel(const __grid_constant__ KvcLaunch a)
{
    constexpr uint32_t SH = VB == 32 ? 5 : 4;
    constexpr uint32_t U = VB == 32 ? 4 : 8;     // 128 bytes in flight per lane
    const uint32_t WARPS = blockDim.x / 32u;
    constexpr uint32_t FULL = 0xffffffffu;
    const uint32_t lane = threadIdx.x & 31u;
    const uint32_t ksh = a.group_shift, R = 1u << ksh;
    const uint32_t vps = a.g.slab_bytes >> SH;    // vectors per slab
    const uint32_t total = R * vps;               // vectors per item
    const uint64_t magic = a.vec_magic;
    const uint64_t n_items = a.n_items, n_slabs = a.n_slabs;
    const uint64_t stride = (uint64_t)gridDim.x * WARPS;
    uint64_t w = (uint64_t)blockIdx.x * WARPS + (threadIdx.x >> 5);
    grid_dependency_wait(a.pdl == 2u);
    if (w >= n_items)
        return;
    auto decode_mine = [&](uint64_t item) {
        Item it;
        it.pool = it.slot = 0;
        it.len = 0;
        const uint64_t r = (item << ksh) + lane;
        if (lane < R && r < n_slabs)
            it = decode<TABLE>(a, (uint32_t)r, true);
        return it;
    };
    Item cur = decode_mine(w);
    while (true) {
        const uint64_t wn = w + stride;
        const bool more = wn < n_items;
        Item nxt = cur;
        if (more)
            nxt = decode_mine(wn);
        const uint64_t my_src = DIR == KVC_DIR_PACK ? cur.pool : cur.slot;
        const uint64_t my_dst = DIR == KVC_DIR_PACK ? cur.slot : cur.pool;
        for (uint32_t v0 = 0; v0 < total; v0 += 32u * U) {
            Vec<VB> r[U];
            uint64_t d[U];
            bool live[U];
#pragma unroll
            for (uint32_t u = 0; u < U; ++u) {
                const uint32_t v = v0 + u * 32u + lane;
                uint32_t slab = (uint32_t)(((uint64_t)v * magic) >> 32);  // v / vps
                slab = min(slab, R - 1u);
                const uint32_t off = (v - slab * vps) << SH;
                const uint64_t sa = __shfl_sync(FULL, my_src, slab);
                const uint64_t da = __shfl_sync(FULL, my_dst, slab);
                const uint32_t len = __shfl_sync(FULL, cur.len, slab);
                live[u] = v < total && len != 0;
                d[u] = da + off;
                if (live[u])
                    r[u].load(sa + off);
            }
#pragma unroll
            for (uint32_t u = 0; u < U; ++u)
                if (live[u])
                    r[u].store(d[u]);
        }
        if (!more)
            break;
        cur = nxt;
        w = wn;
    }
}

// ------------------------------------------------------------------------------------ BULK

__device__ __forceinline__ uint32_t smem_u32(const void *p)
{
    return (uint32_t)__cvta_generic_to_shared(p);
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}

__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
                 : "memory");
}

// Bounded wait for a phase of an mbarrier.  Returns false if it gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity)
{
    for (uint32_t i = 0; i < KVC_WAIT_LIMIT; ++i) {
        uint32_t done;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done)
            : "r"(bar), "r"(parity)
            : "memory");
        if (done)
            return true;
    }
    return false;
}

__device__ __forceinline__ void bulk_load(uint32_t dst_smem, uint64_t src, uint32_t bytes,
                                          uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.shared::cta.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::
            "r"(dst_smem),
        "l"(src), "r"(bytes), "r"(bar)
        : "memory");
}

__device__ __forceinline__ void bulk_store(uint64_t dst, uint32_t src_smem, uint32_t bytes)
{
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst),
                 "r"(src_smem), "r"(bytes)
                 : "memory");
}

__device__ __forceinline__ uint64_t policy_evict_first()
{
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}

__device__ __forceinline__ void bulk_load_hint(uint32_t dst_smem, uint64_t src, uint32_t bytes,
                                               uint32_t bar, uint64_t pol)
{
    asm volatile(
        "cp.async.bulk.shared::cta.global.mbarrier::complete_tx::bytes.L2::cache_hint "
        "[%0], [%1], %2, [%3], %4;" ::"r"(dst_smem),
        "l"(src), "r"(bytes), "r"(bar), "l"(pol)
        : "memory");
}

__device__ __forceinline__ void bulk_store_hint(uint64_t dst, uint32_t src_smem, uint32_t bytes,
                                                uint64_t pol)
{
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group.L2::cache_hint [%0], [%1], %2, %3;" ::
                     "l"(dst),
                 "r"(src_smem), "r"(bytes), "l"(pol)
                 : "memory");
}

__device__ __forceinline__ void bulk_commit()
{
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}

// Wait until at most N of this thread's most recent bulk groups still read shared memory.
template <int N>
__device__ __forceinline__ void bulk_wait_read()
{
    asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}

// The instruction takes an immediate; the launch picks how many stores may stay outstanding.
__device__ __forceinline__ void bulk_wait_read_n(uint32_t n)
{
    switch (n) {
    case 0: bulk_wait_read<0>(); break;
    case 1: bulk_wait_read<1>(); break;
    case 2: bulk_wait_read<2>(); break;
    case 3: bulk_wait_read<3>(); break;
    case 4: bulk_wait_read<4>(); break;
    case 5: bulk_wait_read<5>(); break;
    case 6: bulk_wait_read<6>(); break;
    default: bulk_wait_read<7>(); break;
    }
}

__device__ __forceinline__ void bulk_wait_all()
{
    asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
}

#define KVC_BULK_PENDING 1  // stores allowed to be still reading shared memory when a stage is reused

// One warp per block.  Item k of this block uses stage k % stages.  Step k issues the load of
// item k and the store of item k - lag, so `lag` loads are in flight while stores drain.
template <int DIR, bool TABLE>
__global__ void __launch_bounds__(KVC_BULK_THREADS, 1)
kvc_bulk_kernel(const __grid_constant__ KvcLaunch a)
{
    extern __shared__ __align__(1024) unsigned char smem[];
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem);                       // [stages]
    uint64_t *st_dst = reinterpret_cast<uint64_t *>(smem + 128);               // [stages]
    uint32_t *st_len = reinterpret_cast<uint32_t *>(smem + 256);               // [stages]
    unsigned char *data = smem + KVC_BULK_SMEM_HEADER;

    const uint32_t lane = threadIdx.x;
    const uint32_t stages = a.stages, lag = a.lag, tile = a.g.tile_bytes;
    const uint32_t n_items = (uint32_t)a.n_items;
    if (blockIdx.x >= n_items) {
        grid_dependency_wait(a.pdl == 2u);
        return;
    }
    const uint32_t K = (n_items - blockIdx.x + gridDim.x - 1) / gridDim.x;  // my items

    if (lane == 0) {
        for (uint32_t s = 0; s < stages; ++s)
            mbar_init(smem_u32(&bars[s]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    grid_dependency_wait(a.pdl == 2u);
    __syncwarp();

    const bool hint_ld = (a.l2_evict_first & 1u) != 0, hint_st = (a.l2_evict_first & 2u) != 0;
    const uint64_t pol = policy_evict_first();
    bool ok = true;          // lane 0: no wait has expired
    uint32_t loads_done = 0; // lane 0: items whose load was issued (for the drain on failure)
    uint32_t stores_done = 0;
    Item mine;
    mine.pool = mine.slot = 0;
    mine.len = 0;
    for (uint32_t k0 = 0; k0 < K + lag; k0 += 32) {
        // every lane decodes one of the next 32 items of this block
        uint32_t kk = k0 + lane;
        if (kk < K)
            mine = decode<TABLE>(a, blockIdx.x + kk * gridDim.x, true);
        else
            mine.len = 0;
        for (uint32_t i = 0; i < 32; ++i) {
            const uint32_t k = k0 + i;
            if (k >= K + lag)
                break;
            // broadcast item k from lane i
            uint64_t pool = __shfl_sync(0xffffffffu, mine.pool, i);
            uint64_t slot = __shfl_sync(0xffffffffu, mine.slot, i);
            uint32_t len = __shfl_sync(0xffffffffu, mine.len, i);
            if (lane == 0 && ok) {
                if (k < K) {
                    const uint32_t s = k % stages;
                    if (k >= stages)
                        bulk_wait_read<KVC_BULK_PENDING>();  // store of item k-stages has left stage s
                    const uint32_t bar = smem_u32(&bars[s]);
                    st_dst[s] = DIR == KVC_DIR_PACK ? slot : pool;
                    st_len[s] = len;
                    mbar_expect_tx(bar, len);
                    if (len) {
                        const uint64_t from = DIR == KVC_DIR_PACK ? pool : slot;
                        if (hint_ld)
                            bulk_load_hint(smem_u32(data + (size_t)s * tile), from, len, bar, pol);
                        else
                            bulk_load(smem_u32(data + (size_t)s * tile), from, len, bar);
                    }
                    loads_done = k + 1;
                }
                if (k >= lag) {
                    const uint32_t m = k - lag;
                    const uint32_t s = m % stages;
                    if (mbar_wait(smem_u32(&bars[s]), (m / stages) & 1u)) {
                        const uint32_t l2 = st_len[s];
                        if (l2) {
                            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                            if (hint_st)
                                bulk_store_hint(st_dst[s], smem_u32(data + (size_t)s * tile), l2, pol);
                            else
                                bulk_store(st_dst[s], smem_u32(data + (size_t)s * tile), l2);
                        }
                        bulk_commit();
                        stores_done = m + 1;
                    } else {
                        ok = false;
                        atomicAdd(a.status + 1, 1u);
                    }
                }
            }
        }
    }
    if (lane == 0) {
        if (!ok) {
            // A wait gave up.  Loads that were issued may still land in shared memory: give each
            // one more bounded wait so the block does not retire under an incoming copy.
            for (uint32_t m = stores_done; m < loads_done; ++m)
                (void)mbar_wait(smem_u32(&bars[m % stages]), (m / stages) & 1u);
        }
        bulk_wait_all();
    }
}


// ------------------------------------------------------------------------------------ BULK, several slabs per item
//
// For slabs much smaller than a tile the per-item cost of the kernel above (decode, one mbarrier
// round trip, one bulk group) is paid per slab and the throughput falls with the slab size.  Here
// a work item is a run of k = 2^group_shift consecutive slabs in the order the chunk's bytes lie
// in the slot -- at most one tile.  Consecutive slabs of a chunk are contiguous on the slot side
// (both chunk byte orders), so an item is k copies on the pool side and ONE copy on the slot side
// (two where the run crosses into the next chunk; contiguity is detected from the addresses, so
// any traversal order stays correct).  The k lanes of a segment of the warp each decode one slab
// and issue their own pool-side copy; all completions of an item count, in bytes, on the stage's
// one mbarrier.  Every lane commits one bulk group per item, issued or not, so group counts are
// the same on all lanes and one wait_group.read per lane orders the whole warp's stage reuse.
struct GroupStageInfo {
    uint64_t dst[KVC_GROUP_MAX_SLABS];  // where the stage's stores go
    uint32_t len[KVC_GROUP_MAX_SLABS];  // bytes of each (0 = none)
};
static_assert(sizeof(GroupStageInfo) == KVC_GROUP_STAGE_INFO_BYTES, "shared-memory header layout");

template <int DIR, bool TABLE>
__global__ void __launch_bounds__(KVC_BULK_THREADS, 1)
kvc_bulk_group_kernel(const __grid_constant__ KvcLaunch a)
{
    extern __shared__ __align__(1024) unsigned char smem[];
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem);                       // [stages]
    GroupStageInfo *info = reinterpret_cast<GroupStageInfo *>(smem + 128);     // [stages]
    constexpr uint32_t FULL = 0xffffffffu;

    const uint32_t lane = threadIdx.x;
    const uint32_t stages = a.stages, lag = a.lag, tile = a.g.tile_bytes, S = a.g.slab_bytes;
    const uint32_t ksh = a.group_shift, k = 1u << ksh;
    const uint32_t n_items = (uint32_t)a.n_items;
    const uint64_t n_slabs = a.n_slabs;
    unsigned char *data = smem + KVC_GROUP_SMEM_HEADER(stages);
    if (blockIdx.x >= n_items) {
        grid_dependency_wait(a.pdl == 2u);
        return;
    }
    const uint32_t K = (n_items - blockIdx.x + gridDim.x - 1) / gridDim.x;  // my items

    if (lane == 0) {
        for (uint32_t s = 0; s < stages; ++s)
            mbar_init(smem_u32(&bars[s]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    grid_dependency_wait(a.pdl == 2u);
    __syncwarp();

    const uint32_t per_round = 32u >> ksh;          // items decoded per round
    const uint32_t seg = lane >> ksh, sub = lane & (k - 1u);
    bool ok = true;                                  // no wait has expired (same on all lanes)
    uint32_t loads_done = 0, stores_done = 0;
    Item mine;
    mine.pool = mine.slot = 0;
    mine.len = 0;
    for (uint32_t k0 = 0; k0 < K + lag; k0 += per_round) {
        // lane (seg, sub) decodes slab `sub` of this block's item k0 + seg
        mine.len = 0;
        if (k0 + seg < K) {
            const uint64_t r = (((uint64_t)blockIdx.x + (uint64_t)(k0 + seg) * gridDim.x) << ksh) + sub;
            if (r < n_slabs)
                mine = decode<TABLE>(a, (uint32_t)r, true);
        }
        for (uint32_t m = 0; m < per_round; ++m) {
            const uint32_t step = k0 + m;
            if (step >= K + lag)
                break;
            if (ok && step < K) {
                const uint32_t s = step % stages;
                if (step >= stages)
                    bulk_wait_read_n(a.pending);  // the stores that last drained stage s have left it
                __syncwarp();
                const bool active = seg == m;
                const bool valid = active && mine.len != 0;
                // runs of slabs that are contiguous on the slot side
                const uint64_t prev_slot = __shfl_up_sync(FULL, mine.slot, 1);
                const uint32_t prev_len = __shfl_up_sync(FULL, mine.len, 1);
                const bool head = valid && (sub == 0 || prev_len == 0 || prev_slot + prev_len != mine.slot);
                const uint32_t vmask = __ballot_sync(FULL, valid);
                const uint32_t hmask = __ballot_sync(FULL, head);
                const uint32_t seg_lo = m << ksh;
                const uint32_t segmask = k == 32u ? FULL : (((1u << k) - 1u) << seg_lo);
                uint32_t run = 0;  // bytes of the merged copy this lane heads
                if (head) {
                    const uint32_t bound = (hmask | ~vmask) & segmask;
                    const uint32_t above = lane == 31u ? 0u : (bound & (FULL << (lane + 1u)));
                    const uint32_t next = above ? (uint32_t)__ffs((int)above) - 1u : seg_lo + k;
                    run = (next - lane) * S;
                }
                const uint32_t bar = smem_u32(&bars[s]);
                if (active && sub == 0)
                    mbar_expect_tx(bar, (uint32_t)__popc(vmask) * S);
                __syncwarp();
                const uint32_t stage_at = smem_u32(data + (size_t)s * tile + (size_t)sub * S);
                if (DIR == KVC_DIR_PACK) {
                    if (valid)
                        bulk_load(stage_at, mine.pool, S, bar);
                    if (active) {
                        info[s].dst[sub] = mine.slot;
                        info[s].len[sub] = run;
                    }
                } else {
                    if (head)
                        bulk_load(stage_at, mine.slot, run, bar);
                    if (active) {
                        info[s].dst[sub] = mine.pool;
                        info[s].len[sub] = valid ? S : 0u;
                    }
                }
                loads_done = step + 1;
            }
            if (ok && step >= lag) {
                const uint32_t mm = step - lag;
                const uint32_t s = mm % stages;
                __syncwarp();
                const bool done =
                    __all_sync(FULL, mbar_wait(smem_u32(&bars[s]), (mm / stages) & 1u));
                if (done) {
                    if (lane < k) {
                        const uint32_t len = info[s].len[lane];
                        if (len) {
                            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                            bulk_store(info[s].dst[lane],
                                       smem_u32(data + (size_t)s * tile + (size_t)lane * S), len);
                        }
                    }
                    bulk_commit();
                    stores_done = mm + 1;
                } else {
                    ok = false;
                    if (lane == 0)
                        atomicAdd(a.status + 1, 1u);
                }
            }
        }
    }
    if (!ok) {
        // A wait gave up.  Loads that were issued may still land in shared memory: give each one
        // more bounded wait so the block does not retire under an incoming copy.
        for (uint32_t m = stores_done; m < loads_done; ++m)
            (void)mbar_wait(smem_u32(&bars[m % stages]), (m / stages) & 1u);
    }
    bulk_wait_all();
}

template <typename K>
cudaError_t launch_cfg(K kernel, const KvcLaunch &a, uint32_t grid, uint32_t block, uint32_t smem,
                       cudaStream_t stream)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(block);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = a.pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, a);
}

// The opt-in dynamic shared-memory size is a per-device attribute of each kernel and is only
// ever raised.  Handles on different host threads may make their first launches at the same
// time with different tunings: the raise happens under a lock, the common case is one atomic load.
template <typename K>
cudaError_t ensure_smem(K kernel, int which, uint32_t smem)
{
    static std::atomic<int> configured[64][8];
    static std::mutex mu;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess)
        return e;
    if (dev < 0 || dev >= 64)
        return cudaErrorInvalidDevice;
    std::atomic<int> &have = configured[dev][which];
    if ((int)smem <= have.load(std::memory_order_acquire))
        return cudaSuccess;
    std::lock_guard<std::mutex> lock(mu);
    if ((int)smem > have.load(std::memory_order_relaxed)) {
        e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess)
            return e;
        have.store((int)smem, std::memory_order_release);
    }
    return cudaSuccess;
}

template <int DIR, bool TABLE>
cudaError_t launch_one(int variant, const KvcLaunch &a, uint32_t grid, uint32_t smem,
                       cudaStream_t stream)
{
    if (variant == KVC_VARIANT_BULK) {
        cudaError_t e = ensure_smem(kvc_bulk_kernel<DIR, TABLE>, DIR * 2 + (TABLE ? 1 : 0), smem);
        if (e != cudaSuccess)
            return e;
        return launch_cfg(kvc_bulk_kernel<DIR, TABLE>, a, grid, KVC_BULK_THREADS, smem, stream);
    }
    if (variant == KVC_VARIANT_BULK_GROUP) {
        cudaError_t e = ensure_smem(kvc_bulk_group_kernel<DIR, TABLE>, 4 + DIR * 2 + (TABLE ? 1 : 0), smem);
        if (e != cudaSuccess)
            return e;
        return launch_cfg(kvc_bulk_group_kernel<DIR, TABLE>, a, grid, KVC_BULK_THREADS, smem, stream);
    }
    // kernels that give every warp its own work item run with any whole number of warps per block
    const uint32_t wt = a.vec_threads ? a.vec_threads : KVC_VEC_THREADS;
    if (variant == KVC_VARIANT_VEC32_GROUP)
        return launch_cfg(kvc_vec_group_kernel<DIR, TABLE, 32>, a, grid, wt, 0, stream);
    if (variant == KVC_VARIANT_VEC_GROUP)
        return launch_cfg(kvc_vec_group_kernel<DIR, TABLE, 16>, a, grid, wt, 0, stream);
    const bool warp_team = a.g.tile_bytes <= KVC_VEC_WARP_TEAM_MAX_TILE;
    if (variant == KVC_VARIANT_VEC32)
        return warp_team
                   ? launch_cfg(kvc_vec_kernel<DIR, TABLE, 32, 32>, a, grid, wt, 0, stream)
                   : launch_cfg(kvc_vec_kernel<DIR, TABLE, 32, KVC_VEC_THREADS>, a, grid, KVC_VEC_THREADS,
                                0, stream);
    return warp_team
               ? launch_cfg(kvc_vec_kernel<DIR, TABLE, 16, 32>, a, grid, wt, 0, stream)
               : launch_cfg(kvc_vec_kernel<DIR, TABLE, 16, KVC_VEC_THREADS>, a, grid, KVC_VEC_THREADS, 0,
                            stream);
}

}  // namespace

cudaError_t kvc_launch_copy(int dir, int variant, const KvcLaunch &a, uint32_t grid,
                            uint32_t smem_bytes, cudaStream_t stream)
{
    const bool table = a.table != nullptr;
    if (dir == KVC_DIR_PACK)
        return table ? launch_one<KVC_DIR_PACK, true>(variant, a, grid, smem_bytes, stream)
                     : launch_one<KVC_DIR_PACK, false>(variant, a, grid, smem_bytes, stream);
    return table ? launch_one<KVC_DIR_UNPACK, true>(variant, a, grid, smem_bytes, stream)
                 : launch_one<KVC_DIR_UNPACK, false>(variant, a, grid, smem_bytes, stream);
}

cudaError_t kvc_kernel_limits(int *sm_count, int *vec_blocks_per_sm, int *max_smem_optin)
{
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess)
        return e;
    if ((e = cudaDeviceGetAttribute(sm_count, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess)
        return e;
    if ((e = cudaDeviceGetAttribute(max_smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev)) !=
        cudaSuccess)
        return e;
    return cudaOccupancyMaxActiveBlocksPerMultiprocessor(
        vec_blocks_per_sm, kvc_vec_kernel<KVC_DIR_PACK, true, 32, KVC_VEC_THREADS>, KVC_VEC_THREADS, 0);
}
