// The host side of the layout / mapper / launch front ends (kvc_layout.cu) under AddressSanitizer
// and UBSan on a machine without a GPU.  The file is compiled as plain C++; the CUDA runtime calls
// it names are replaced by host stand-ins (allocations come from malloc, copies are memcpy, events
// are dummies) and the kernel launch is replaced by a recorder that checks the plan it is given:
// nothing is copied -- what runs here is validation, the chunk mapper, the shared-prefix trie and
// the building of the per-block tables, i.e. everything that indexes host memory.
#include <cuda_runtime.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <vector>

#include "kvc_internal.h"

extern "C" {
cudaError_t cudaGetDevice(int *d) { *d = 0; return cudaSuccess; }
cudaError_t cudaGetLastError(void) { return cudaSuccess; }
cudaError_t cudaMalloc(void **p, size_t n) { *p = malloc(n ? n : 1); return *p ? cudaSuccess : cudaErrorMemoryAllocation; }
cudaError_t cudaFree(void *p) { free(p); return cudaSuccess; }
cudaError_t cudaHostAlloc(void **p, size_t n, unsigned) { *p = malloc(n ? n : 1); return *p ? cudaSuccess : cudaErrorMemoryAllocation; }
cudaError_t cudaFreeHost(void *p) { free(p); return cudaSuccess; }
cudaError_t cudaMemcpy(void *d, const void *s, size_t n, cudaMemcpyKind) { memcpy(d, s, n); return cudaSuccess; }
cudaError_t cudaMemcpyAsync(void *d, const void *s, size_t n, cudaMemcpyKind, cudaStream_t) { memcpy(d, s, n); return cudaSuccess; }
cudaError_t cudaMemset(void *d, int v, size_t n) { memset(d, v, n); return cudaSuccess; }
cudaError_t cudaMemsetAsync(void *d, int v, size_t n, cudaStream_t) { memset(d, v, n); return cudaSuccess; }
cudaError_t cudaStreamCreateWithFlags(cudaStream_t *s, unsigned) { *s = (cudaStream_t)malloc(1); return cudaSuccess; }
cudaError_t cudaStreamDestroy(cudaStream_t s) { free(s); return cudaSuccess; }
cudaError_t cudaStreamSynchronize(cudaStream_t) { return cudaSuccess; }
cudaError_t cudaStreamWaitEvent(cudaStream_t, cudaEvent_t, unsigned) { return cudaSuccess; }
cudaError_t cudaEventCreate(cudaEvent_t *e) { *e = (cudaEvent_t)malloc(1); return cudaSuccess; }
cudaError_t cudaEventCreateWithFlags(cudaEvent_t *e, unsigned) { *e = (cudaEvent_t)malloc(1); return cudaSuccess; }
cudaError_t cudaEventDestroy(cudaEvent_t e) { free(e); return cudaSuccess; }
cudaError_t cudaEventRecord(cudaEvent_t, cudaStream_t) { return cudaSuccess; }
cudaError_t cudaEventSynchronize(cudaEvent_t) { return cudaSuccess; }
cudaError_t cudaEventElapsedTime(float *ms, cudaEvent_t, cudaEvent_t) { *ms = 0.5f; return cudaSuccess; }
cudaError_t cudaPointerGetAttributes(cudaPointerAttributes *a, const void *)
{
    memset(a, 0, sizeof(*a));
    a->type = cudaMemoryTypeDevice;
    return cudaSuccess;
}
}

#define CHECK(x)                                                      \
    do {                                                              \
        if (!(x)) {                                                   \
            printf("FAILED line %d: %s\n", __LINE__, #x);             \
            exit(1);                                                  \
        }                                                             \
    } while (0)

// ---- stand-ins for the kernel side
static uint64_t g_launches = 0;
static uint32_t g_last_n_ent = 0;
cudaError_t kvc_kernel_limits(int *sm_count, int *vec_blocks_per_sm, int *max_smem_optin)
{
    *sm_count = 148;
    *vec_blocks_per_sm = 4;
    *max_smem_optin = 232448;
    return cudaSuccess;
}
cudaError_t kvc_launch_copy(int dir, int variant, const KvcLaunch &a, uint32_t grid, uint32_t smem, cudaStream_t)
{
    // what any kernel relies on
    CHECK(dir == KVC_DIR_PACK || dir == KVC_DIR_UNPACK);
    CHECK(grid >= 1 && (uint64_t)grid <= a.n_items && a.n_items >= 1);
    CHECK(smem <= 232448u && a.g.tile_bytes % 16 == 0 && a.g.tile_bytes >= 16);
    CHECK(a.g.slab_bytes % 16 == 0 && a.n_ent >= 1);
    const bool bulk = variant == KVC_VARIANT_BULK || variant == KVC_VARIANT_BULK_GROUP;
    if (bulk) {
        CHECK(a.stages >= 2 && a.stages <= KVC_BULK_MAX_STAGES && a.lag + 2 <= a.stages);
        CHECK(a.pending >= 1 && a.pending <= a.stages - 1 - a.lag);
        const uint32_t hdr = variant == KVC_VARIANT_BULK ? KVC_BULK_SMEM_HEADER : KVC_GROUP_SMEM_HEADER(a.stages);
        CHECK(smem == hdr + a.stages * a.g.tile_bytes);
    }
    if (variant == KVC_VARIANT_BULK_GROUP || variant == KVC_VARIANT_VEC_GROUP || variant == KVC_VARIANT_VEC32_GROUP) {
        CHECK(a.g.parts == 1 && (1u << a.group_shift) <= KVC_GROUP_MAX_SLABS);
        CHECK(a.g.tile_bytes == (a.g.slab_bytes << a.group_shift));
        CHECK(a.n_slabs == (uint64_t)a.n_ent * a.g.planes_total);
        CHECK(a.n_items == ((a.n_slabs + (1u << a.group_shift) - 1) >> a.group_shift));
    } else {
        CHECK(a.n_items == (uint64_t)a.n_ent * a.g.planes_total * a.g.parts);
        CHECK((uint64_t)a.g.parts * a.g.tile_bytes >= a.g.slab_bytes);
    }
    if (a.table) {  // the batched table: every entry readable, chunks consistent
        for (uint32_t i = 0; i < a.n_ent; ++i) {
            const KvcEnt &e = a.table[i];
            const uint32_t nb = e.nb_c & ~KVC_ENT_ID_IS_PTR;
            CHECK(nb >= 1 && e.first_ent <= i && i < e.first_ent + nb && e.first_ent + nb <= a.n_ent);
            CHECK(e.slot_addr % 16 == 0);
            if (!(e.nb_c & KVC_ENT_ID_IS_PTR))
                CHECK(e.id_or_ptr < a.g.num_blocks);
        }
    }
    g_last_n_ent = a.n_ent;
    ++g_launches;
    return cudaSuccess;
}

static uint32_t rnd(uint32_t *s)
{
    *s = *s * 1664525u + 1013904223u;
    return *s >> 8;
}

int main()
{
    uint32_t seed = 2609;
    std::vector<unsigned char> fake_pool(1 << 20), fake_slot(1 << 20);
    for (int round = 0; round < 200; ++round) {
        // a random geometry; the pool pointer is never dereferenced here
        kvc_layout_desc d;
        const uint32_t e = 1u << (rnd(&seed) % 3), H = 1 + rnd(&seed) % 8, D = 8u << (rnd(&seed) % 5);
        const uint32_t B = 1 + rnd(&seed) % 16, L = 1 + rnd(&seed) % 6, P = 1 + rnd(&seed) % 2;
        const uint32_t NB = 2 + rnd(&seed) % 300, bpc = 1 + rnd(&seed) % 20;
        CHECK(kvc_layout_desc_init_dense(&d, fake_pool.data(), L, P, NB, B, H, D, e, bpc * B,
                                         rnd(&seed) % 2) == KVC_OK);
        kvc_layout *lay = nullptr;
        kvc_status s = kvc_layout_create(&d, &lay);
        if ((uint64_t)B * H * D * e % 16) {
            CHECK(s == KVC_ERR_ALIGNMENT);
            continue;
        }
        CHECK(s == KVC_OK);
        kvc_tuning t;
        memset(&t, 0, sizeof(t));
        t.variant = rnd(&seed) % 3;
        t.group = rnd(&seed) % 4 == 0 ? 1 : (rnd(&seed) % 3 == 0 ? (1u << (rnd(&seed) % 6)) : 0);
        t.stages = rnd(&seed) % 3 == 0 ? 2 + rnd(&seed) % 15 : 0;
        t.lag = t.stages > 2 ? rnd(&seed) % (t.stages - 1) : 0;
        t.max_ctas = rnd(&seed) % 3 == 0 ? 1 + rnd(&seed) % 300 : 0;
        t.items_per_cta = rnd(&seed) % 4 == 0 ? 1 + rnd(&seed) % 50 : 0;
        t.tile_bytes = rnd(&seed) % 4 == 0 ? 16 * (1 + rnd(&seed) % 2048) : 0;
        t.vec_threads = rnd(&seed) % 4 == 0 ? 32 * (1 + rnd(&seed) % 8) : 0;
        t.order = rnd(&seed) % 4;
        t.slot_memory = rnd(&seed) % 2;
        CHECK(kvc_layout_set_tuning(lay, &t) == KVC_OK);
        if (round % 3 == 0)
            CHECK(kvc_layout_set_kernel_timing(lay, 1) == KVC_OK);
        // requests: random tables, some sharing a prefix
        const uint32_t n_req = 1 + rnd(&seed) % 6;
        std::vector<std::vector<int32_t>> tables(n_req);
        std::vector<int32_t> shared(rnd(&seed) % 40);
        for (int32_t &x : shared)
            x = (int32_t)(rnd(&seed) % NB);
        for (auto &tb : tables) {
            const uint32_t take = shared.empty() ? 0 : rnd(&seed) % (shared.size() + 1);
            tb.assign(shared.begin(), shared.begin() + take);
            for (uint32_t k = rnd(&seed) % 60; k; --k)
                tb.push_back((int32_t)(rnd(&seed) % NB));
        }
        std::vector<const int32_t *> ptrs;
        std::vector<uint32_t> lens;
        for (auto &tb : tables) {
            ptrs.push_back(tb.empty() ? nullptr : tb.data());
            lens.push_back((uint32_t)tb.size());
        }
        uint32_t n_desc = 0;
        uint64_t uniq = 0;
        CHECK(kvc_map_requests_shared(lay, ptrs.data(), lens.data(), n_req, 0, nullptr, 0, &n_desc, &uniq) == KVC_OK);
        std::vector<kvc_chunk_desc> descs(n_desc ? n_desc : 1);
        uint32_t n2 = 0;
        CHECK(kvc_map_requests_shared(lay, ptrs.data(), lens.data(), n_req, 0, descs.data(), n_desc, &n2, &uniq) == KVC_OK);
        CHECK(n2 == n_desc);
        uint64_t covered = 0;
        std::vector<kvc_chunk_op> ops;
        for (uint32_t i = 0; i < n_desc; ++i) {
            const kvc_chunk_desc &c = descs[i];
            CHECK(c.request < n_req && c.first + c.n_blocks <= lens[c.request] && c.n_blocks >= 1 && c.n_blocks <= bpc);
            CHECK(c.bytes == kvc_layout_chunk_bytes(lay, c.n_blocks));
            covered += c.n_blocks;
            kvc_chunk_op op;
            op.slot = fake_slot.data() + 16 * (rnd(&seed) % 64);
            op.ids = tables[c.request].data() + c.first;
            op.n_blocks = c.n_blocks;
            op.reserved = 0;
            ops.push_back(op);
        }
        CHECK(covered >= uniq);
        const uint64_t before = g_launches;
        s = kvc_pack_batch(lay, ops.data(), (uint32_t)ops.size(), 0, nullptr);
        CHECK(s == KVC_OK);
        CHECK(g_launches == before + (covered ? 1 : 0) && (!covered || g_last_n_ent == covered));
        s = kvc_unpack_batch(lay, ops.data(), (uint32_t)ops.size(), 0, nullptr);
        CHECK(s == KVC_OK || s == KVC_ERR_CONFLICT);  // random tables repeat ids
        // single-chunk calls: short (ids in the parameters) and long (through the table path)
        for (auto &tb : tables) {
            if (tb.empty())
                continue;
            const uint32_t nb = (uint32_t)tb.size();
            s = kvc_pack(lay, tb.data(), nb, 0, fake_slot.data(), kvc_layout_chunk_bytes(lay, nb), nullptr);
            CHECK(s == KVC_OK);
            CHECK(kvc_pack(lay, tb.data(), nb, 0, fake_slot.data(), kvc_layout_chunk_bytes(lay, nb) - 1, nullptr) ==
                  KVC_ERR_INVALID_ARG);
            tb[rnd(&seed) % nb] = (int32_t)NB;  // out of range
            CHECK(kvc_unpack(lay, fake_slot.data(), kvc_layout_chunk_bytes(lay, nb), tb.data(), nb, 0, nullptr) ==
                  KVC_ERR_OUT_OF_RANGE);
        }
        uint32_t timed = 0;
        double total = 0, lo = 0, hi = 0;
        CHECK(kvc_layout_kernel_time(lay, &timed, &total, &lo, &hi) == KVC_OK);
        CHECK(round % 3 != 0 || timed >= 1);
        uint32_t a = 7, b = 7;
        CHECK(kvc_poll_device_status(lay, nullptr, &a, &b) == KVC_OK && a == 0 && b == 0);
        CHECK(kvc_layout_destroy(lay) == KVC_OK);
    }
    CHECK(g_launches > 300);
    printf("ok\n");
    return 0;
}
