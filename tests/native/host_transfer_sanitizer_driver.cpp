// kvc_offload_to_host / kvc_load_from_host under AddressSanitizer and UBSan on a machine without
// a GPU.  The library's host code (layout front ends, ring, slot policy, the host-transfer loop) is
// compiled as plain C++; the CUDA runtime is replaced by host stand-ins (memory from malloc, copies
// are memcpy, events complete at once) and the kernel launch by a plain loop that moves the slabs
// the launch parameters name.  So whole requests really travel pool -> ring slots -> host buffer and
// back on the host, every buffer is exactly as large as the interface says it must be, and the
// sanitizers watch every byte.  Expected bytes come from the chunk layout written out below.
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
cudaError_t cudaHostGetDevicePointer(void **d, void *h, unsigned) { *d = h; return cudaSuccess; }
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
cudaError_t cudaEventQuery(cudaEvent_t) { return cudaSuccess; }
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

static uint64_t g_launches = 0;
cudaError_t kvc_kernel_limits(int *sm_count, int *vec_blocks_per_sm, int *max_smem_optin)
{
    *sm_count = 148;
    *vec_blocks_per_sm = 4;
    *max_smem_optin = 232448;
    return cudaSuccess;
}

// The copy a launch stands for, slab by slab, on the host.
cudaError_t kvc_launch_copy(int dir, int, const KvcLaunch &a, uint32_t, uint32_t, cudaStream_t)
{
    const KvcGeom &g = a.g;
    for (uint32_t ent = 0; ent < a.n_ent; ++ent) {
        uint64_t slot_j, plane_step;
        int64_t id;
        if (a.table) {
            const KvcEnt &e = a.table[ent];
            slot_j = e.slot_addr;
            plane_step = e.plane_step;
            id = (e.nb_c & KVC_ENT_ID_IS_PTR) ? (int64_t) * reinterpret_cast<const int32_t *>((uintptr_t)e.id_or_ptr)
                                              : (int64_t)(int32_t)e.id_or_ptr;
        } else {
            slot_j = a.slot + (uint64_t)ent * a.ent_step;
            plane_step = a.plane_step;
            id = a.dev_ids ? a.dev_ids[ent] : a.ids[ent];
        }
        CHECK(id >= 0 && id < (int64_t)g.num_blocks);
        for (uint32_t lp = 0; lp < g.planes_total; ++lp) {
            const uint32_t l = lp / g.planes_per_layer, p = lp % g.planes_per_layer;
            const uint64_t plane = g.plane_table ? (uint64_t)(uintptr_t)g.plane_table[lp]
                                                 : (uint64_t)(uintptr_t)g.base + l * g.layer_stride + p * g.plane_stride;
            unsigned char *pool = reinterpret_cast<unsigned char *>((uintptr_t)(plane + (uint64_t)id * g.block_stride));
            unsigned char *slot = reinterpret_cast<unsigned char *>((uintptr_t)(slot_j + (uint64_t)lp * plane_step));
            if (dir == KVC_DIR_PACK)
                memcpy(slot, pool, g.slab_bytes);
            else
                memcpy(pool, slot, g.slab_bytes);
        }
    }
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
    uint32_t seed = 1744;
    for (int round = 0; round < 120; ++round) {
        const uint32_t e = 1u << (rnd(&seed) % 3), H = 1 + rnd(&seed) % 4, D = 16u << (rnd(&seed) % 3);
        const uint32_t B = 1 + rnd(&seed) % 8, L = 1 + rnd(&seed) % 4, P = 1 + rnd(&seed) % 2;
        const uint32_t NB = 4 + rnd(&seed) % 60, bpc = 1 + rnd(&seed) % 9;
        const int block_major = (int)(rnd(&seed) % 2);
        const uint64_t S = (uint64_t)B * H * D * e, LP = (uint64_t)L * P;
        if (S % 16)
            continue;
        std::vector<unsigned char> pool(LP * NB * S), pool0;
        for (unsigned char &b : pool)
            b = (unsigned char)rnd(&seed);
        pool0 = pool;
        kvc_layout_desc d;
        CHECK(kvc_layout_desc_init_dense(&d, pool.data(), L, P, NB, B, H, D, e, bpc * B, block_major) == KVC_OK);
        kvc_layout *lay = nullptr;
        CHECK(kvc_layout_create(&d, &lay) == KVC_OK);
        CHECK(kvc_layout_num_blocks(lay) == NB);
        // distinct source and destination ids (a random permutation each)
        const uint32_t n = 1 + rnd(&seed) % NB;
        std::vector<int32_t> perm(NB), src, dst;
        for (int pass = 0; pass < 2; ++pass) {
            for (uint32_t i = 0; i < NB; ++i)
                perm[i] = (int32_t)i;
            for (uint32_t i = NB - 1; i > 0; --i)
                std::swap(perm[i], perm[rnd(&seed) % (i + 1)]);
            (pass ? dst : src).assign(perm.begin(), perm.begin() + n);
        }
        const uint64_t total = kvc_layout_chunk_bytes(lay, n);
        const uint64_t slot_bytes = (kvc_layout_chunk_bytes(lay, bpc) + 4095) / 4096 * 4096;
        const uint32_t n_slots = 1 + rnd(&seed) % 4;
        const kvc_ring_kind kind = (kvc_ring_kind)(rnd(&seed) % 3);
        kvc_ring *ring = nullptr;
        CHECK(kvc_staging_ring_create(slot_bytes, n_slots, kind, nullptr, 0, &ring) == KVC_OK);
        // the expected host image: chunk after chunk, each in the layout's chunk byte order
        std::vector<unsigned char> want(total);
        uint64_t off = 0;
        for (uint32_t first = 0; first < n; first += bpc) {
            const uint32_t nb = n - first < bpc ? n - first : bpc;
            for (uint64_t lp = 0; lp < LP; ++lp)
                for (uint32_t j = 0; j < nb; ++j) {
                    const uint64_t at = block_major ? (j * LP + lp) * S : (lp * nb + j) * S;
                    memcpy(&want[off + at], &pool0[(lp * NB + (uint64_t)src[first + j]) * S], S);
                }
            off += LP * nb * S;
        }
        CHECK(off == total);
        unsigned char *host = static_cast<unsigned char *>(malloc(total));  // exactly the bytes the call may touch
        memset(host, 0xEE, total);
        kvc_host_transfer_stats st;
        const uint64_t l0 = g_launches;
        CHECK(kvc_offload_to_host(lay, ring, src.data(), n, host, total, nullptr, nullptr, 1000, &st) == KVC_OK);
        const uint32_t n_chunks = (n + bpc - 1) / bpc;
        CHECK(st.chunks == n_chunks && st.total_chunks == n_chunks && st.bytes == total);
        CHECK(g_launches == l0 + n_chunks);
        CHECK(memcmp(host, want.data(), total) == 0);
        CHECK(pool == pool0);
        // back into other blocks
        CHECK(kvc_load_from_host(lay, ring, host, total, dst.data(), n, nullptr, nullptr, 1000, &st) == KVC_OK);
        CHECK(st.chunks == n_chunks && st.bytes == total);
        // destination block dst[i] now holds what source block src[i] held; every other block is unchanged
        {
            std::vector<unsigned char> expect = pool0;
            for (uint64_t lp = 0; lp < LP; ++lp)
                for (uint32_t i = 0; i < n; ++i)
                    memcpy(&expect[(lp * NB + (uint64_t)dst[i]) * S], &pool0[(lp * NB + (uint64_t)src[i]) * S], S);
            CHECK(pool == expect);
        }
        uint32_t in_flight = 9;
        uint64_t acquires = 0;
        CHECK(kvc_staging_ring_stats(ring, &in_flight, &acquires, nullptr) == KVC_OK);
        CHECK(in_flight == 0 && acquires == 2 * n_chunks);
        // refusals take no slot and touch nothing
        std::vector<unsigned char> before = pool;
        std::vector<int32_t> bad = dst;
        bad[n - 1] = (int32_t)NB;
        CHECK(kvc_load_from_host(lay, ring, host, total, bad.data(), n, nullptr, nullptr, 1000, &st) == KVC_ERR_OUT_OF_RANGE);
        CHECK(kvc_offload_to_host(lay, ring, bad.data(), n, host, total, nullptr, nullptr, 1000, &st) == KVC_ERR_OUT_OF_RANGE);
        if (n > 1) {
            bad = dst;
            bad[n - 1] = bad[0];
            CHECK(kvc_load_from_host(lay, ring, host, total, bad.data(), n, nullptr, nullptr, 1000, &st) == KVC_ERR_CONFLICT);
            CHECK(kvc_offload_to_host(lay, ring, bad.data(), n, host, total, nullptr, nullptr, 1000, &st) == KVC_OK);  // pack may repeat
        }
        CHECK(kvc_offload_to_host(lay, ring, src.data(), n, host, total - 1, nullptr, nullptr, 1000, &st) == KVC_ERR_INVALID_ARG);
        CHECK(kvc_offload_to_host(lay, ring, src.data(), n, host, total, nullptr, nullptr, 0, &st) == KVC_ERR_INVALID_ARG);
        CHECK(pool == before);
        CHECK(kvc_staging_ring_stats(ring, &in_flight, nullptr, nullptr) == KVC_OK && in_flight == 0);
        free(host);
        CHECK(kvc_staging_ring_destroy(ring) == KVC_OK);
        CHECK(kvc_layout_destroy(lay) == KVC_OK);
    }
    CHECK(g_launches > 200);
    printf("ok\n");
    return 0;
}
