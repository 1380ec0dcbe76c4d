/* Plain C use of the library through its header: one pack and one unpack of a small request on
 * the current GPU, then the same request to a pinned host buffer and back through a two-slot ring
 * in chunks of four blocks, all checked against a straightforward host loop.  Exit code 0 on success. */
#include <cuda_runtime.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include "kvc.h"

#define CK(x)                                                                                  \
    do {                                                                                       \
        kvc_status s_ = (x);                                                                   \
        if (s_ != KVC_OK) {                                                                    \
            printf("line %d: %s\n", __LINE__, kvc_status_str(s_));                             \
            return 1;                                                                          \
        }                                                                                      \
    } while (0)

int main(void)
{
    const uint32_t L = 3, P = 2, NB = 40, B = 16, H = 4, D = 64, e = 2, n = 9;
    const size_t slab = (size_t)B * H * D * e, plane = slab * NB, pool_bytes = plane * L * P;
    unsigned char *h_pool = malloc(pool_bytes), *d_pool = NULL, *d_slot = NULL;
    for (size_t i = 0; i < pool_bytes; ++i)
        h_pool[i] = (unsigned char)(i * 2654435761u >> 13);
    if (cudaMalloc((void **)&d_pool, pool_bytes) != cudaSuccess) {
        printf("no CUDA device\n");
        return 2;
    }
    cudaMemcpy(d_pool, h_pool, pool_bytes, cudaMemcpyHostToDevice);
    kvc_layout_desc desc;
    CK(kvc_layout_desc_init_dense(&desc, d_pool, L, P, NB, B, H, D, e, 16 * 16, KVC_CHUNK_LAYER_MAJOR));
    if (desc.plane_stride != plane || desc.layer_stride != plane * P || desc.block_stride != slab) {
        printf("dense strides wrong\n");
        return 1;
    }
    kvc_layout *lay = NULL;
    CK(kvc_layout_create(&desc, &lay));
    int32_t ids[9] = {7, 39, 0, 12, 5, 21, 33, 2, 18}, dst[9] = {1, 3, 4, 6, 8, 9, 10, 11, 13};
    const uint64_t cb = kvc_layout_chunk_bytes(lay, n);
    cudaMalloc((void **)&d_slot, cb);
    CK(kvc_pack(lay, ids, n, 0, d_slot, cb, NULL));
    CK(kvc_unpack(lay, d_slot, cb, dst, n, 0, NULL));
    unsigned char *h_slot = malloc(cb), *h_after = malloc(pool_bytes);
    cudaMemcpy(h_slot, d_slot, cb, cudaMemcpyDeviceToHost);
    cudaMemcpy(h_after, d_pool, pool_bytes, cudaMemcpyDeviceToHost);
    int bad = 0;
    for (uint32_t lp = 0; lp < L * P; ++lp)
        for (uint32_t j = 0; j < n; ++j) {
            bad |= memcmp(h_slot + ((size_t)lp * n + j) * slab, h_pool + lp * plane + ids[j] * slab, slab);
            bad |= memcmp(h_after + lp * plane + dst[j] * slab, h_pool + lp * plane + ids[j] * slab, slab);
        }
    uint32_t skipped = 9, expired = 9;
    CK(kvc_poll_device_status(lay, NULL, &skipped, &expired));
    CK(kvc_layout_destroy(lay));

    /* request <-> host buffer: chunks of 4 blocks (4 + 4 + 1) through a ring of two slots */
    CK(kvc_layout_desc_init_dense(&desc, d_pool, L, P, NB, B, H, D, e, 4 * 16, KVC_CHUNK_LAYER_MAJOR));
    CK(kvc_layout_create(&desc, &lay));
    kvc_ring *ring = NULL;
    CK(kvc_staging_ring_create(kvc_layout_chunk_bytes(lay, 4), 2, KVC_RING_DEVICE, NULL, 0, &ring));
    unsigned char *h_req = NULL;
    if (cudaMallocHost((void **)&h_req, cb) != cudaSuccess)
        return 2;
    cudaMemcpy(d_pool, h_pool, pool_bytes, cudaMemcpyHostToDevice);
    kvc_host_transfer_stats ts;
    CK(kvc_offload_to_host(lay, ring, ids, n, h_req, cb, NULL, NULL, 1000000, &ts));
    cudaDeviceSynchronize();
    bad |= ts.chunks != 3 || ts.bytes != cb;
    size_t off = 0;
    for (uint32_t first = 0; first < n; first += 4) {
        const uint32_t nb = n - first < 4 ? n - first : 4;
        for (uint32_t lp = 0; lp < L * P; ++lp)
            for (uint32_t j = 0; j < nb; ++j)
                bad |= memcmp(h_req + off + ((size_t)lp * nb + j) * slab,
                              h_pool + lp * plane + ids[first + j] * slab, slab);
        off += (size_t)L * P * nb * slab;
    }
    CK(kvc_load_from_host(lay, ring, h_req, cb, dst, n, NULL, NULL, 1000000, &ts));
    cudaDeviceSynchronize();
    cudaMemcpy(h_after, d_pool, pool_bytes, cudaMemcpyDeviceToHost);
    for (uint32_t lp = 0; lp < L * P; ++lp)
        for (uint32_t j = 0; j < n; ++j)
            bad |= memcmp(h_after + lp * plane + dst[j] * slab, h_pool + lp * plane + ids[j] * slab, slab);
    CK(kvc_staging_ring_destroy(ring));
    CK(kvc_layout_destroy(lay));
    printf(bad || skipped || expired ? "MISMATCH\n" : "ok\n");
    return bad || skipped || expired;
}
