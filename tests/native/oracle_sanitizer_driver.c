/* Drives the C oracle over small layouts under AddressSanitizer / UBSan: every buffer is
 * allocated at its exact size, so any access outside the pool, the planes or the chunk aborts. */
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

typedef struct { uint32_t L, P, NB, B, H, D, e; } kvc_oracle_dims;
int kvc_oracle_pack_chunk_mono(const kvc_oracle_dims *, const uint8_t *, const int32_t *, uint32_t,
                               uint8_t *, uint32_t, uint32_t);
int kvc_oracle_unpack_chunk_mono(const kvc_oracle_dims *, uint8_t *, const int32_t *, uint32_t,
                                 const uint8_t *, uint32_t, uint32_t);
int kvc_oracle_pack_chunk_planes(const kvc_oracle_dims *, const uint8_t *const *, uint64_t,
                                 const int32_t *, uint32_t, uint8_t *, uint32_t, uint32_t);
int kvc_oracle_unpack_chunk_planes(const kvc_oracle_dims *, uint8_t *const *, uint64_t, const int32_t *,
                                   uint32_t, const uint8_t *, uint32_t, uint32_t);
int kvc_oracle_pack_chunk_planes_block_major(const kvc_oracle_dims *, const uint8_t *const *, uint64_t,
                                             const int32_t *, uint32_t, uint8_t *);
int kvc_oracle_unpack_chunk_planes_block_major(const kvc_oracle_dims *, uint8_t *const *, uint64_t,
                                               const int32_t *, uint32_t, const uint8_t *);

static int run(kvc_oracle_dims g, uint32_t n, uint64_t pad_elems)
{
    const uint64_t slab = (uint64_t)g.B * g.H * g.D * g.e;
    const uint64_t pool_bytes = (uint64_t)g.L * g.P * g.NB * slab;
    const uint64_t chunk_bytes = (uint64_t)g.L * g.P * n * slab;
    uint8_t *pool = malloc(pool_bytes), *chunk = malloc(chunk_bytes), *back = malloc(pool_bytes);
    int32_t *ids = malloc(n * sizeof(int32_t));
    for (uint64_t i = 0; i < pool_bytes; ++i)
        pool[i] = (uint8_t)(i * 131 + 7);
    for (uint32_t j = 0; j < n; ++j)
        ids[j] = (int32_t)((j * 5 + g.NB - 1) % g.NB);   /* includes the last block */
    memset(back, 0, pool_bytes);
    int rc = kvc_oracle_pack_chunk_mono(&g, pool, ids, n, chunk, 0, g.L * g.P);
    rc |= kvc_oracle_unpack_chunk_mono(&g, back, ids, n, chunk, 0, g.L * g.P);
    /* separately allocated planes with padded blocks: the last block ends exactly at the buffer end */
    const uint64_t stride_elems = (uint64_t)g.B * g.H * g.D + pad_elems;
    const uint64_t plane_bytes = ((uint64_t)(g.NB - 1) * stride_elems + (uint64_t)g.B * g.H * g.D) * g.e;
    uint8_t **planes = malloc(sizeof(uint8_t *) * g.L * g.P);
    for (uint32_t i = 0; i < g.L * g.P; ++i) {
        planes[i] = malloc(plane_bytes);
        memset(planes[i], (int)i, plane_bytes);
    }
    rc |= kvc_oracle_pack_chunk_planes(&g, (const uint8_t *const *)planes, stride_elems, ids, n, chunk, 0,
                                       g.L * g.P);
    rc |= kvc_oracle_unpack_chunk_planes(&g, planes, stride_elems, ids, n, chunk, 0, g.L * g.P);
    rc |= kvc_oracle_pack_chunk_planes_block_major(&g, (const uint8_t *const *)planes, stride_elems, ids,
                                                   n, chunk);
    rc |= kvc_oracle_unpack_chunk_planes_block_major(&g, planes, stride_elems, ids, n, chunk);
    int32_t bad = (int32_t)g.NB;   /* out of range: must be refused before any access */
    if (kvc_oracle_pack_chunk_mono(&g, pool, &bad, 1, chunk, 0, g.L * g.P) != -1)
        rc |= 2;
    for (uint32_t i = 0; i < g.L * g.P; ++i)
        free(planes[i]);
    free(planes);
    free(pool);
    free(chunk);
    free(back);
    free(ids);
    return rc;
}

int main(void)
{
    kvc_oracle_dims a = {2, 2, 7, 3, 2, 5, 2}, b = {1, 1, 3, 1, 1, 16, 1}, c = {3, 2, 9, 4, 3, 8, 4};
    int rc = run(a, 5, 0) | run(a, 7, 11) | run(b, 3, 0) | run(c, 1, 3) | run(c, 9, 0);
    printf(rc ? "FAILED %d\n" : "ok\n", rc);
    return rc;
}
