/*
 * TEST INFRASTRUCTURE -- not part of the product.
 *
 * Plain, slow, single-purpose CPU statement of what "pack" and "unpack" of a
 * paged KV cache compute.  Only tests, the smoke check and the CPU-baseline
 * leg of the benchmark may build, load or call this file; the CUDA library
 * shares no code with it.
 *
 * What is computed (paper Sec. 2.1: a KV cache is kept as fixed-size token
 * blocks, bytes/token = layers x 2 x KV heads x head dim x element size;
 * Sec. 6.4: a storage block ("chunk") groups several GPU blocks of one
 * request, in request order, and is moved through one staging slot):
 *
 *   paged pool     [L][P][NB][B][H][D]      element index pool_elem(l,p,b,t,h,d)
 *   chunk of nb_c  [L][P][nb_c][B][H][D]    element index chunk_elem(l,p,j,t,h,d)
 *
 *   pack  : chunk[chunk_elem(l,p,j,t,h,d)]        = pool[pool_elem(l,p,ids[j],t,h,d)]
 *   unpack: pool[pool_elem(l,p,ids[j],t,h,d)]     = chunk[chunk_elem(l,p,j,t,h,d)]
 *
 * for every l<L, p<P, j<nb_c, t<B, h<H, d<D.  Elements are opaque e-byte
 * values; they are moved byte by byte and never interpreted.
 *
 * Everything is written as six nested loops over element coordinates, with
 * the index formulas spelt out, so the code can be checked against the
 * definition by eye.  There is no blocking, no slab-sized memcpy and no
 * reordering.  The [lp_begin, lp_end) argument restricts the two outermost
 * loops (flattened l*P+p) so that a caller can hand disjoint (layer, plane)
 * ranges to several threads; it changes nothing about what is computed.
 */
#include <stddef.h>
#include <stdint.h>

typedef struct {
    uint32_t L;  /* layers */
    uint32_t P;  /* planes per layer (K and V -> 2) */
    uint32_t NB; /* blocks in the pool */
    uint32_t B;  /* tokens per block */
    uint32_t H;  /* kv heads */
    uint32_t D;  /* head dim */
    uint32_t e;  /* bytes per element */
} kvc_oracle_dims;

/* Element index in the dense paged pool [L][P][NB][B][H][D]. */
uint64_t kvc_oracle_pool_elem(const kvc_oracle_dims *g, uint64_t l, uint64_t p,
                              uint64_t b, uint64_t t, uint64_t h, uint64_t d)
{
    return ((((l * g->P + p) * g->NB + b) * g->B + t) * g->H + h) * g->D + d;
}

/* Element index inside one plane [NB][B][H][D] whose blocks are
 * block_stride_elems apart (>= B*H*D; larger when blocks are padded). */
static uint64_t plane_elem(const kvc_oracle_dims *g, uint64_t block_stride_elems,
                           uint64_t b, uint64_t t, uint64_t h, uint64_t d)
{
    return b * block_stride_elems + (t * g->H + h) * g->D + d;
}

/* Element index in a chunk of nb_c blocks, [L][P][nb_c][B][H][D]. */
uint64_t kvc_oracle_chunk_elem(const kvc_oracle_dims *g, uint64_t nb_c, uint64_t l,
                               uint64_t p, uint64_t j, uint64_t t, uint64_t h,
                               uint64_t d)
{
    return ((((l * g->P + p) * nb_c + j) * g->B + t) * g->H + h) * g->D + d;
}

/* Element index in a block-major chunk of nb_c blocks, [nb_c][L][P][B][H][D]: every block's
 * data for all layers is one contiguous run (an alternative file layout; the paper does not fix
 * the byte order inside a storage block). */
uint64_t kvc_oracle_chunk_elem_block_major(const kvc_oracle_dims *g, uint64_t nb_c, uint64_t l,
                                           uint64_t p, uint64_t j, uint64_t t, uint64_t h,
                                           uint64_t d)
{
    (void)nb_c;
    return ((((j * g->L + l) * g->P + p) * g->B + t) * g->H + h) * g->D + d;
}

static int ids_in_range(const kvc_oracle_dims *g, const int32_t *ids, uint32_t nb_c)
{
    for (uint32_t j = 0; j < nb_c; ++j)
        if (ids[j] < 0 || (uint32_t)ids[j] >= g->NB)
            return 0;
    return 1;
}

/* pack, dense monolithic pool.  Returns 0, or -1 if an id is out of range. */
int kvc_oracle_pack_chunk_mono(const kvc_oracle_dims *g, const uint8_t *pool,
                               const int32_t *ids, uint32_t nb_c, uint8_t *chunk,
                               uint32_t lp_begin, uint32_t lp_end)
{
    if (!ids_in_range(g, ids, nb_c))
        return -1;
    for (uint32_t lp = lp_begin; lp < lp_end; ++lp) {
        uint32_t l = lp / g->P, p = lp % g->P;
        for (uint32_t j = 0; j < nb_c; ++j)
            for (uint32_t t = 0; t < g->B; ++t)
                for (uint32_t h = 0; h < g->H; ++h)
                    for (uint32_t d = 0; d < g->D; ++d) {
                        uint64_t src = kvc_oracle_pool_elem(g, l, p, (uint64_t)ids[j], t, h, d);
                        uint64_t dst = kvc_oracle_chunk_elem(g, nb_c, l, p, j, t, h, d);
                        for (uint32_t k = 0; k < g->e; ++k)
                            chunk[dst * g->e + k] = pool[src * g->e + k];
                    }
    }
    return 0;
}

/* unpack, dense monolithic pool. */
int kvc_oracle_unpack_chunk_mono(const kvc_oracle_dims *g, uint8_t *pool,
                                 const int32_t *ids, uint32_t nb_c, const uint8_t *chunk,
                                 uint32_t lp_begin, uint32_t lp_end)
{
    if (!ids_in_range(g, ids, nb_c))
        return -1;
    for (uint32_t lp = lp_begin; lp < lp_end; ++lp) {
        uint32_t l = lp / g->P, p = lp % g->P;
        for (uint32_t j = 0; j < nb_c; ++j)
            for (uint32_t t = 0; t < g->B; ++t)
                for (uint32_t h = 0; h < g->H; ++h)
                    for (uint32_t d = 0; d < g->D; ++d) {
                        uint64_t dst = kvc_oracle_pool_elem(g, l, p, (uint64_t)ids[j], t, h, d);
                        uint64_t src = kvc_oracle_chunk_elem(g, nb_c, l, p, j, t, h, d);
                        for (uint32_t k = 0; k < g->e; ++k)
                            pool[dst * g->e + k] = chunk[src * g->e + k];
                    }
    }
    return 0;
}

/* pack, one separately allocated plane per (layer, K|V): planes[l*P+p] points
 * at a [NB][B][H][D] array whose blocks are block_stride_elems apart. */
int kvc_oracle_pack_chunk_planes(const kvc_oracle_dims *g, const uint8_t *const *planes,
                                 uint64_t block_stride_elems, const int32_t *ids,
                                 uint32_t nb_c, uint8_t *chunk, uint32_t lp_begin,
                                 uint32_t lp_end)
{
    if (!ids_in_range(g, ids, nb_c))
        return -1;
    for (uint32_t lp = lp_begin; lp < lp_end; ++lp) {
        uint32_t l = lp / g->P, p = lp % g->P;
        const uint8_t *plane = planes[l * g->P + p];
        for (uint32_t j = 0; j < nb_c; ++j)
            for (uint32_t t = 0; t < g->B; ++t)
                for (uint32_t h = 0; h < g->H; ++h)
                    for (uint32_t d = 0; d < g->D; ++d) {
                        uint64_t src = plane_elem(g, block_stride_elems, (uint64_t)ids[j], t, h, d);
                        uint64_t dst = kvc_oracle_chunk_elem(g, nb_c, l, p, j, t, h, d);
                        for (uint32_t k = 0; k < g->e; ++k)
                            chunk[dst * g->e + k] = plane[src * g->e + k];
                    }
    }
    return 0;
}

/* unpack, separately allocated planes. */
int kvc_oracle_unpack_chunk_planes(const kvc_oracle_dims *g, uint8_t *const *planes,
                                   uint64_t block_stride_elems, const int32_t *ids,
                                   uint32_t nb_c, const uint8_t *chunk, uint32_t lp_begin,
                                   uint32_t lp_end)
{
    if (!ids_in_range(g, ids, nb_c))
        return -1;
    for (uint32_t lp = lp_begin; lp < lp_end; ++lp) {
        uint32_t l = lp / g->P, p = lp % g->P;
        uint8_t *plane = planes[l * g->P + p];
        for (uint32_t j = 0; j < nb_c; ++j)
            for (uint32_t t = 0; t < g->B; ++t)
                for (uint32_t h = 0; h < g->H; ++h)
                    for (uint32_t d = 0; d < g->D; ++d) {
                        uint64_t dst = plane_elem(g, block_stride_elems, (uint64_t)ids[j], t, h, d);
                        uint64_t src = kvc_oracle_chunk_elem(g, nb_c, l, p, j, t, h, d);
                        for (uint32_t k = 0; k < g->e; ++k)
                            plane[dst * g->e + k] = chunk[src * g->e + k];
                    }
    }
    return 0;
}

/* pack / unpack with the block-major chunk order, separately allocated (or strided) planes. */
int kvc_oracle_pack_chunk_planes_block_major(const kvc_oracle_dims *g, const uint8_t *const *planes,
                                             uint64_t block_stride_elems, const int32_t *ids,
                                             uint32_t nb_c, uint8_t *chunk)
{
    if (!ids_in_range(g, ids, nb_c))
        return -1;
    for (uint32_t j = 0; j < nb_c; ++j)
        for (uint32_t l = 0; l < g->L; ++l)
            for (uint32_t p = 0; p < g->P; ++p) {
                const uint8_t *plane = planes[l * g->P + p];
                for (uint32_t t = 0; t < g->B; ++t)
                    for (uint32_t h = 0; h < g->H; ++h)
                        for (uint32_t d = 0; d < g->D; ++d) {
                            uint64_t src = plane_elem(g, block_stride_elems, (uint64_t)ids[j], t, h, d);
                            uint64_t dst = kvc_oracle_chunk_elem_block_major(g, nb_c, l, p, j, t, h, d);
                            for (uint32_t k = 0; k < g->e; ++k)
                                chunk[dst * g->e + k] = plane[src * g->e + k];
                        }
            }
    return 0;
}

int kvc_oracle_unpack_chunk_planes_block_major(const kvc_oracle_dims *g, uint8_t *const *planes,
                                               uint64_t block_stride_elems, const int32_t *ids,
                                               uint32_t nb_c, const uint8_t *chunk)
{
    if (!ids_in_range(g, ids, nb_c))
        return -1;
    for (uint32_t j = 0; j < nb_c; ++j)
        for (uint32_t l = 0; l < g->L; ++l)
            for (uint32_t p = 0; p < g->P; ++p) {
                uint8_t *plane = planes[l * g->P + p];
                for (uint32_t t = 0; t < g->B; ++t)
                    for (uint32_t h = 0; h < g->H; ++h)
                        for (uint32_t d = 0; d < g->D; ++d) {
                            uint64_t dst = plane_elem(g, block_stride_elems, (uint64_t)ids[j], t, h, d);
                            uint64_t src = kvc_oracle_chunk_elem_block_major(g, nb_c, l, p, j, t, h, d);
                            for (uint32_t k = 0; k < g->e; ++k)
                                plane[dst * g->e + k] = chunk[src * g->e + k];
                        }
            }
    return 0;
}
