// Copy-engine variants of pack / unpack: the same byte movement expressed as strided asynchronous
// memory copies, so that the GPU's DMA engines do the work and no SM is used.  This is how the
// paper's own system moves blocks (Sec. 6.2, 6.4: a DMA-based batched block copy between the KV
// tensors and pinned staging slots; Sec. 5.1 contrasts it with kernel copies, which take SM time
// away from the model).  It exists here to put numbers on that trade-off next to the kernels.
//
// One 2-D copy moves one block: its L*P slabs are `plane pitch` apart in the pool and
// nb_c * S apart in the chunk, so pool -> chunk is a copy of L*P rows of S bytes.  When the planes
// are not equally spaced (separately allocated planes, or layer stride != planes * plane stride)
// the copy is split per layer or per plane.  The other side may be device memory or pinned host
// memory; in the second case the data crosses the host link directly and needs no staging slot.
#include "kvc_internal.h"

namespace {

kvc_status copy_engine(kvc_layout *lay, int dir, const int32_t *ids, uint32_t n_blocks, void *chunk,
                       uint64_t chunk_bytes, cudaStream_t st)
{
    if (!lay || (!ids && n_blocks) || (!chunk && n_blocks))
        return KVC_ERR_INVALID_ARG;
    if (n_blocks == 0)
        return KVC_OK;
    if (chunk_bytes < kvc_layout_chunk_bytes(lay, n_blocks))
        return KVC_ERR_INVALID_ARG;
    if (((uintptr_t)chunk & 15u) != 0)
        return KVC_ERR_ALIGNMENT;
    for (uint32_t j = 0; j < n_blocks; ++j)
        if (ids[j] < 0 || (uint32_t)ids[j] >= lay->d.num_blocks)
            return KVC_ERR_OUT_OF_RANGE;
    if (dir == KVC_DIR_UNPACK)
        for (uint32_t j = 0; j < n_blocks; ++j)
            for (uint32_t k = 0; k < j; ++k)
                if (ids[k] == ids[j])
                    return KVC_ERR_CONFLICT;

    const uint64_t S = lay->slab_bytes;
    uint64_t ent_step, chunk_pitch;  // chunk_pitch: distance of consecutive planes in the chunk
    kvc_chunk_steps(lay, n_blocks, &ent_step, &chunk_pitch);
    const uint32_t P = lay->d.kv_planes, L = lay->d.num_layers;
    const uint64_t max_pitch = 0x7FFFFFFFull;
    // rows per copy: all planes, the planes of one layer, or a single plane
    uint32_t rows, groups;
    uint64_t pool_pitch, group_stride;
    const bool dense = lay->plane_ptrs.empty();
    if (dense && lay->d.layer_stride == (uint64_t)P * lay->d.plane_stride &&
        lay->d.plane_stride <= max_pitch && chunk_pitch <= max_pitch) {
        rows = L * P, groups = 1, pool_pitch = lay->d.plane_stride, group_stride = 0;
    } else if (dense && lay->d.plane_stride <= max_pitch && chunk_pitch <= max_pitch) {
        rows = P, groups = L, pool_pitch = lay->d.plane_stride, group_stride = lay->d.layer_stride;
    } else {
        rows = 1, groups = L * P, pool_pitch = S, group_stride = 0;
    }
    unsigned char *cbase = static_cast<unsigned char *>(chunk);
    for (uint32_t j = 0; j < n_blocks; ++j) {
        for (uint32_t gi = 0; gi < groups; ++gi) {
            const uint32_t lp0 = gi * rows;  // first plane of this copy
            const unsigned char *pool_ptr;
            if (dense)
                pool_ptr = static_cast<const unsigned char *>(lay->d.base) +
                           (rows == 1 ? (uint64_t)(lp0 / P) * lay->d.layer_stride +
                                            (uint64_t)(lp0 % P) * lay->d.plane_stride
                                      : (uint64_t)gi * group_stride);
            else
                pool_ptr = static_cast<const unsigned char *>(lay->plane_ptrs[lp0]);
            pool_ptr += (uint64_t)ids[j] * lay->block_stride;
            unsigned char *chunk_ptr = cbase + (uint64_t)j * ent_step + (uint64_t)lp0 * chunk_pitch;
            cudaError_t e;
            if (dir == KVC_DIR_PACK)
                e = cudaMemcpy2DAsync(chunk_ptr, rows == 1 ? S : chunk_pitch, pool_ptr, pool_pitch, S,
                                      rows, cudaMemcpyDefault, st);
            else
                e = cudaMemcpy2DAsync(const_cast<unsigned char *>(pool_ptr), pool_pitch, chunk_ptr,
                                      rows == 1 ? S : chunk_pitch, S, rows, cudaMemcpyDefault, st);
            if (e != cudaSuccess) {
                (void)cudaGetLastError();
                return KVC_ERR_CUDA;
            }
        }
    }
    return KVC_OK;
}

}  // namespace

extern "C" {

kvc_status kvc_pack_copy_engine(kvc_layout *lay, const int32_t *ids, uint32_t n_blocks, void *dst,
                                uint64_t dst_bytes, void *stream)
{
    return copy_engine(lay, KVC_DIR_PACK, ids, n_blocks, dst, dst_bytes, (cudaStream_t)stream);
}

kvc_status kvc_unpack_copy_engine(kvc_layout *lay, const void *src, uint64_t src_bytes,
                                  const int32_t *ids, uint32_t n_blocks, void *stream)
{
    return copy_engine(lay, KVC_DIR_UNPACK, ids, n_blocks, const_cast<void *>(src), src_bytes,
                       (cudaStream_t)stream);
}

}  // extern "C"
