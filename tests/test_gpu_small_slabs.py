"""GPU parity for layouts with small slabs, where the bulk kernel moves several slabs per work
item: tensor-parallel shards of the KV heads, 1-byte elements, small block sizes.  The slot side
of such an item is one copy that may span many blocks (and cross into the next chunk), the pool
side one copy per slab, so the cases below vary the slab size, the slabs per item, the request
length against the chunk length (ragged last chunk, runs that straddle chunks), the chunk byte
order, the traversal order and the launch shape.  Everything is compared byte for byte with the
CPU oracle."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")

from oracle import oracle as orc
from paper_2609_11744_b200 import kvc
import workloads as wl
from test_gpu_parity import DEV, dense_layout, run_pack_unpack, to_dev

pytestmark = pytest.mark.gpu
BULK, VEC = kvc.KVC_VARIANT_BULK, kvc.KVC_VARIANT_VEC

# (L, P, NB, B, H, D, e): slab bytes = B*H*D*e
GEOMS = {
    "S64": (3, 2, 90, 4, 2, 8, 1),            # 64 B: 32 slabs per item, 2 KiB items
    "S48": (2, 1, 70, 1, 1, 24, 2),           # 48 B: not a power of two, one plane per layer
    "S256": (4, 2, 96, 16, 1, 8, 2),          # 256 B
    "S1K": (4, 2, 96, 16, 1, 32, 2),          # 1 KiB: 32 per item
    "S2K": (6, 2, 80, 16, 1, 128, 1),         # 2 KiB: one KV head, 1-byte elements
    "S4K": (5, 2, 72, 16, 1, 128, 2),         # 4 KiB: one KV head of an 8-head model (TP = 8)
    "S12K": (3, 2, 40, 16, 3, 128, 2),        # 12 KiB: two per item, 24 KiB items
    "S16K": (3, 2, 40, 16, 4, 128, 2),        # 16 KiB: two per item
}


def _case(name, n, chunk_blocks, **kw):
    g = orc.Dims(*GEOMS[name])
    pool = wl.random_bits(300 + g.L * 7 + g.H, g.pool_bytes)
    src = wl.block_ids(11, g.NB, n)
    dst = wl.block_ids(12, g.NB, n)
    return g, pool, src, dst, chunk_blocks * g.B


@pytest.mark.parametrize("variant", [BULK, VEC])
@pytest.mark.parametrize("name", sorted(GEOMS))
@pytest.mark.parametrize("mode", ["chunk", "chunk_dev", "batch", "batch_dev"])
def test_default_grouping_every_slab_size(name, mode, variant):
    # 37 blocks in chunks of 8: four full chunks and a ragged one of 5; planes * blocks per chunk
    # is not a multiple of the slabs per item, so items straddle planes and chunks
    g, pool, src, dst, ct = _case(name, 37, 8)
    run_pack_unpack(g, pool, src, dst, ct, variant, 0, mode)


@pytest.mark.parametrize("variant", [BULK, VEC])
@pytest.mark.parametrize("group", [2, 4, 8, 32, 1, kvc.KVC_GROUP_FORCE_KERNEL | 1])
@pytest.mark.parametrize("order", [kvc.KVC_ORDER_CHUNK_MAJOR, kvc.KVC_ORDER_PLANE_MAJOR,
                                   kvc.KVC_ORDER_BLOCK_MAJOR])
def test_slabs_per_item_and_traversal_orders(group, order, variant):
    g, pool, src, dst, ct = _case("S1K", 45, 16)
    for mode in ("chunk", "batch_dev"):
        run_pack_unpack(g, pool, src, dst, ct, variant, order, mode, group=group)


@pytest.mark.parametrize("tuning", [dict(max_ctas=2), dict(items_per_cta=1), dict(items_per_cta=9),
                                    dict(pdl=1), dict(group=2, max_ctas=5), dict(vec_threads=32),
                                    dict(vec_threads=96, max_ctas=7), dict(vec_threads=32, max_ctas=40)],
                         ids=lambda t: ",".join("%s=%s" % kv for kv in t.items()))
def test_vector_kernel_launch_shapes_with_grouped_items(tuning):
    for name, n, cb in (("S64", 71, 16), ("S2K", 61, 16), ("S4K", 35, 4), ("S48", 50, 8)):
        g, pool, src, dst, ct = _case(name, n, cb)
        run_pack_unpack(g, pool, src, dst, ct, VEC, 0, "batch", **tuning)


@pytest.mark.parametrize("tuning", [
    dict(max_ctas=3), dict(max_ctas=148, stages=4, lag=2), dict(stages=2), dict(stages=16, lag=14),
    dict(stages=8, lag=1), dict(items_per_cta=1), dict(items_per_cta=7, stages=3),
    dict(tile_bytes=8192), dict(tile_bytes=4096, stages=5, lag=3), dict(pdl=1), dict(l2_hint=2),
], ids=lambda t: ",".join("%s=%s" % kv for kv in t.items()))
def test_launch_shapes_with_grouped_items(tuning):
    tuning = dict(tuning)
    tile = tuning.pop("tile_bytes", 0)
    g, pool, src, dst, ct = _case("S2K", 61, 16)
    run_pack_unpack(g, pool, src, dst, ct, BULK, 0, "batch", tile, **tuning)
    g, pool, src, dst, ct = _case("S256", 33, 4)
    run_pack_unpack(g, pool, src, dst, ct, BULK, 0, "chunk", tile, **tuning)


def test_multi_slab_kernel_with_one_slab_per_item_on_8b_shape():
    """The 8B KV shape (32 KiB slabs) through the multi-slab kernel: one slab per item."""
    s = wl.LLAMA_8B
    g = orc.Dims(4, s.P, 96, s.B, s.H, s.D, s.e)
    pool = wl.random_bits(411, g.pool_bytes)
    src, dst = wl.block_ids(13, g.NB, 41), wl.block_ids(14, g.NB, 41)
    for mode in ("chunk", "batch"):
        run_pack_unpack(g, pool, src, dst, 256, BULK, 0, mode, group=kvc.KVC_GROUP_FORCE_KERNEL)


@pytest.mark.parametrize("variant", [BULK, VEC])
@pytest.mark.parametrize("name", ["S64", "S1K", "S4K", "S12K"])
def test_block_major_chunks_with_grouped_items(name, variant):
    """Chunk byte order [n][L][P]..: consecutive slabs of the slot are the planes of ONE block."""
    g = orc.Dims(*GEOMS[name])
    pool = wl.random_bits(500 + g.H, g.pool_bytes)
    planes = orc.dense_planes(g, pool)
    pool_t = to_dev(pool)
    lay = kvc.kvc_layout_create_dense(pool_t, g.L, g.P, g.NB, g.B, g.H, g.D, g.e, 8 * g.B,
                                      chunk_order=kvc.KVC_CHUNK_BLOCK_MAJOR)
    kvc.kvc_layout_set_tuning(lay, variant=variant)
    n = 29
    src, dst = wl.block_ids(15, g.NB, n), wl.block_ids(16, g.NB, n)
    staging = torch.full((n * g.bytes_per_block + 4096,), 0x5A, dtype=torch.uint8, device=DEV)
    ops, keep, nbytes, dev = kvc.request_chunk_ops(lay, src, staging)
    kvc.kvc_pack_batch(lay, ops, dev)
    torch.cuda.synchronize()
    host = staging.cpu().numpy()
    want, off = [], 0
    for f, nb in orc.chunk_ranges(n, 8):
        c = orc.pack_chunk_planes_block_major(g, planes, src[f:f + nb], g.slab_bytes)
        assert np.array_equal(host[off:off + c.size], c), "chunk at block %d" % f
        want.append(c)
        off += c.size
    assert (host[off:] == 0x5A).all()
    ops2, keep2, _, _ = kvc.request_chunk_ops(lay, dst, staging)
    kvc.kvc_unpack_batch(lay, ops2, dev)
    torch.cuda.synchronize()
    want_pool = pool.copy()
    want_planes = orc.dense_planes(g, want_pool)
    for c, (f, nb) in zip(want, orc.chunk_ranges(n, 8)):
        orc.unpack_chunk_planes_block_major(g, want_planes, c, dst[f:f + nb], g.slab_bytes)
    assert np.array_equal(pool_t.cpu().numpy(), want_pool)
    assert kvc.kvc_poll_device_status(lay) == (0, 0)


@pytest.mark.parametrize("variant", [BULK, VEC])
def test_bad_device_ids_inside_grouped_items(variant):
    """A bad id in the middle of an item: its slabs are skipped, the slot-side copy is split
    around the hole, and nothing else is disturbed."""
    g = orc.Dims(*GEOMS["S1K"])
    pool = wl.random_bits(77, g.pool_bytes)
    pool_t = to_dev(pool)
    lay = dense_layout(pool_t, g, 16 * g.B)
    kvc.kvc_layout_set_tuning(lay, variant=variant)
    ids = np.array([3, 95, 96, 7, -1, 9, 1 << 30, 0, 31, 2, 5, -7, 11], dtype=np.int32)
    good = (ids >= 0) & (ids < g.NB)
    n_bad = int((~good).sum())
    cb = kvc.kvc_layout_chunk_bytes(lay, len(ids))
    staging = torch.full((cb,), 0x11, dtype=torch.uint8, device=DEV)
    kvc.kvc_pack(lay, to_dev(ids), staging)
    assert kvc.kvc_poll_device_status(lay) == (n_bad, 0)
    got = staging.cpu().numpy().reshape(g.L * g.P, len(ids), g.slab_bytes)
    safe = np.where(good, ids, 0).astype(np.int32)
    want = orc.pack_chunk(g, pool, safe).reshape(g.L * g.P, len(ids), g.slab_bytes)
    assert np.array_equal(got[:, good], want[:, good])
    assert (got[:, ~good] == 0x11).all()
    chunk = wl.random_bits(78, cb)
    kvc.kvc_unpack(lay, to_dev(chunk), to_dev(ids))
    assert kvc.kvc_poll_device_status(lay) == (n_bad, 0)
    want_pool = pool.copy()
    c3 = chunk.reshape(g.L * g.P, len(ids), g.slab_bytes)
    p3 = want_pool.reshape(g.L * g.P, g.NB, g.slab_bytes)
    for j in np.flatnonzero(good):
        p3[:, ids[j]] = c3[:, j]
    assert np.array_equal(pool_t.cpu().numpy(), want_pool)


@pytest.mark.parametrize("variant", [BULK, VEC])
def test_many_requests_in_one_launch_small_slabs(variant):
    """Chunks of many requests, of different lengths, in one launch: items cross from one
    request's slot into the next one's, which lies somewhere else."""
    g = orc.Dims(*GEOMS["S2K"])
    pool = wl.random_bits(91, g.pool_bytes)
    pool_t = to_dev(pool)
    lay = dense_layout(pool_t, g, 4 * g.B)
    kvc.kvc_layout_set_tuning(lay, variant=variant)
    rng = np.random.default_rng(5)
    perm = rng.permutation(g.NB).astype(np.int32)
    lens = [1, 4, 3, 7, 2, 9, 5]
    tables, cur = [], 0
    for n in lens:
        tables.append(np.ascontiguousarray(perm[cur:cur + n]))
        cur += n
    slots, ids_addr, nbs, want = [], [], [], []
    bufs = []
    for t in tables:
        for f, nb in orc.chunk_ranges(len(t), 4):
            buf = torch.full((nb * g.bytes_per_block + 256,), 0x77, dtype=torch.uint8, device=DEV)
            bufs.append(buf)
            slots.append(buf.data_ptr())
            ids_addr.append(t.ctypes.data + 4 * f)
            nbs.append(nb)
            want.append(orc.pack_chunk(g, pool, t[f:f + nb]))
    ops = kvc.make_chunk_ops(slots, ids_addr, nbs)
    kvc.kvc_pack_batch(lay, ops, 0)
    torch.cuda.synchronize()
    for buf, w in zip(bufs, want):
        h = buf.cpu().numpy()
        assert np.array_equal(h[:w.size], w)
        assert (h[w.size:] == 0x77).all()
    # scatter the same chunks into other blocks
    dst_perm = rng.permutation(g.NB).astype(np.int32)
    want_pool = pool.copy()
    ids2, cur = [], 0
    for nb, w in zip(nbs, want):
        d = np.ascontiguousarray(dst_perm[cur:cur + nb])
        cur += nb
        ids2.append(d)
        orc.unpack_chunk(g, want_pool, w, d)
    ops2 = kvc.make_chunk_ops(slots, [d.ctypes.data for d in ids2], nbs)
    kvc.kvc_unpack_batch(lay, ops2, 0)
    torch.cuda.synchronize()
    assert np.array_equal(pool_t.cpu().numpy(), want_pool)
    assert kvc.kvc_poll_device_status(lay) == (0, 0)
