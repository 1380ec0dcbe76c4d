"""GPU parity: the CUDA path, called through the C-ABI binding, against the CPU oracle on the
same seeded inputs, byte for byte.  Pure byte movement, so the bar is bit-exact equality."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")

from oracle import oracle as orc
from paper_2609_11744_b200 import cuda_rt, kvc
import workloads as wl

pytestmark = pytest.mark.gpu

DEV = "cuda:0"
VARIANTS = [kvc.KVC_VARIANT_VEC, kvc.KVC_VARIANT_BULK]


def dims_of(shape: wl.KVShape, NB: int) -> orc.Dims:
    return orc.Dims(shape.L, shape.P, NB, shape.B, shape.H, shape.D, shape.e)


def dense_layout(pool_t, g: orc.Dims, chunk_tokens: int):
    return kvc.kvc_layout_create_dense(pool_t, g.L, g.P, g.NB, g.B, g.H, g.D, g.e, chunk_tokens)


def to_dev(a: np.ndarray):
    return torch.from_numpy(a).to(DEV)


def staged_chunks(staging_t, sizes):
    host = staging_t.cpu().numpy()
    out, off = [], 0
    for s in sizes:
        out.append(host[off:off + s])
        off += s
    return out, host[off:]


_ORACLE_CACHE = {}


def _oracle_results(g, pool_np, src_ids, dst_ids, chunk_tokens):
    """Oracle chunks of pack(src) and the pool after unpacking them into dst (cached: the
    oracle is slow and many launch configurations share the same expected bytes)."""
    key = (g, id(pool_np), src_ids.tobytes(), dst_ids.tobytes(), chunk_tokens)
    if key not in _ORACLE_CACHE:
        chunks = orc.pack_request(g, pool_np, src_ids, chunk_tokens)
        pool2 = pool_np.copy()
        orc.unpack_request(g, pool2, chunks, dst_ids, chunk_tokens)
        if len(_ORACLE_CACHE) > 4:
            _ORACLE_CACHE.clear()
        _ORACLE_CACHE[key] = (chunks, pool2, pool_np)
    return _ORACLE_CACHE[key][:2]


def run_pack_unpack(g, pool_np, src_ids, dst_ids, chunk_tokens, variant, order, mode, tile=0,
                    layout_factory=None, pool_dev=None, **tuning):
    """Pack src_ids into a staging area, unpack into dst_ids of the same pool, and compare both
    results with the oracle.  mode: 'chunk' (one call per chunk, host ids), 'chunk_dev'
    (device ids), 'batch' / 'batch_dev' (one launch)."""
    pool_t = to_dev(pool_np) if pool_dev is None else pool_dev
    lay = (layout_factory or dense_layout)(pool_t, g, chunk_tokens)
    kvc.kvc_layout_set_tuning(lay, variant=variant, order=order, tile_bytes=tile, **tuning)
    descs = kvc.kvc_map_request(lay, len(src_ids))
    sizes = [d[4] for d in descs]
    total = sum(sizes)
    guard = 4096
    staging = torch.full((total + guard,), 0xAB, dtype=torch.uint8, device=DEV)
    want_chunks, want_pool = _oracle_results(g, pool_np, src_ids, dst_ids, chunk_tokens)

    def go(direction, ids_np):
        ids_dev = to_dev(ids_np) if mode.endswith("_dev") else None
        if mode.startswith("batch"):
            ops, keep, nbytes, dev = kvc.request_chunk_ops(
                lay, ids_dev if ids_dev is not None else ids_np, staging)
            assert nbytes == total
            (kvc.kvc_pack_batch if direction == "pack" else kvc.kvc_unpack_batch)(lay, ops, dev)
        else:
            off = 0
            for (_, _, first, nb, nbytes) in descs:
                ids_c = (ids_dev if ids_dev is not None else ids_np)[first:first + nb]
                if ids_dev is not None:
                    ids_c = ids_c.contiguous()
                slot = staging[off:off + nbytes]
                if direction == "pack":
                    kvc.kvc_pack(lay, ids_c, slot)
                else:
                    kvc.kvc_unpack(lay, slot, ids_c)
                off += nbytes
        torch.cuda.synchronize()

    go("pack", src_ids)
    got_chunks, tail = staged_chunks(staging, sizes)
    for c, (a, b) in enumerate(zip(got_chunks, want_chunks)):
        assert np.array_equal(a, b), "pack chunk %d differs" % c
    assert (tail == 0xAB).all(), "bytes past the last chunk were written"

    go("unpack", dst_ids)
    got_pool = pool_t.cpu().numpy().reshape(-1)
    assert np.array_equal(got_pool, want_pool), "pool after unpack differs"
    assert kvc.kvc_poll_device_status(lay) == (0, 0)
    kvc.kvc_layout_destroy(lay)


# ------------------------------------------------------------------ config 1: tiny, K/V separate buffers
@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("mode", ["chunk", "chunk_dev", "batch", "batch_dev"])
def test_tiny_separate_planes(variant, mode):
    w = wl.WORKLOADS["tiny"]
    g = dims_of(w.shape, w.pool_blocks)
    plane_bytes = g.NB * g.slab_bytes
    planes_np = [wl.random_bits(w.seed + 10 + i, plane_bytes) for i in range(g.L * g.P)]
    src = wl.block_ids(w.seed, g.NB, w.request_blocks)
    dst = wl.block_ids(w.dst_seed, g.NB, w.request_blocks)
    assert not np.array_equal(src, dst)
    planes_t = [to_dev(p) for p in planes_np]
    lay = kvc.kvc_layout_create(g.L, g.P, g.NB, g.B, g.H, g.D, g.e, 256, plane_ptrs=planes_t)
    kvc.kvc_layout_set_tuning(lay, variant=variant)
    assert kvc.kvc_layout_num_chunks(lay, len(src)) == 4
    cb = kvc.kvc_layout_chunk_bytes(lay, 16)
    assert cb == 512 * 1024
    staging = torch.full((4 * cb + 4096,), 0x5C, dtype=torch.uint8, device=DEV)
    ids_s = to_dev(src) if mode.endswith("dev") else src
    ids_d = to_dev(dst) if mode.endswith("dev") else dst
    if mode.startswith("batch"):
        ops, keep, nbytes, dev = kvc.request_chunk_ops(lay, ids_s, staging)
        kvc.kvc_pack_batch(lay, ops, dev)
    else:
        for c in range(4):
            kvc.kvc_pack(lay, ids_s[c * 16:(c + 1) * 16], staging[c * cb:(c + 1) * cb])
    torch.cuda.synchronize()
    host = staging.cpu().numpy()
    for c in range(4):
        want = orc.pack_chunk_planes(g, planes_np, src[c * 16:(c + 1) * 16])
        assert np.array_equal(host[c * cb:(c + 1) * cb], want)
    assert (host[4 * cb:] == 0x5C).all()
    # the separate-plane chunk equals the chunk of the same data laid out as one dense pool
    mono = np.concatenate(planes_np)
    assert np.array_equal(host[:cb], orc.pack_chunk(g, mono, src[:16]))
    if mode.startswith("batch"):
        ops, keep, nbytes, dev = kvc.request_chunk_ops(lay, ids_d, staging)
        kvc.kvc_unpack_batch(lay, ops, dev)
    else:
        for c in range(4):
            kvc.kvc_unpack(lay, staging[c * cb:(c + 1) * cb], ids_d[c * 16:(c + 1) * 16])
    torch.cuda.synchronize()
    want_planes = [p.copy() for p in planes_np]
    for c in range(4):
        orc.unpack_chunk_planes(g, want_planes, host[c * cb:(c + 1) * cb], dst[c * 16:(c + 1) * 16])
    for t, wnt in zip(planes_t, want_planes):
        assert np.array_equal(t.cpu().numpy(), wnt)
    assert kvc.kvc_poll_device_status(lay) == (0, 0)


# ------------------------------------------------------------------ 8B shape, several tiles + ragged tail
@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("order", [kvc.KVC_ORDER_PLANE_MAJOR, kvc.KVC_ORDER_BLOCK_MAJOR,
                                   kvc.KVC_ORDER_CHUNK_MAJOR])
@pytest.mark.parametrize("mode,chunk_tokens", [("chunk", 256), ("batch", 256), ("batch", 16),
                                               ("batch_dev", 2048), ("chunk", 2048)])
def test_8b_shape_reduced_pool(variant, order, mode, chunk_tokens):
    """Llama-3.1-8B KV shape with a 384-block pool (768 MiB); 136-block request: 8 full
    256-token chunks and a short one of 8 blocks; one full 2048-token chunk plus the same tail."""
    w = wl.WORKLOADS["8b_8k"]
    g = dims_of(w.shape, 384)
    pool = _pool_8b_384()
    src = wl.block_ids(w.seed, g.NB, 136)
    dst = wl.block_ids(w.dst_seed, g.NB, 136)
    run_pack_unpack(g, pool, src, dst, chunk_tokens, variant, order, mode)


_POOL_CACHE = {}


def _pool_8b_384():
    if "p" not in _POOL_CACHE:
        w = wl.WORKLOADS["8b_8k"]
        _POOL_CACHE["p"] = wl.random_bits(w.seed + 1, dims_of(w.shape, 384).pool_bytes)
    return _POOL_CACHE["p"]


def test_single_call_with_more_ids_than_fit_in_parameters():
    w = wl.WORKLOADS["8b_8k"]
    g = dims_of(w.shape, 384)
    pool = _pool_8b_384()
    src = wl.block_ids(5, g.NB, 136)
    dst = wl.block_ids(6, g.NB, 136)
    # one chunk of 136 blocks: more ids than the kernel parameters hold (128) -> id-table path
    run_pack_unpack(g, pool, src, dst, 136 * 16, kvc.KVC_VARIANT_AUTO, 0, "chunk")
    # the same with device-resident ids: read straight from the caller's array, any length
    run_pack_unpack(g, pool, src, dst, 136 * 16, kvc.KVC_VARIANT_AUTO, 0, "chunk_dev")


# ------------------------------------------------------------------ odd geometries
@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("geom,tile", [
    ((3, 2, 40, 4, 2, 8, 1), 0),        # fp8-like, S = 64 B
    ((2, 1, 33, 1, 1, 24, 2), 0),       # one plane per layer, S = 48 B: 16-byte vectors only
    ((2, 2, 50, 16, 4, 64, 2), 3088),   # S = 8 KiB cut into ragged tiles 3088+3088+2016
    ((1, 2, 19, 16, 8, 128, 4), 20480), # fp32, S = 64 KiB, tiles 20480*3 + 4096
    ((5, 2, 64, 8, 2, 128, 2), 0),      # block_size 8
])
def test_odd_geometries(variant, geom, tile):
    g = orc.Dims(*geom)
    pool = wl.random_bits(99 + g.L, g.pool_bytes)
    n = min(g.NB - 2, 27)
    src = wl.block_ids(1, g.NB, n)
    dst = wl.block_ids(2, g.NB, n)
    for mode in ("chunk", "batch"):
        run_pack_unpack(g, pool, src, dst, 4 * g.B, variant, kvc.KVC_ORDER_PLANE_MAJOR, mode, tile)


@pytest.mark.parametrize("variant", VARIANTS)
def test_padded_block_stride_and_plane_pointers(variant):
    """Blocks 1.5 slabs apart inside separately allocated planes: padding is never read or written."""
    g = orc.Dims(3, 2, 24, 16, 4, 64, 2)
    bs = g.slab_bytes * 3 // 2
    planes_np = []
    for i in range(g.L * g.P):
        q = np.full(g.NB * bs, 0xCC, dtype=np.uint8)
        q.reshape(g.NB, bs)[:, :g.slab_bytes] = wl.random_bits(40 + i, g.NB * g.slab_bytes).reshape(
            g.NB, g.slab_bytes)
        planes_np.append(q)
    planes_t = [to_dev(p) for p in planes_np]
    lay = kvc.kvc_layout_create(g.L, g.P, g.NB, g.B, g.H, g.D, g.e, 64, block_stride=bs,
                                plane_ptrs=planes_t)
    kvc.kvc_layout_set_tuning(lay, variant=variant)
    src = wl.block_ids(3, g.NB, 10)
    dst = wl.block_ids(4, g.NB, 10)
    staging = torch.zeros(10 * g.bytes_per_block, dtype=torch.uint8, device=DEV)
    ops, keep, nbytes, dev = kvc.request_chunk_ops(lay, src, staging)
    kvc.kvc_pack_batch(lay, ops, dev)
    ops2, keep2, _, _ = kvc.request_chunk_ops(lay, dst, staging)
    kvc.kvc_unpack_batch(lay, ops2, dev)
    torch.cuda.synchronize()
    host = staging.cpu().numpy()
    want_planes = [p.copy() for p in planes_np]
    off = 0
    for f, nb in orc.chunk_ranges(10, 4):
        want = orc.pack_chunk_planes(g, planes_np, src[f:f + nb], bs)
        assert np.array_equal(host[off:off + want.size], want)
        orc.unpack_chunk_planes(g, want_planes, want, dst[f:f + nb], bs)
        off += want.size
    for t, wnt in zip(planes_t, want_planes):
        got = t.cpu().numpy()
        assert np.array_equal(got, wnt)
        assert (got.reshape(g.NB, bs)[:, g.slab_bytes:] == 0xCC).all()


# ------------------------------------------------------------------ device-side id check
@pytest.mark.parametrize("variant", VARIANTS)
def test_bad_device_ids_are_skipped_and_counted(variant):
    g = orc.Dims(2, 2, 32, 16, 4, 64, 2)
    pool = wl.random_bits(77, g.pool_bytes)
    pool_t = to_dev(pool)
    lay = dense_layout(pool_t, g, 128)
    kvc.kvc_layout_set_tuning(lay, variant=variant)
    ids = np.array([3, 32, 7, -1, 9, 1 << 30, 0, 31], dtype=np.int32)   # three bad ids
    good = (ids >= 0) & (ids < g.NB)
    cb = kvc.kvc_layout_chunk_bytes(lay, 8)
    staging = torch.full((cb,), 0x11, dtype=torch.uint8, device=DEV)
    kvc.kvc_pack(lay, to_dev(ids), staging)
    assert kvc.kvc_poll_device_status(lay) == (3, 0)
    got = staging.cpu().numpy().reshape(g.L * g.P, 8, g.slab_bytes)
    safe = np.where(good, ids, 0).astype(np.int32)
    want = orc.pack_chunk(g, pool, safe).reshape(g.L * g.P, 8, g.slab_bytes)
    assert np.array_equal(got[:, good], want[:, good])
    assert (got[:, ~good] == 0x11).all()           # slabs of bad ids are left alone
    # unpack with bad ids: only the good blocks change
    chunk = wl.random_bits(78, cb)
    kvc.kvc_unpack(lay, to_dev(chunk), to_dev(ids))
    assert kvc.kvc_poll_device_status(lay) == (3, 0)
    assert kvc.kvc_poll_device_status(lay) == (0, 0)   # cleared by the poll
    want_pool = pool.copy()
    c3 = chunk.reshape(g.L * g.P, 8, g.slab_bytes)
    p3 = want_pool.reshape(g.L * g.P, g.NB, g.slab_bytes)
    for j in np.flatnonzero(good):
        p3[:, ids[j]] = c3[:, j]
    assert np.array_equal(pool_t.cpu().numpy(), want_pool)


def test_duplicate_source_blocks_in_pack():
    g = orc.Dims(2, 2, 16, 16, 4, 64, 2)
    pool = wl.random_bits(79, g.pool_bytes)
    lay = dense_layout(to_dev(pool), g, 16 * 6)
    ids = np.array([5, 5, 0, 15, 5, 0], dtype=np.int32)
    staging = torch.zeros(kvc.kvc_layout_chunk_bytes(lay, 6), dtype=torch.uint8, device=DEV)
    kvc.kvc_pack(lay, ids, staging)
    torch.cuda.synchronize()
    assert np.array_equal(staging.cpu().numpy(), orc.pack_chunk(g, pool, ids))


def test_limited_grid_still_correct():
    """max_ctas caps the launch (used to leave SMs to a compute stream); results do not change."""
    w = wl.WORKLOADS["8b_8k"]
    g = dims_of(w.shape, 384)
    pool = _pool_8b_384()
    src, dst = wl.block_ids(8, g.NB, 40), wl.block_ids(9, g.NB, 40)
    for variant in VARIANTS:
        pool_t = to_dev(pool)
        lay = dense_layout(pool_t, g, 256)
        kvc.kvc_layout_set_tuning(lay, variant=variant, max_ctas=3, stages=3)
        staging = torch.zeros(40 * g.bytes_per_block, dtype=torch.uint8, device=DEV)
        ops, keep, nbytes, dev = kvc.request_chunk_ops(lay, src, staging)
        kvc.kvc_pack_batch(lay, ops, dev)
        torch.cuda.synchronize()
        want = np.concatenate(orc.pack_request(g, pool, src, 256))
        assert np.array_equal(staging.cpu().numpy(), want)


# ------------------------------------------------------------------ config 4 (reduced): many requests, one launch
def test_batched_unpack_of_many_requests_with_shared_prefix():
    """70B-class geometry cut to 4 layers, lengths scaled by 1/8, chunk 64 tokens: every kept
    chunk of every request unpacked by ONE kvc_unpack_batch call; shared chunks staged once."""
    w = wl.WORKLOADS["70b_batch"]
    nb_pool, tables = wl.batch_workload(w, scale=1 / 8)
    g = orc.Dims(4, 2, nb_pool, 16, 8, 128, 2)
    chunk_tokens = 64
    pool = wl.random_bits(w.seed + 1, g.pool_bytes)
    pool_t = to_dev(pool)
    lay = dense_layout(pool_t, g, chunk_tokens)
    descs, uniq = kvc.kvc_map_requests_shared(lay, tables)
    assert uniq == len({int(b) for t in tables for b in t}) < sum(len(t) for t in tables)
    total = sum(d[4] for d in descs)
    assert total == uniq * g.bytes_per_block
    staged = wl.random_bits(w.seed + 2, total)            # "chunks as read from storage"
    staging = to_dev(staged)
    tabs_dev = [to_dev(t) for t in tables]
    launches0 = kvc.kvc_layout_launch_count(lay)
    for ids_on_device in (0, 1):
        pool_t.copy_(to_dev(pool))
        slot_addrs, ids_addrs, nbs, off = [], [], [], 0
        for (r, c, first, nb, nbytes) in descs:
            slot_addrs.append(staging.data_ptr() + off)
            base = tabs_dev[r].data_ptr() if ids_on_device else tables[r].ctypes.data
            ids_addrs.append(base + 4 * first)
            nbs.append(nb)
            off += nbytes
        ops = kvc.make_chunk_ops(slot_addrs, ids_addrs, nbs)
        kvc.kvc_unpack_batch(lay, ops, ids_on_device)
        torch.cuda.synchronize()
        want = pool.copy()
        off = 0
        for (r, c, first, nb, nbytes) in descs:
            orc.unpack_chunk(g, want, staged[off:off + nbytes], tables[r][first:first + nb])
            off += nbytes
        assert np.array_equal(pool_t.cpu().numpy(), want)
    assert kvc.kvc_layout_launch_count(lay) - launches0 == 2
    assert kvc.kvc_poll_device_status(lay) == (0, 0)


# ------------------------------------------------------------------ config 5 (reduced): ring streaming
@pytest.mark.parametrize("variant", VARIANTS)
def test_small_slabs_through_mapped_host_slots(variant):
    """Slabs of 512 bytes (the vector kernel gives each to one warp) packed straight into a slot in
    mapped pinned host memory and unpacked from it."""
    g = orc.Dims(6, 2, 200, 4, 2, 32, 2)              # S = 512 B
    pool = wl.random_bits(1500, g.pool_bytes)
    pool_t = to_dev(pool)
    lay = dense_layout(pool_t, g, 4 * 32)
    kvc.kvc_layout_set_tuning(lay, variant=variant)
    src, dst = wl.block_ids(15, g.NB, 70), wl.block_ids(16, g.NB, 70)
    cb = kvc.kvc_layout_chunk_bytes(lay, 32)
    ring = kvc.kvc_staging_ring_create((cb + 4095) // 4096 * 4096, 3, kvc.KVC_RING_HOST_MAPPED)
    want_chunks = orc.pack_request(g, pool, src, 4 * 32)
    want_pool = pool.copy()
    orc.unpack_request(g, want_pool, want_chunks, dst, 4 * 32)
    import ctypes
    held = []
    for c, (first, nb) in enumerate(orc.chunk_ranges(70, 32)):     # 3 chunks, 3 slots: pack them all
        slot, dptr, hptr = kvc.kvc_staging_ring_acquire(ring, 1_000_000)
        nbytes = kvc.kvc_layout_chunk_bytes(lay, nb)
        kvc.kvc_pack(lay, src[first:first + nb], dptr, nbytes)
        kvc.kvc_staging_ring_commit(ring, slot)
        kvc.kvc_staging_ring_sync_filled(ring, slot)
        got = np.ctypeslib.as_array((ctypes.c_uint8 * nbytes).from_address(hptr))
        assert np.array_equal(got, want_chunks[c]), "chunk %d" % c
        held.append((slot, dptr, first, nb, nbytes))
    for slot, dptr, first, nb, nbytes in held:                      # then unpack them from the slots
        kvc.kvc_unpack(lay, dptr, dst[first:first + nb], nbytes)
        kvc.kvc_staging_ring_release(ring, slot)
    torch.cuda.synchronize()
    assert np.array_equal(pool_t.cpu().numpy(), want_pool)
    assert kvc.kvc_poll_device_status(lay) == (0, 0)
    kvc.kvc_staging_ring_destroy(ring)


@pytest.mark.parametrize("kind", [kvc.KVC_RING_DEVICE, kvc.KVC_RING_HOST_MAPPED])
def test_prefix_streamed_through_ring_equals_one_shot_pack(kind):
    """A 2048-token prefix (8 chunks of 256 tokens) through a 3-slot ring while the copy stream
    drains each slot to host memory: host bytes equal the oracle's pack of the whole prefix; then
    the reverse (host -> ring -> unpack) restores a second pool."""
    w = wl.WORKLOADS["8b_ring"]
    g = dims_of(w.shape, 384)
    pool = _pool_8b_384()
    pool_t = to_dev(pool)
    lay = dense_layout(pool_t, g, 256)
    src = wl.block_ids(w.seed, g.NB, 128)
    dst = wl.block_ids(w.dst_seed, g.NB, 128)
    descs = kvc.kvc_map_request(lay, len(src))
    cb = kvc.kvc_layout_chunk_bytes(lay, 16)
    ring = kvc.kvc_staging_ring_create(cb, 3, kind)
    host_out = torch.empty(len(descs) * cb, dtype=torch.uint8).pin_memory()
    s_pack, s_copy = torch.cuda.Stream(), torch.cuda.Stream()
    for (_, c, first, nb, nbytes) in descs:
        slot, dptr, hptr = kvc.kvc_staging_ring_acquire(ring, timeout_us=5_000_000)
        assert slot == c % 3
        kvc.kvc_pack(lay, src[first:first + nb], dptr, cb, stream=s_pack)
        kvc.kvc_staging_ring_commit(ring, slot, s_pack)
        kvc.kvc_staging_ring_wait_filled(ring, slot, s_copy)
        src_addr = dptr if kind == kvc.KVC_RING_DEVICE else hptr
        kind_flag = cuda_rt.D2H if kind == kvc.KVC_RING_DEVICE else cuda_rt.H2H
        cuda_rt.memcpy_async(host_out.data_ptr() + c * cb, src_addr, nbytes, kind_flag, s_copy)
        kvc.kvc_staging_ring_release(ring, slot, s_copy)
    torch.cuda.synchronize()
    want = np.concatenate(orc.pack_request(g, pool, src, 256))
    assert np.array_equal(host_out.numpy(), want)
    in_flight, acquires, stalls = kvc.kvc_staging_ring_stats(ring)
    assert acquires == len(descs)
    # load direction: host -> ring slot -> unpack into other blocks
    for (_, c, first, nb, nbytes) in descs:
        slot, dptr, hptr = kvc.kvc_staging_ring_acquire(ring, timeout_us=5_000_000)
        dst_addr = dptr if kind == kvc.KVC_RING_DEVICE else hptr
        kind_flag = cuda_rt.H2D if kind == kvc.KVC_RING_DEVICE else cuda_rt.H2H
        cuda_rt.memcpy_async(dst_addr, host_out.data_ptr() + c * cb, nbytes, kind_flag, s_copy)
        kvc.kvc_staging_ring_commit(ring, slot, s_copy)       # here the copy stream is the producer
        kvc.kvc_staging_ring_wait_filled(ring, slot, s_pack)
        kvc.kvc_unpack(lay, dptr, dst[first:first + nb], cb, stream=s_pack)
        kvc.kvc_staging_ring_release(ring, slot, s_pack)
    torch.cuda.synchronize()
    want_pool = pool.copy()
    orc.unpack_request(g, want_pool, orc.pack_request(g, pool, src, 256), dst, 256)
    assert np.array_equal(pool_t.cpu().numpy(), want_pool)
    kvc.kvc_staging_ring_destroy(ring)
    assert kvc.kvc_poll_device_status(lay) == (0, 0)


# ------------------------------------------------------------------ copy-engine variants (DMA, no kernel)
@pytest.mark.parametrize("pool_kind", ["dense", "layer_gap", "separate_planes"])
@pytest.mark.parametrize("host_side", [False, True])
def test_copy_engine_variants_match_oracle(pool_kind, host_side):
    """kvc_pack_copy_engine / kvc_unpack_copy_engine move the same bytes with strided DMA copies:
    one per block (dense pool), one per layer (layers not equally spaced) or one per plane
    (separate allocations); the chunk may live in device memory or in pinned host memory."""
    g = orc.Dims(3, 2, 40, 16, 4, 64, 2)
    plane_bytes = g.NB * g.slab_bytes
    planes_np = [wl.random_bits(300 + i, plane_bytes) for i in range(g.L * g.P)]
    if pool_kind == "separate_planes":
        planes_t = [to_dev(p) for p in planes_np]
        lay = kvc.kvc_layout_create(g.L, g.P, g.NB, g.B, g.H, g.D, g.e, 64, plane_ptrs=planes_t)
        views = planes_t
    else:
        gap = 4096 if pool_kind == "layer_gap" else 0
        layer_stride = g.P * plane_bytes + gap
        buf = torch.full((g.L * layer_stride,), 0xEE, dtype=torch.uint8, device=DEV)
        views = []
        for l in range(g.L):
            for p in range(g.P):
                v = buf[l * layer_stride + p * plane_bytes:][:plane_bytes]
                v.copy_(to_dev(planes_np[l * g.P + p]))
                views.append(v)
        lay = kvc.kvc_layout_create(g.L, g.P, g.NB, g.B, g.H, g.D, g.e, 64, base=buf,
                                    layer_stride=layer_stride, plane_stride=plane_bytes)
    src, dst = wl.block_ids(31, g.NB, 11), wl.block_ids(32, g.NB, 11)
    total = 11 * g.bytes_per_block
    if host_side:
        staging = torch.full((total + 4096,), 0x44, dtype=torch.uint8).pin_memory()
    else:
        staging = torch.full((total + 4096,), 0x44, dtype=torch.uint8, device=DEV)
    launches0 = kvc.kvc_layout_launch_count(lay)
    off = 0
    want_chunks = []
    for f, nb in orc.chunk_ranges(11, 4):
        nbytes = kvc.kvc_layout_chunk_bytes(lay, nb)
        kvc.kvc_pack_copy_engine(lay, src[f:f + nb], staging.data_ptr() + off, nbytes)
        want_chunks.append(orc.pack_chunk_planes(g, planes_np, src[f:f + nb]))
        off += nbytes
    torch.cuda.synchronize()
    host = staging.cpu().numpy()
    assert np.array_equal(host[:total], np.concatenate(want_chunks))
    assert (host[total:] == 0x44).all()
    off = 0
    want_planes = [p.copy() for p in planes_np]
    for (f, nb), ch in zip(orc.chunk_ranges(11, 4), want_chunks):
        kvc.kvc_unpack_copy_engine(lay, staging.data_ptr() + off, dst[f:f + nb], ch.size)
        orc.unpack_chunk_planes(g, want_planes, ch, dst[f:f + nb])
        off += ch.size
    torch.cuda.synchronize()
    for v, wnt in zip(views, want_planes):
        assert np.array_equal(v.cpu().numpy(), wnt)
    if pool_kind == "layer_gap":
        b2 = buf.cpu().numpy().reshape(g.L, -1)
        assert (b2[:, g.P * plane_bytes:] == 0xEE).all()      # the gap between layers is untouched
    assert kvc.kvc_layout_launch_count(lay) == launches0      # no kernel ran
    with pytest.raises(kvc.KvcError) as e:
        kvc.kvc_unpack_copy_engine(lay, staging.data_ptr(), np.array([1, 2, 1], np.int32), total)
    assert e.value.status == kvc.KVC_ERR_CONFLICT
    with pytest.raises(kvc.KvcError) as e:
        kvc.kvc_pack_copy_engine(lay, np.array([g.NB], np.int32), staging.data_ptr(), total)
    assert e.value.status == kvc.KVC_ERR_OUT_OF_RANGE


# ------------------------------------------------------------------ random tiny layouts
def test_random_tiny_layouts():
    """Seeded random geometries (any element size, planes per layer, block size; slab bytes a
    multiple of 16), random tables, chunk sizes, kernels, tiles and traversal orders; host and
    device ids; per-chunk and batched calls.  Every case byte for byte against the oracle."""
    rng = np.random.default_rng(20260911)
    done = 0
    while done < 40:
        e = int(rng.choice([1, 2, 4]))
        L, P = int(rng.integers(1, 5)), int(rng.integers(1, 3))
        B, H = int(rng.integers(1, 9)), int(rng.integers(1, 5))
        D = int(rng.choice([8, 16, 24, 32, 40, 64, 128]))
        S = B * H * D * e
        if S % 16:
            continue
        NB = int(rng.integers(2, 60))
        g = orc.Dims(L, P, NB, B, H, D, e)
        n = int(rng.integers(1, NB + 1))
        bpc = int(rng.integers(1, n + 2))
        pool = wl.random_bits(int(rng.integers(1 << 30)), g.pool_bytes + (g.pool_bytes & 1))[:g.pool_bytes]
        src = rng.permutation(NB)[:n].astype(np.int32)
        dst = rng.permutation(NB)[:n].astype(np.int32)
        variant = int(rng.choice(VARIANTS))
        order = int(rng.choice([1, 2, 3]))
        tile = int(rng.choice([0, 16, 48, 256, 4096]))
        mode = str(rng.choice(["chunk", "chunk_dev", "batch", "batch_dev"]))
        run_pack_unpack(g, pool, src, dst, bpc * B, variant, order, mode, tile)
        done += 1


@pytest.mark.parametrize("seed", [7, 8, 9])
def test_random_layouts_with_random_launch_shapes(seed):
    """As above, and the launch shape is drawn at random too: slabs per work item, stages, loads
    ahead, blocks (persistent or streaming), items per block, threads per vector block, L2 hints,
    dependent launch on or off.  No knob may change a byte."""
    rng = np.random.default_rng(seed)
    done = 0
    while done < 30:
        e = int(rng.choice([1, 2, 4]))
        L, P = int(rng.integers(1, 6)), int(rng.integers(1, 3))
        B, H = int(rng.integers(1, 17)), int(rng.integers(1, 9))
        D = int(rng.choice([8, 16, 32, 64, 128]))
        S = B * H * D * e
        if S % 16 or S > 65536:
            continue
        NB = int(rng.integers(2, 80))
        if L * P * NB * S > (96 << 20):
            continue
        g = orc.Dims(L, P, NB, B, H, D, e)
        n = int(rng.integers(1, NB + 1))
        bpc = int(rng.integers(1, n + 2))
        pool = wl.random_bits(int(rng.integers(1 << 30)), g.pool_bytes + (g.pool_bytes & 1))[:g.pool_bytes]
        src = rng.permutation(NB)[:n].astype(np.int32)
        dst = rng.permutation(NB)[:n].astype(np.int32)
        variant = int(rng.choice(VARIANTS))
        stages = int(rng.choice([0, 2, 3, 4, 8, 16]))
        tuning = dict(
            group=int(rng.choice([0, 1, 2, 4, 8, 16, 32, kvc.KVC_GROUP_FORCE_KERNEL])),
            stages=stages,
            lag=int(rng.integers(0, max(1, stages - 1))) if stages > 2 else 0,
            max_ctas=int(rng.choice([0, 0, 1, 3, 17, 148])),
            items_per_cta=int(rng.choice([0, 1, 2, 5, 40])),
            vec_threads=int(rng.choice([0, 32, 64, 128, 256])),
            l2_hint=int(rng.integers(0, 5)),
            pdl=int(rng.integers(0, 3)),
        )
        tile = int(rng.choice([0, 0, 1024, 4096, 8192, 16384]))
        order = int(rng.choice([0, 1, 2, 3]))
        mode = str(rng.choice(["chunk", "chunk_dev", "batch", "batch_dev"]))
        try:
            run_pack_unpack(g, pool, src, dst, bpc * B, variant, order, mode, tile, **tuning)
        except AssertionError as err:
            raise AssertionError("%s with geometry %r, %d blocks in chunks of %d, variant %d, order %d, "
                                 "mode %s, tile %d, tuning %r" % (err, g, n, bpc, variant, order, mode,
                                                                  tile, tuning))
        done += 1


# ------------------------------------------------------------------ layout variants
@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("mode", ["chunk", "batch_dev", "copy_engine", "static"])
def test_block_major_chunk_order(variant, mode):
    """Chunks in block-major order [n][L][P][B][H][D] through every entry point."""
    g = orc.Dims(4, 2, 48, 16, 4, 64, 2)
    pool = wl.random_bits(500, g.pool_bytes)
    pool_t = to_dev(pool)
    lay = kvc.kvc_layout_create_dense(pool_t, g.L, g.P, g.NB, g.B, g.H, g.D, g.e, 64,
                                      chunk_order=kvc.KVC_CHUNK_BLOCK_MAJOR)
    kvc.kvc_layout_set_tuning(lay, variant=variant, order=kvc.KVC_ORDER_CHUNK_MAJOR if variant == 2
                              else kvc.KVC_ORDER_PLANE_MAJOR)
    src, dst = wl.block_ids(51, g.NB, 14), wl.block_ids(52, g.NB, 14)
    total = 14 * g.bytes_per_block
    staging = torch.full((total + 4096,), 0x66, dtype=torch.uint8, device=DEV)
    ranges = orc.chunk_ranges(14, 4)
    planes = orc.dense_planes(g, pool)
    want_chunks = [orc.pack_chunk_planes_block_major(g, planes, src[f:f + nb]) for f, nb in ranges]

    def run(direction, ids):
        if mode == "batch_dev" or (mode == "static" and direction == 1):
            ops, keep, nbytes, dev = kvc.request_chunk_ops(lay, to_dev(ids), staging)
            (kvc.kvc_pack_batch if direction == 0 else kvc.kvc_unpack_batch)(lay, ops, dev)
        elif mode == "static":
            ops, keep, nbytes, dev = kvc.request_chunk_ops(lay, ids, staging)
            kvc.kvc_pack_batch_static(lay, ops)
        else:
            off = 0
            for f, nb in ranges:
                nbytes = kvc.kvc_layout_chunk_bytes(lay, nb)
                slot = staging[off:off + nbytes]
                if mode == "chunk":
                    (kvc.kvc_pack(lay, ids[f:f + nb], slot) if direction == 0
                     else kvc.kvc_unpack(lay, slot, ids[f:f + nb]))
                else:
                    (kvc.kvc_pack_copy_engine(lay, ids[f:f + nb], slot) if direction == 0
                     else kvc.kvc_unpack_copy_engine(lay, slot, ids[f:f + nb]))
                off += nbytes
        torch.cuda.synchronize()

    run(0, src)
    host = staging.cpu().numpy()
    assert np.array_equal(host[:total], np.concatenate(want_chunks))
    assert (host[total:] == 0x66).all()
    # the short last chunk is a prefix of what a full chunk starting there would be
    run(1, dst)
    want_pool = pool.copy()
    for (f, nb), ch in zip(ranges, want_chunks):
        orc.unpack_chunk_planes_block_major(g, orc.dense_planes(g, want_pool), ch, dst[f:f + nb])
    assert np.array_equal(pool_t.cpu().numpy(), want_pool)
    assert kvc.kvc_poll_device_status(lay) == (0, 0)


@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("chunk_order", [kvc.KVC_CHUNK_LAYER_MAJOR, kvc.KVC_CHUNK_BLOCK_MAJOR])
def test_pool_with_kv_inside_the_block_axis(variant, chunk_order):
    """Pool order [L][NB][P][B][H][D] (K and V of a block adjacent): described by plane stride S and
    block stride P*S.  Chunks equal those of the same data in the dense order."""
    g = orc.Dims(3, 2, 30, 16, 4, 64, 2)
    S = g.slab_bytes
    dense = wl.random_bits(600, g.pool_bytes)
    inter = np.ascontiguousarray(dense.reshape(g.L, g.P, g.NB, S).transpose(0, 2, 1, 3)).reshape(-1)
    pool_t = to_dev(inter)
    lay = kvc.kvc_layout_create(g.L, g.P, g.NB, g.B, g.H, g.D, g.e, 64, base=pool_t,
                                layer_stride=g.NB * g.P * S, plane_stride=S, block_stride=g.P * S,
                                chunk_order=chunk_order)
    kvc.kvc_layout_set_tuning(lay, variant=variant)
    src, dst = wl.block_ids(61, g.NB, 9), wl.block_ids(62, g.NB, 9)
    staging = torch.zeros(9 * g.bytes_per_block, dtype=torch.uint8, device=DEV)
    ops, keep, nbytes, dev = kvc.request_chunk_ops(lay, src, staging)
    kvc.kvc_pack_batch(lay, ops, dev)
    torch.cuda.synchronize()
    planes = orc.dense_planes(g, dense)
    packer = (orc.pack_chunk_planes if chunk_order == kvc.KVC_CHUNK_LAYER_MAJOR
              else orc.pack_chunk_planes_block_major)
    unpacker = (orc.unpack_chunk_planes if chunk_order == kvc.KVC_CHUNK_LAYER_MAJOR
                else orc.unpack_chunk_planes_block_major)
    chunks = [packer(g, planes, src[f:f + nb]) for f, nb in orc.chunk_ranges(9, 4)]
    assert np.array_equal(staging.cpu().numpy(), np.concatenate(chunks))
    # copy-engine pack of the first chunk gives the same bytes
    again = torch.zeros(chunks[0].size, dtype=torch.uint8, device=DEV)
    kvc.kvc_pack_copy_engine(lay, src[:4], again)
    ops2, keep2, _, _ = kvc.request_chunk_ops(lay, dst, staging)
    kvc.kvc_unpack_batch(lay, ops2, dev)
    torch.cuda.synchronize()
    assert np.array_equal(again.cpu().numpy(), chunks[0])
    want = dense.copy()
    for (f, nb), ch in zip(orc.chunk_ranges(9, 4), chunks):
        unpacker(g, orc.dense_planes(g, want), ch, dst[f:f + nb])
    want_inter = np.ascontiguousarray(want.reshape(g.L, g.P, g.NB, S).transpose(0, 2, 1, 3)).reshape(-1)
    assert np.array_equal(pool_t.cpu().numpy(), want_inter)


# ------------------------------------------------------------------ many launches in flight, two streams
def test_many_batched_launches_on_two_streams_share_one_handle():
    """More batched launches than the handle has id-table buffers, issued back to back on two
    streams without synchronising: every launch must read its own table.  Some ops are empty."""
    g = orc.Dims(2, 2, 64, 16, 4, 64, 2)
    pool = wl.random_bits(800, g.pool_bytes)
    pool_t = to_dev(pool)
    lay = dense_layout(pool_t, g, 64)
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    n_launch, per = 24, 10
    staging = torch.zeros(n_launch * per * g.bytes_per_block, dtype=torch.uint8, device=DEV)
    tables, keep = [], []
    for k in range(n_launch):
        ids = wl.block_ids(900 + k, g.NB, per)
        tables.append(ids)
        base = staging.data_ptr() + k * per * g.bytes_per_block
        sizes = [kvc.kvc_layout_chunk_bytes(lay, nb) for _, nb in orc.chunk_ranges(per, 4)]
        offs = np.concatenate([[0], np.cumsum(sizes)[:-1]])
        slot_addrs = [base + int(o) for o in offs] + [base]            # last op is empty
        id_addrs = [ids.ctypes.data + 4 * f for f, _ in orc.chunk_ranges(per, 4)] + [ids.ctypes.data]
        nbs = [nb for _, nb in orc.chunk_ranges(per, 4)] + [0]
        ops = kvc.make_chunk_ops(slot_addrs, id_addrs, nbs)
        keep.append(ops)
        kvc.kvc_pack_batch(lay, ops, 0, stream=streams[k % 2])
    torch.cuda.synchronize()
    host = staging.cpu().numpy()
    for k in range(n_launch):
        want = np.concatenate(orc.pack_request(g, pool, tables[k], 64))
        got = host[k * per * g.bytes_per_block:(k + 1) * per * g.bytes_per_block]
        assert np.array_equal(got, want), "launch %d" % k
    assert kvc.kvc_layout_launch_count(lay) == n_launch
    assert kvc.kvc_poll_device_status(lay) == (0, 0)


# ------------------------------------------------------------------ CUDA graph capture of per-chunk calls
def test_per_chunk_calls_replay_from_a_cuda_graph():
    """kvc_pack / kvc_unpack with at most 128 host ids (they travel in the kernel parameters) or
    with device ids enqueue exactly one kernel and nothing else, so a sequence of them can be
    captured into a CUDA graph once the handle has made its first launch, and replayed."""
    g = orc.Dims(4, 2, 64, 16, 8, 128, 2)
    pool = wl.random_bits(950, g.pool_bytes)
    pool_t = to_dev(pool)
    lay = dense_layout(pool_t, g, 64)
    src, dst = wl.block_ids(95, g.NB, 16), wl.block_ids(96, g.NB, 16)
    dst_dev = to_dev(dst)
    cb = kvc.kvc_layout_chunk_bytes(lay, 4)
    staging = torch.zeros(4 * cb, dtype=torch.uint8, device=DEV)
    kvc.kvc_pack(lay, src[:4], staging[:cb])          # first launch: allocates the handle's device state
    torch.cuda.synchronize()
    staging.zero_()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        for c in range(4):
            kvc.kvc_pack(lay, src[4 * c:4 * c + 4], staging[c * cb:(c + 1) * cb])
        for c in range(4):
            kvc.kvc_unpack(lay, staging[c * cb:(c + 1) * cb], dst_dev[4 * c:4 * c + 4].contiguous())
    torch.cuda.synchronize()
    assert bool((staging == 0).all())                 # capture enqueued nothing
    want_chunks = orc.pack_request(g, pool, src, 64)
    want_pool = pool.copy()
    orc.unpack_request(g, want_pool, want_chunks, dst, 64)
    for _ in range(2):
        pool_t.copy_(to_dev(pool))
        staging.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert np.array_equal(staging.cpu().numpy(), np.concatenate(want_chunks))
        assert np.array_equal(pool_t.cpu().numpy(), want_pool)
    assert kvc.kvc_poll_device_status(lay) == (0, 0)


# ------------------------------------------------------------------ every tuning knob keeps the bytes right
@pytest.mark.parametrize("tuning", [
    dict(variant=2, stages=2), dict(variant=2, stages=3, lag=1), dict(variant=2, stages=7, lag=5),
    dict(variant=2, stages=16, tile_bytes=8192, lag=3), dict(variant=2, stages=6, lag=2, max_ctas=5),
    dict(variant=2, ctas_per_sm=2, stages=3), dict(variant=2, ctas_per_sm=4, tile_bytes=16384),
    dict(variant=2, l2_hint=2), dict(variant=2, pdl=1), dict(variant=1, pdl=1, tile_bytes=32768),
    dict(variant=1, max_ctas=1), dict(variant=2, max_ctas=1, stages=2),
    dict(items_per_cta=1), dict(items_per_cta=7, stages=3), dict(variant=1, items_per_cta=3),
    dict(variant=2, order=1, items_per_cta=5), dict(variant=1, order=2, tile_bytes=4096),
])
def test_tuning_knobs_do_not_change_results(tuning):
    g = orc.Dims(8, 2, 96, 16, 8, 128, 2)
    key = "tuning_pool"
    if key not in _POOL_CACHE:
        _POOL_CACHE[key] = wl.random_bits(1234, g.pool_bytes)
    pool = _POOL_CACHE[key]
    src, dst = wl.block_ids(12, g.NB, 37), wl.block_ids(13, g.NB, 37)
    pool_t = to_dev(pool)
    lay = dense_layout(pool_t, g, 256)
    kvc.kvc_layout_set_tuning(lay, **tuning)
    want_chunks, want_pool = _oracle_results(g, pool, src, dst, 256)
    total = 37 * g.bytes_per_block
    staging = torch.zeros(total, dtype=torch.uint8, device=DEV)
    off = 0
    for f, nb in orc.chunk_ranges(37, 16):            # per-chunk calls, back to back
        nbytes = kvc.kvc_layout_chunk_bytes(lay, nb)
        kvc.kvc_pack(lay, src[f:f + nb], staging[off:off + nbytes])
        off += nbytes
    ops, keep, _, dev = kvc.request_chunk_ops(lay, dst, staging)
    kvc.kvc_unpack_batch(lay, ops, dev)
    torch.cuda.synchronize()
    assert np.array_equal(staging.cpu().numpy(), np.concatenate(want_chunks))
    assert np.array_equal(pool_t.cpu().numpy(), want_pool)
    assert kvc.kvc_poll_device_status(lay) == (0, 0)


# ------------------------------------------------------------------ the C ABI from plain C
def test_plain_c_program_links_and_runs(tmp_path):
    """include/kvc.h is a C header: a C99 program built with gcc against libkvc.so packs and
    unpacks on the GPU and checks the bytes itself."""
    import os
    import shutil
    import subprocess
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    cuda = os.environ.get("CUDA_HOME", "/usr/local/cuda")
    if shutil.which("gcc") is None or not os.path.isdir(os.path.join(cuda, "include")):
        pytest.skip("needs gcc and the CUDA toolkit headers")
    exe = str(tmp_path / "c_abi_smoke")
    pkg = os.path.join(root, "paper_2609_11744_b200")
    build = subprocess.run(
        ["gcc", "-std=c99", "-O1", "-Wall", os.path.join(root, "tests", "native", "c_abi_smoke.c"),
         "-I", os.path.join(root, "include"), "-I", os.path.join(cuda, "include"),
         "-L", pkg, "-lkvc", "-L", os.path.join(cuda, "lib64"), "-lcudart",
         "-Wl,-rpath," + pkg, "-Wl,-rpath," + os.path.join(cuda, "lib64"), "-o", exe],
        capture_output=True, text=True)
    assert build.returncode == 0, build.stderr
    run = subprocess.run([exe], capture_output=True, text=True, timeout=120)
    assert run.returncode == 0 and run.stdout.strip() == "ok", run.stdout + run.stderr


@pytest.mark.parametrize("vec_threads", [32, 64, 224])
def test_vector_kernel_with_small_blocks_on_8b_shape(vec_threads):
    """Blocks of fewer than 256 threads: every warp copies its own 4 KiB tile of the 32 KiB slabs."""
    g = dims_of(wl.LLAMA_8B, 384)
    pool = _pool_8b_384()
    src, dst = wl.block_ids(8, g.NB, 40), wl.block_ids(9, g.NB, 40)
    for mode, tuning in (("batch", dict()), ("chunk", dict(max_ctas=24))):
        run_pack_unpack(g, pool, src, dst, 256, kvc.KVC_VARIANT_VEC, 0, mode, vec_threads=vec_threads,
                        **tuning)


def test_kernel_timing_and_slot_memory_hint():
    """Diagnostics and hints do not change a byte: with kernel timing on, every launch is reported
    with a positive duration; with the slot_memory hint the pointer query is skipped and the right
    kernel family still runs for device slots (hint 1) and mapped host slots (hint 2)."""
    g = dims_of(wl.LLAMA_8B, 384)
    pool = _pool_8b_384()
    pool_t = to_dev(pool)
    ids = wl.block_ids(88, g.NB, 37)
    want = np.concatenate(orc.pack_request(g, pool, ids, 256))
    lay = dense_layout(pool_t, g, 256)
    kvc.kvc_layout_set_tuning(lay, slot_memory=1)
    kvc.kvc_layout_set_kernel_timing(lay, True)
    out = torch.zeros(want.size, dtype=torch.uint8, device=DEV)
    ops, keep, nbytes, dev = kvc.request_chunk_ops(lay, ids, out)
    kvc.kvc_pack_batch(lay, ops, dev)
    kvc.kvc_pack(lay, ids[:16], out[:kvc.kvc_layout_chunk_bytes(lay, 16)])
    n, total, lo, hi = kvc.kvc_layout_kernel_time(lay)
    assert n == 2 and 0 < lo <= hi and abs(total - (lo + hi)) < 1e-6
    assert kvc.kvc_layout_kernel_time(lay)[0] == 0               # collected once
    kvc.kvc_layout_set_kernel_timing(lay, False)
    kvc.kvc_pack_batch(lay, ops, dev)
    assert kvc.kvc_layout_kernel_time(lay)[0] == 0
    torch.cuda.synchronize()
    assert np.array_equal(out.cpu().numpy(), want)
    # mapped host slots with the hint
    cb = kvc.kvc_layout_chunk_bytes(lay, 16)
    ring = kvc.kvc_staging_ring_create(cb, 1, kvc.KVC_RING_HOST_MAPPED)
    kvc.kvc_layout_set_tuning(lay, slot_memory=2)
    slot, dptr, hptr = kvc.kvc_staging_ring_acquire(ring, 1_000_000)
    kvc.kvc_pack(lay, ids[:16], dptr, cb)
    kvc.kvc_staging_ring_commit(ring, slot)
    kvc.kvc_staging_ring_sync_filled(ring, slot)
    import ctypes
    got = np.ctypeslib.as_array((ctypes.c_uint8 * cb).from_address(hptr))
    assert np.array_equal(got, want[:cb])
    kvc.kvc_staging_ring_release(ring, slot)
    with pytest.raises(kvc.KvcError):
        kvc.kvc_layout_set_tuning(lay, slot_memory=3)
    assert kvc.kvc_poll_device_status(lay) == (0, 0)
    kvc.kvc_staging_ring_destroy(ring)
