"""Store / load pipelines on a GPU: request -> mapped-host ring -> chunk files -> ring -> other
blocks, against the oracle; shared entries are written once; loads stop at the first gap."""
import os

import numpy as np
import pytest

torch = pytest.importorskip("torch")

from oracle import oracle as orc
from paper_2609_11744_b200 import kvc
import workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.mark.parametrize("ring_kind", [kvc.KVC_RING_HOST_MAPPED, kvc.KVC_RING_DEVICE_STAGED])
@pytest.mark.parametrize("use_copy_engine", [False, True])
def test_store_then_load_through_files(tmp_path, use_copy_engine, ring_kind):
    g = orc.Dims(6, 2, 96, 16, 8, 128, 2)            # 8B shape cut to 6 layers; chunk = 6 MiB
    pool = wl.random_bits(700, g.pool_bytes)
    pool_t = torch.from_numpy(pool).to(DEV)
    lay = kvc.kvc_layout_create_dense(pool_t, g.L, g.P, g.NB, g.B, g.H, g.D, g.e, 256)
    src, dst = wl.block_ids(71, g.NB, 44), wl.block_ids(72, g.NB, 44)     # 2 full chunks + 12 blocks
    cb = kvc.kvc_layout_chunk_bytes(lay, 16)
    ring = kvc.kvc_staging_ring_create(cb, 2, ring_kind)                  # request > ring
    if ring_kind == kvc.KVC_RING_DEVICE_STAGED and not use_copy_engine:
        # device halves at HBM speed, copy engines across the link: the set-up for a busy GPU
        kvc.kvc_layout_set_tuning(lay, **kvc.kvc_tuning_preset(kvc.KVC_PRESET_BESIDE_COMPUTE))
    store = kvc.kvc_store_open(str(tmp_path), "shape-6x2x8x128-bf16", direct_io=True)
    tokens = np.arange(44 * 16, dtype=np.int32) * 7 + 3
    hashes, h = [], 0
    for c in range(3):
        h = kvc.kvc_chain_hash(h, tokens[c * 256:(c + 1) * 256])
        hashes.append(h)
    st = kvc.kvc_pipeline_store(lay, ring, store, src, hashes, io_threads=3,
                                use_copy_engine=use_copy_engine)
    assert (st["chunks"], st["published"], st["already_present"]) == (3, 3, 0)
    assert st["bytes"] == 44 * g.bytes_per_block
    want_chunks = orc.pack_request(g, pool, src, 256)
    for c, hh in enumerate(hashes):                   # files hold exactly the oracle's chunks
        path = kvc.kvc_store_path(store, hh)
        assert np.array_equal(np.fromfile(path, dtype=np.uint8), want_chunks[c])
    # a second instance storing the same prefix writes nothing
    st2 = kvc.kvc_pipeline_store(lay, ring, store, src, hashes, use_copy_engine=use_copy_engine)
    assert (st2["published"], st2["already_present"]) == (0, 3)
    # load into other blocks
    ld = kvc.kvc_pipeline_load(lay, ring, store, dst, hashes, io_threads=2,
                               use_copy_engine=use_copy_engine)
    torch.cuda.synchronize()
    assert ld["chunks"] == 3 and ld["bytes"] == 44 * g.bytes_per_block
    want_pool = pool.copy()
    orc.unpack_request(g, want_pool, want_chunks, dst, 256)
    assert np.array_equal(pool_t.cpu().numpy(), want_pool)
    # a gap: without the second chunk only the first one is loaded (contiguous prefix)
    os.unlink(kvc.kvc_store_path(store, hashes[1]))
    pool_t.copy_(torch.from_numpy(pool))
    ld2 = kvc.kvc_pipeline_load(lay, ring, store, dst, hashes, use_copy_engine=use_copy_engine)
    torch.cuda.synchronize()
    assert ld2["chunks"] == 1
    want_pool = pool.copy()
    orc.unpack_chunk(g, want_pool, want_chunks[0], dst[:16])
    assert np.array_equal(pool_t.cpu().numpy(), want_pool)
    assert kvc.kvc_staging_ring_stats(ring)[0] <= 2
    assert kvc.kvc_poll_device_status(lay) == (0, 0)
    # a device ring has no host-visible slots: refused
    dring = kvc.kvc_staging_ring_create(cb, 2, kvc.KVC_RING_DEVICE)
    with pytest.raises(kvc.KvcError) as e:
        kvc.kvc_pipeline_store(lay, dring, store, src, hashes)
    assert e.value.status == kvc.KVC_ERR_INVALID_ARG
    assert kvc.kvc_staging_ring_stats(dring)[0] == 0


def _hashes(seed, n_chunks, shared=0, shared_seed=999):
    """Chain hashes (Sec. 2.1) of a request whose first `shared` chunks hold a common prefix."""
    out, h = [], 0
    for c in range(n_chunks):
        rng = np.random.default_rng((shared_seed if c < shared else seed) * 1000 + c)
        h = kvc.kvc_chain_hash(h, rng.integers(0, 50000, 256).astype(np.int32))
        out.append(h)
    return out


@pytest.mark.parametrize("ring_kind", [kvc.KVC_RING_HOST_MAPPED, kvc.KVC_RING_DEVICE_STAGED])
@pytest.mark.parametrize("pool_mode", [False, True])
def test_failing_pack_inside_the_store_pipeline_returns_every_slot(tmp_path, pool_mode, ring_kind):
    """An out-of-range block id in the third chunk: the call reports OUT_OF_RANGE, no slot stays
    taken, and the next store on the same ring runs normally."""
    g = orc.Dims(4, 2, 96, 16, 8, 128, 2)
    pool = wl.random_bits(701, g.pool_bytes)
    pool_t = torch.from_numpy(pool).to(DEV)
    lay = kvc.kvc_layout_create_dense(pool_t, g.L, g.P, g.NB, g.B, g.H, g.D, g.e, 256)
    cb = kvc.kvc_layout_chunk_bytes(lay, 16)
    ring = kvc.kvc_staging_ring_create(cb, 3, ring_kind)
    if pool_mode:
        kvc.kvc_staging_ring_set_policy(ring, 1)
    store = kvc.kvc_store_open(str(tmp_path), "m", direct_io=True)
    src = wl.block_ids(73, g.NB, 80)                       # 5 chunks
    bad = src.copy()
    bad[37] = g.NB                                         # inside chunk 2
    hashes = _hashes(1, 5)
    with pytest.raises(kvc.KvcError) as e:
        kvc.kvc_pipeline_store(lay, ring, store, bad, hashes, io_threads=2)
    assert e.value.status == kvc.KVC_ERR_OUT_OF_RANGE
    torch.cuda.synchronize()
    if pool_mode:
        c = kvc.kvc_staging_ring_policy_counters(ring)
        assert (c["n_free"], c["n_in_flight"], c["n_staged"]) == (3, 0, 0)
    else:
        assert kvc.kvc_staging_ring_stats(ring)[0] == 0
    # chunks before the failure may have been published; none after it
    assert kvc.kvc_store_lookup(store, hashes[3]) is None and kvc.kvc_store_lookup(store, hashes[4]) is None
    st = kvc.kvc_pipeline_store(lay, ring, store, src, hashes, io_threads=2)
    assert st["chunks"] == 5 and st["published"] + st["already_present"] == 5
    want = orc.pack_request(g, pool, src, 256)
    for c, hh in enumerate(hashes):
        assert np.array_equal(np.fromfile(kvc.kvc_store_path(store, hh), dtype=np.uint8), want[c])
    # the same for loads: a bad destination id in the second chunk
    dst = wl.block_ids(74, g.NB, 80)
    bad = dst.copy()
    bad[20] = -5
    with pytest.raises(kvc.KvcError) as e:
        kvc.kvc_pipeline_load(lay, ring, store, bad, hashes, io_threads=2)
    assert e.value.status == kvc.KVC_ERR_OUT_OF_RANGE
    torch.cuda.synchronize()
    if pool_mode:
        c = kvc.kvc_staging_ring_policy_counters(ring)
        assert (c["n_free"], c["n_in_flight"], c["n_staged"]) == (3, 0, 0)
    else:
        assert kvc.kvc_staging_ring_stats(ring)[0] == 0
    pool_t.copy_(torch.from_numpy(pool))
    ld = kvc.kvc_pipeline_load(lay, ring, store, dst, hashes, io_threads=2)
    torch.cuda.synchronize()
    assert ld["chunks"] == 5
    want_pool = pool.copy()
    orc.unpack_request(g, want_pool, want, dst, 256)
    assert np.array_equal(pool_t.cpu().numpy(), want_pool)
    assert kvc.kvc_poll_device_status(lay) == (0, 0)


@pytest.mark.parametrize("ring_kind", [kvc.KVC_RING_HOST_MAPPED, kvc.KVC_RING_DEVICE_STAGED])
def test_four_requests_sharing_a_prefix_are_served_from_one_pool(tmp_path, ring_kind):
    """Four requests whose first 1024 tokens (4 chunks) are the same prefix, loaded at once through
    files and one staging pool (Sec. 6.5): every shared chunk is read once and joined by the other
    three requests, every request's blocks equal the oracle's, and chunks preloaded by an earlier
    call are claimed by the demand loads instead of being read again."""
    g = orc.Dims(4, 2, 640, 16, 8, 128, 2)                 # 8B shape cut to 4 layers; chunk = 4 MiB
    pool = wl.random_bits(702, g.pool_bytes)
    pool_t = torch.from_numpy(pool).to(DEV)
    lay = kvc.kvc_layout_create_dense(pool_t, g.L, g.P, g.NB, g.B, g.H, g.D, g.e, 256)
    cb = kvc.kvc_layout_chunk_bytes(lay, 16)
    store = kvc.kvc_store_open(str(tmp_path), "m", direct_io=True)
    # what is in the store: a "source" request per stored request, all with the same first 64 blocks
    perm = np.random.default_rng(8).permutation(g.NB).astype(np.int32)
    shared_src = perm[:64]
    lens = [64 + 40, 64 + 16, 64 + 75, 64]                 # blocks; two ragged tails, one prefix-only
    srcs, cur = [], 64
    for n in lens:
        srcs.append(np.ascontiguousarray(np.concatenate([shared_src, perm[cur:cur + n - 64]])))
        cur += n - 64
    hashes = [_hashes(10 + r, kvc.kvc_layout_num_chunks(lay, n), shared=4) for r, n in enumerate(lens)]
    fifo = kvc.kvc_staging_ring_create(cb, 4, kvc.KVC_RING_HOST_MAPPED)
    for r in range(4):
        kvc.kvc_pipeline_store(lay, fifo, store, srcs[r], hashes[r], io_threads=3)
    kvc.kvc_staging_ring_destroy(fifo)
    want_chunks = [orc.pack_request(g, pool, s, 256) for s in srcs]
    n_files = len({h for hs in hashes for h in hs})
    assert kvc.kvc_store_get_counters(store)["publishes"] == n_files == 4 + 3 + 1 + 5
    # destination blocks: distinct for every request
    dsts = []
    for n in lens:
        dsts.append(np.ascontiguousarray(perm[cur:cur + n]))
        cur += n
    assert cur <= g.NB
    want_pool = pool.copy()
    for r in range(4):
        orc.unpack_request(g, want_pool, want_chunks[r], dsts[r], 256)

    ring = kvc.kvc_staging_ring_create(cb, 6, ring_kind)
    kvc.kvc_staging_ring_set_policy(ring, foreground_reserve=2, max_speculative=4)
    reads0 = kvc.kvc_store_get_counters(store)["reads"]
    # 1. a preload of request 2's prefix, issued before anything is scheduled
    stats, res = kvc.kvc_pipeline_load_many(lay, ring, store, [
        dict(hashes=hashes[2], n_blocks=lens[2], cls=kvc.KVC_CLASS_PRELOAD)], io_threads=3)
    staged = res[0]["loaded_chunks"]
    assert 1 <= staged <= 4                                  # bounded by the reserve: 6 slots - 2
    assert stats["reads"] == staged and stats["unpack_launches"] == 0
    c = kvc.kvc_staging_ring_policy_counters(ring)
    assert c["n_staged"] == staged and c["n_in_flight"] == 0
    # 2. all four requests as demand loads in one call
    reqs = [dict(ids=dsts[r], hashes=hashes[r], cls=kvc.KVC_CLASS_DEMAND_LOAD) for r in range(4)]
    stats, res = kvc.kvc_pipeline_load_many(lay, ring, store, reqs, io_threads=3)
    torch.cuda.synchronize()
    assert [x["loaded_chunks"] for x in res] == [kvc.kvc_layout_num_chunks(lay, n) for n in lens]
    assert np.array_equal(pool_t.cpu().numpy(), want_pool)
    total_pairs = sum(kvc.kvc_layout_num_chunks(lay, n) for n in lens)
    assert stats["chunks"] == total_pairs
    # every file is read at most once over both calls; the shared chunks exactly once
    reads = kvc.kvc_store_get_counters(store)["reads"] - reads0
    assert reads == n_files
    assert stats["reads"] == n_files - staged
    assert stats["joins"] == total_pairs - stats["reads"]
    assert stats["claims"] >= 1                              # the preload was claimed, not re-read
    assert stats["unpack_launches"] <= stats["reads"] + 2   # fused: never one launch per (request, chunk)
    assert all(x["ready_seconds"] > 0 for x in res)
    c = kvc.kvc_staging_ring_policy_counters(ring)
    assert (c["n_free"], c["n_in_flight"], c["n_staged"]) == (6, 0, 0)
    assert kvc.kvc_poll_device_status(lay) == (0, 0)
    # a FIFO ring is refused by the many-request call
    fifo = kvc.kvc_staging_ring_create(cb, 2, kvc.KVC_RING_HOST_MAPPED)
    with pytest.raises(kvc.KvcError) as e:
        kvc.kvc_pipeline_load_many(lay, fifo, store, reqs)
    assert e.value.status == kvc.KVC_ERR_STATE


def test_retained_chunks_serve_a_later_call_without_a_read(tmp_path):
    """Retention (the paper's optional DRAM cache inside the pool, Sec. 6.4): chunks of a finished
    load stay in their slots, so a second request with the same hashes is served without touching
    the files, until foreground work needs the slots."""
    g = orc.Dims(4, 2, 256, 16, 8, 128, 2)
    pool = wl.random_bits(703, g.pool_bytes)
    pool_t = torch.from_numpy(pool).to(DEV)
    lay = kvc.kvc_layout_create_dense(pool_t, g.L, g.P, g.NB, g.B, g.H, g.D, g.e, 256)
    cb = kvc.kvc_layout_chunk_bytes(lay, 16)
    store = kvc.kvc_store_open(str(tmp_path), "m", direct_io=True)
    perm = wl.block_ids(75, g.NB, g.NB)
    src, dst1, dst2, dst3 = (np.ascontiguousarray(perm[i * 48:(i + 1) * 48]) for i in range(4))
    hashes = _hashes(3, 3)
    fifo = kvc.kvc_staging_ring_create(cb, 2, kvc.KVC_RING_HOST_MAPPED)
    kvc.kvc_pipeline_store(lay, fifo, store, src, hashes)
    kvc.kvc_staging_ring_destroy(fifo)
    chunks = orc.pack_request(g, pool, src, 256)
    ring = kvc.kvc_staging_ring_create(cb, 4, kvc.KVC_RING_HOST_MAPPED)
    kvc.kvc_staging_ring_set_policy(ring, foreground_reserve=1, max_speculative=1, retain_completed=True)
    want_pool = pool.copy()
    s1, _ = kvc.kvc_pipeline_load_many(lay, ring, store, [dict(ids=dst1, hashes=hashes, cls=kvc.KVC_CLASS_DEMAND_LOAD)])
    torch.cuda.synchronize()
    orc.unpack_request(g, want_pool, chunks, dst1, 256)
    assert s1["reads"] == 3 and s1["joins"] == 0
    c = kvc.kvc_staging_ring_policy_counters(ring)
    assert (c["n_retained"], c["n_free"]) == (3, 1)
    reads0 = kvc.kvc_store_get_counters(store)["reads"]
    s2, _ = kvc.kvc_pipeline_load_many(lay, ring, store, [dict(ids=dst2, hashes=hashes, cls=kvc.KVC_CLASS_DEMAND_LOAD)])
    torch.cuda.synchronize()
    orc.unpack_request(g, want_pool, chunks, dst2, 256)
    assert s2["reads"] == 0 and s2["joins"] == 3 and s2["unpack_launches"] == 1
    assert kvc.kvc_store_get_counters(store)["reads"] == reads0
    assert np.array_equal(pool_t.cpu().numpy(), want_pool)
    # other work needs the slots: cached chunks give way, least recently used first
    other = _hashes(4, 3)
    kvc.kvc_pipeline_store(lay, ring, store, dst1, other)            # three stores through the same pool
    c = kvc.kvc_staging_ring_policy_counters(ring)
    assert c["reclaims"] >= 2
    s3, _ = kvc.kvc_pipeline_load_many(lay, ring, store, [dict(ids=dst3, hashes=hashes, cls=kvc.KVC_CLASS_DEMAND_LOAD)])
    torch.cuda.synchronize()
    orc.unpack_request(g, want_pool, chunks, dst3, 256)
    assert s3["reads"] >= 2                                          # evicted chunks are read again
    assert np.array_equal(pool_t.cpu().numpy(), want_pool)
    assert kvc.kvc_poll_device_status(lay) == (0, 0)


# ------------------------------------------------------------------ request <-> host buffer, one call each way
@pytest.mark.parametrize("ring_kind", [kvc.KVC_RING_DEVICE, kvc.KVC_RING_HOST_MAPPED, kvc.KVC_RING_DEVICE_STAGED])
@pytest.mark.parametrize("two_streams", [False, True])
def test_offload_to_host_and_load_back_match_the_oracle(ring_kind, two_streams):
    """kvc_offload_to_host / kvc_load_from_host: 139 blocks (8 chunks of 16 and one of 11) through
    a 3-slot ring into a pinned host buffer and back into other blocks, on one stream or on a kernel
    stream and a copy stream; host bytes and the pool against the oracle, twice in a row (the
    second pass reuses slots whose events the first pass recorded)."""
    g = orc.Dims(6, 2, 200, 16, 8, 128, 2)
    pool = wl.random_bits(760, g.pool_bytes)
    pool_t = torch.from_numpy(pool).to(DEV)
    lay = kvc.kvc_layout_create_dense(pool_t, g.L, g.P, g.NB, g.B, g.H, g.D, g.e, 256)
    src, dst = wl.block_ids(76, g.NB, 139), wl.block_ids(77, g.NB, 139)
    cb = kvc.kvc_layout_chunk_bytes(lay, 16)
    ring = kvc.kvc_staging_ring_create(cb, 3, ring_kind)
    total = 139 * g.bytes_per_block
    host = torch.full((total + 4096,), 0x5A, dtype=torch.uint8).pin_memory()
    s_k = torch.cuda.Stream()
    s_c = torch.cuda.Stream() if two_streams else None
    want_chunks = orc.pack_request(g, pool, src, 256)
    want_pool = pool.copy()
    orc.unpack_request(g, want_pool, want_chunks, dst, 256)
    for rep in range(2):
        host.fill_(0x5A)
        pool_t.copy_(torch.from_numpy(pool))
        torch.cuda.synchronize()
        st = kvc.kvc_offload_to_host(lay, ring, src, host, host_bytes=total, kernel_stream=s_k, copy_stream=s_c)
        assert (st["chunks"], st["total_chunks"], st["bytes"]) == (9, 9, total)
        (s_c or s_k).synchronize()
        h = host.numpy()
        assert np.array_equal(h[:total], np.concatenate(want_chunks)), "offload, pass %d" % rep
        assert (h[total:] == 0x5A).all()
        st = kvc.kvc_load_from_host(lay, ring, host, dst, host_bytes=total, kernel_stream=s_k, copy_stream=s_c)
        assert (st["chunks"], st["bytes"]) == (9, total)
        s_k.synchronize()
        assert np.array_equal(pool_t.cpu().numpy(), want_pool), "load, pass %d" % rep
    torch.cuda.synchronize()
    in_flight, acquires, _ = kvc.kvc_staging_ring_stats(ring)
    assert in_flight == 0 and acquires == 4 * 9
    assert kvc.kvc_poll_device_status(lay) == (0, 0)
    kvc.kvc_staging_ring_destroy(ring)


def test_host_transfers_accept_a_pageable_host_buffer():
    """Pinned memory is a matter of speed, not of correctness: the same round trip through an
    ordinary numpy array."""
    g = orc.Dims(3, 2, 80, 16, 4, 64, 2)
    pool = wl.random_bits(765, g.pool_bytes)
    pool_t = torch.from_numpy(pool).to(DEV)
    lay = kvc.kvc_layout_create_dense(pool_t, g.L, g.P, g.NB, g.B, g.H, g.D, g.e, 128)
    ring = kvc.kvc_staging_ring_create(kvc.kvc_layout_chunk_bytes(lay, 8), 2, kvc.KVC_RING_DEVICE)
    src, dst = wl.block_ids(79, g.NB, 53), wl.block_ids(80, g.NB, 53)
    host = np.full(53 * g.bytes_per_block + 64, 0x42, dtype=np.uint8)
    kvc.kvc_offload_to_host(lay, ring, src, host, host_bytes=53 * g.bytes_per_block)
    torch.cuda.synchronize()
    want_chunks = orc.pack_request(g, pool, src, 128)
    assert np.array_equal(host[:-64], np.concatenate(want_chunks)) and (host[-64:] == 0x42).all()
    kvc.kvc_load_from_host(lay, ring, host, dst, host_bytes=53 * g.bytes_per_block)
    torch.cuda.synchronize()
    want_pool = pool.copy()
    orc.unpack_request(g, want_pool, want_chunks, dst, 128)
    assert np.array_equal(pool_t.cpu().numpy(), want_pool)
    kvc.kvc_staging_ring_destroy(ring)


def test_host_transfer_error_exit_leaves_the_ring_usable():
    """A request whose last id is out of range is refused as a whole: nothing reaches the host
    buffer, no slot is taken, and the next transfer through the same ring works."""
    g = orc.Dims(2, 2, 64, 16, 4, 64, 2)
    pool = wl.random_bits(770, g.pool_bytes)
    pool_t = torch.from_numpy(pool).to(DEV)
    lay = kvc.kvc_layout_create_dense(pool_t, g.L, g.P, g.NB, g.B, g.H, g.D, g.e, 64)
    ring = kvc.kvc_staging_ring_create(kvc.kvc_layout_chunk_bytes(lay, 4), 2, kvc.KVC_RING_DEVICE)
    ids = wl.block_ids(78, g.NB, 30)
    bad = ids.copy()
    bad[-1] = g.NB
    total = 30 * g.bytes_per_block
    host = torch.full((total,), 0x11, dtype=torch.uint8).pin_memory()
    with pytest.raises(kvc.KvcError) as e:
        kvc.kvc_offload_to_host(lay, ring, bad, host)
    assert e.value.status == kvc.KVC_ERR_OUT_OF_RANGE
    torch.cuda.synchronize()
    assert bool((host == 0x11).all())
    assert kvc.kvc_staging_ring_stats(ring)[:2] == (0, 0)
    kvc.kvc_offload_to_host(lay, ring, ids, host)
    torch.cuda.synchronize()
    assert np.array_equal(host.numpy(), np.concatenate(orc.pack_request(g, pool, ids, 64)))
    kvc.kvc_staging_ring_destroy(ring)
