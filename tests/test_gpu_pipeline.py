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


@pytest.mark.parametrize("use_copy_engine", [False, True])
def test_store_then_load_through_files(tmp_path, use_copy_engine):
    g = orc.Dims(6, 2, 96, 16, 8, 128, 2)            # 8B shape cut to 6 layers; chunk = 6 MiB
    pool = wl.random_bits(700, g.pool_bytes)
    pool_t = torch.from_numpy(pool).to(DEV)
    lay = kvc.kvc_layout_create_dense(pool_t, g.L, g.P, g.NB, g.B, g.H, g.D, g.e, 256)
    src, dst = wl.block_ids(71, g.NB, 44), wl.block_ids(72, g.NB, 44)     # 2 full chunks + 12 blocks
    cb = kvc.kvc_layout_chunk_bytes(lay, 16)
    ring = kvc.kvc_staging_ring_create(cb, 2, kvc.KVC_RING_HOST_MAPPED)    # request > ring
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
