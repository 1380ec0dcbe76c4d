"""Full-size GPU checks in the launch configuration the benchmark times (one batched pack and
one batched unpack of the whole prefix).  The pools are tens of GiB and live only on the device,
so the oracle is applied to sampled outputs, one element at a time: for every sample the oracle's
index formulas give the staging position and the pool positions, and the device values there must
agree.  Properties that hold at any size are checked on everything: the staged bytes equal the
gathered pool slabs, and pool blocks that were not named keep their contents."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")

from oracle import oracle as orc
from paper_2609_11744_b200 import kvc
import workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
N_SAMPLES = 300_000


def _sampled_positions(g, src, dst, bpc, seed):
    """Oracle positions (element indices) of N random chunk elements: in the staging area (chunks
    back to back), in the pool at the source block and in the pool at the destination block."""
    n = len(src)
    rng = np.random.default_rng(seed)
    blk = rng.integers(0, n, N_SAMPLES)
    c = blk // bpc
    j = blk - c * bpc
    nb_c = np.minimum(bpc, n - c * bpc)
    l, p = rng.integers(0, g.L, N_SAMPLES), rng.integers(0, g.P, N_SAMPLES)
    t, h, d = (rng.integers(0, k, N_SAMPLES) for k in (g.B, g.H, g.D))
    full_chunk_elems = orc.chunk_bytes(g, bpc) // g.e
    stage = c.astype(np.int64) * full_chunk_elems + orc.chunk_elem(g, nb_c, l, p, j, t, h, d)
    src_pos = orc.pool_elem(g, l, p, src[blk].astype(np.int64), t, h, d)
    dst_pos = orc.pool_elem(g, l, p, dst[blk].astype(np.int64), t, h, d)
    return blk, stage, src_pos, dst_pos


def _full_size_case(w, chunk_tokens, n_free_check=64):
    s = w.shape
    NB, n = w.pool_blocks, w.request_blocks
    free, _ = torch.cuda.mem_get_info()
    need = NB * s.bytes_per_block + 3 * n * s.bytes_per_block + (2 << 30)
    if free < need:
        pytest.skip("needs %.1f GiB of free device memory" % (need / 2**30))
    g = orc.Dims(s.L, s.P, NB, s.B, s.H, s.D, s.e)
    bpc = chunk_tokens // s.B
    pool = wl.random_bits_cuda(w.seed, NB * s.bytes_per_block, DEV)
    src = wl.block_ids(w.seed, NB, n)
    dst = wl.block_ids(w.dst_seed, NB, n)
    one_way = n * s.bytes_per_block
    staging = torch.full((one_way + 4096,), 0x77, dtype=torch.uint8, device=DEV)
    lay = kvc.kvc_layout_create_dense(pool, s.L, s.P, NB, s.B, s.H, s.D, s.e, chunk_tokens)
    assert kvc.kvc_layout_num_chunks(lay, n) == len(orc.chunk_ranges(n, bpc))
    # element-typed views: the oracle's positions are in elements of s.e bytes
    elem_t = {1: torch.uint8, 2: torch.int16, 4: torch.int32}[s.e]
    pool16, stage16 = pool.view(elem_t), staging[:one_way].view(elem_t)
    assert pool16.numel() == g.pool_bytes // g.e
    blk, stage_pos, src_pos, dst_pos = _sampled_positions(g, src, dst, bpc, w.seed)
    # positions are checked here, on the host, before any of them indexes a device tensor
    assert 0 <= stage_pos.min() and stage_pos.max() < stage16.numel()
    assert 0 <= min(src_pos.min(), dst_pos.min()) and max(src_pos.max(), dst_pos.max()) < pool16.numel()
    dev_idx = lambda a: torch.from_numpy(a).to(DEV)

    # ---- pack: one launch
    ops, keep, nbytes, on_dev = kvc.request_chunk_ops(lay, src, staging)
    assert nbytes == one_way
    kvc.kvc_pack_batch(lay, ops, on_dev)
    torch.cuda.synchronize()
    assert torch.equal(stage16[dev_idx(stage_pos)], pool16[dev_idx(src_pos)]), "pack: sampled elements"
    assert bool((staging[one_way:] == 0x77).all()), "pack wrote past the last chunk"
    # property at full size: every chunk equals the pool slabs gathered along the block axis
    pool4 = pool.view(s.L * s.P, NB, s.slab_bytes)
    off = 0
    for first, nb in orc.chunk_ranges(n, bpc)[:: max(1, len(orc.chunk_ranges(n, bpc)) // 24)]:
        off = first * s.bytes_per_block
        ids_t = dev_idx(src[first:first + nb].astype(np.int64))
        want = pool4[:, ids_t].reshape(-1)
        assert torch.equal(staging[off:off + want.numel()], want), "pack: chunk at entry %d" % first

    # ---- unpack: one launch into the second table
    untouched = np.setdiff1d(np.arange(NB), dst)[:n_free_check]
    before = pool4[:, dev_idx(untouched.astype(np.int64))].clone()
    ops2, keep2, _, _ = kvc.request_chunk_ops(lay, dst, staging)
    kvc.kvc_unpack_batch(lay, ops2, on_dev)
    torch.cuda.synchronize()
    assert torch.equal(pool16[dev_idx(dst_pos)], stage16[dev_idx(stage_pos)]), "unpack: sampled elements"
    assert torch.equal(pool4[:, dev_idx(untouched.astype(np.int64))], before), "unpack touched other blocks"
    assert kvc.kvc_poll_device_status(lay) == (0, 0)
    assert kvc.kvc_layout_launch_count(lay) == 2


def test_config2_8b_8k_prefix():
    _full_size_case(wl.WORKLOADS["8b_8k"], 256)


@pytest.mark.parametrize("chunk_tokens", [256, 16, 2048])
def test_config3_8b_80k_prefix(chunk_tokens):
    _full_size_case(wl.WORKLOADS["8b_80k"], chunk_tokens)


def test_config4_70b_batch_one_call_unpack():
    """64 requests (lognormal lengths, shared 1024-token prefix), 70B-class shape, every kept chunk
    unpacked by ONE kvc_unpack_batch call, at full size; sampled elements against the oracle's
    index formulas, plus whole-block equality for a few hundred blocks."""
    w = wl.WORKLOADS["70b_batch"]
    s = w.shape
    NB, tables = wl.batch_workload(w, 1.0)
    lay_probe = kvc.kvc_layout_create_dense(0x100000, s.L, s.P, NB, s.B, s.H, s.D, s.e, 256)
    descs, uniq = kvc.kvc_map_requests_shared(lay_probe, tables)
    total = sum(d[4] for d in descs)
    free, _ = torch.cuda.mem_get_info()
    if free < NB * s.bytes_per_block + total + (4 << 30):
        pytest.skip("needs %.0f GiB of free device memory" % ((NB * s.bytes_per_block + total) / 2**30))
    g = orc.Dims(s.L, s.P, NB, s.B, s.H, s.D, s.e)
    pool = torch.zeros(NB * s.bytes_per_block, dtype=torch.uint8, device=DEV)
    staging = wl.random_bits_cuda(w.seed + 3, total, DEV)
    lay = kvc.kvc_layout_create_dense(pool, s.L, s.P, NB, s.B, s.H, s.D, s.e, 256)
    slot, ids, nbs, offs, off = [], [], [], [], 0
    for (r, c, first, nb, nbytes) in descs:
        slot.append(staging.data_ptr() + off)
        ids.append(tables[r].ctypes.data + 4 * first)
        nbs.append(nb)
        offs.append(off)
        off += nbytes
    kvc.kvc_unpack_batch(lay, kvc.make_chunk_ops(slot, ids, nbs), 0)
    torch.cuda.synchronize()
    assert kvc.kvc_layout_launch_count(lay) == 1 and kvc.kvc_poll_device_status(lay) == (0, 0)
    # sampled elements: op k, block j of it, coordinates (l, p, t, h, d)
    rng = np.random.default_rng(4)
    k = rng.integers(0, len(descs), N_SAMPLES)
    nb_c = np.array(nbs)[k]
    j = (rng.random(N_SAMPLES) * nb_c).astype(np.int64)
    l, p = rng.integers(0, g.L, N_SAMPLES), rng.integers(0, g.P, N_SAMPLES)
    t, h, d = (rng.integers(0, q, N_SAMPLES) for q in (g.B, g.H, g.D))
    first = np.array([dd[2] for dd in descs])[k]
    req = np.array([dd[0] for dd in descs])[k]
    flat_tables = np.concatenate(tables)
    starts = np.concatenate([[0], np.cumsum([len(t_) for t_ in tables])[:-1]])
    blk = flat_tables[starts[req] + first + j].astype(np.int64)
    stage_pos = np.array(offs, dtype=np.int64)[k] // g.e + orc.chunk_elem(g, nb_c, l, p, j, t, h, d)
    pool_pos = orc.pool_elem(g, l, p, blk, t, h, d)
    dev_idx = lambda a: torch.from_numpy(a).to(DEV)
    assert torch.equal(pool.view(torch.int16)[dev_idx(pool_pos)],
                       staging.view(torch.int16)[dev_idx(stage_pos)])
    # blocks of no request stay zero; a few hundred written blocks are compared in full
    named = np.unique(flat_tables)
    assert len(named) == uniq
    untouched = np.setdiff1d(np.arange(NB), named)[:128]
    pool4 = pool.view(s.L * s.P, NB, s.slab_bytes)
    assert bool((pool4[:, dev_idx(untouched.astype(np.int64))] == 0).all())
    for kk in rng.integers(0, len(descs), 12):
        (r, c, f, nb, nbytes) = descs[kk]
        chunk = staging[offs[kk]:offs[kk] + nbytes].view(s.L * s.P, nb, s.slab_bytes)
        ids_t = dev_idx(tables[r][f:f + nb].astype(np.int64))
        assert torch.equal(pool4[:, ids_t], chunk)


def test_config5_32k_prefix_streamed_through_8_slot_ring_to_host():
    """The 32k-token prefix (4 GiB) of the ring config streamed through 8 slots x 256 tokens into
    pinned host memory: sampled host elements against the oracle's positions in the device pool."""
    w = wl.WORKLOADS["8b_ring"]
    s = w.shape
    NB, n = w.pool_blocks, w.request_blocks
    g = orc.Dims(s.L, s.P, NB, s.B, s.H, s.D, s.e)
    from paper_2609_11744_b200 import cuda_rt
    pool = wl.random_bits_cuda(w.seed, NB * s.bytes_per_block, DEV)
    src = wl.block_ids(w.seed, NB, n)
    lay = kvc.kvc_layout_create_dense(pool, s.L, s.P, NB, s.B, s.H, s.D, s.e, 256)
    descs = kvc.kvc_map_request(lay, n)
    assert len(descs) == 128
    cb = kvc.kvc_layout_chunk_bytes(lay, 16)
    ring = kvc.kvc_staging_ring_create(cb, int(w.extra["ring_slots"]), kvc.KVC_RING_DEVICE)
    host = torch.empty(n * s.bytes_per_block, dtype=torch.uint8, pin_memory=True)
    s_k, s_c = torch.cuda.Stream(), torch.cuda.Stream()
    off = 0
    for (_, c, first, nb, nbytes) in descs:
        slot, dptr, _ = kvc.kvc_staging_ring_acquire(ring, 10_000_000)
        assert slot == c % 8
        kvc.kvc_pack(lay, src[first:first + nb], dptr, nbytes, stream=s_k)
        kvc.kvc_staging_ring_commit(ring, slot, s_k)
        kvc.kvc_staging_ring_wait_filled(ring, slot, s_c)
        cuda_rt.memcpy_async(host.data_ptr() + off, dptr, nbytes, cuda_rt.D2H, s_c)
        kvc.kvc_staging_ring_release(ring, slot, s_c)
        off += nbytes
    torch.cuda.synchronize()
    assert kvc.kvc_staging_ring_stats(ring)[1] == 128            # 16 laps of the 8-slot ring
    blk, stage_pos, src_pos, _ = _sampled_positions(g, src, src, 16, w.seed)
    want = pool.view(torch.int16)[torch.from_numpy(src_pos).to(DEV)].cpu()
    got = host.view(torch.int16)[torch.from_numpy(stage_pos)]
    assert torch.equal(got, want)
    kvc.kvc_staging_ring_destroy(ring)


@pytest.mark.parametrize("elem_bytes", [2, 1])
def test_tensor_parallel_shard_of_the_80k_prefix(elem_bytes):
    """The 80k-token prefix as ONE GPU of an 8-way tensor-parallel 8B model sees it: one KV head per
    GPU, so 4 KiB slabs (2 KiB with 1-byte elements) -- the shapes the multi-slab kernels exist for.
    Sampled elements at the oracle's positions over the 20,000-block pool, whole chunks, untouched
    blocks; launch configuration as in the benchmark (one batched call per direction)."""
    shape = wl.KVShape(L=32, P=2, B=16, H=1, D=128, e=elem_bytes)
    w = wl.Workload("8b_80k_tp8", 5 + elem_bytes, shape, 20000, 80000, (256,))
    _full_size_case(w, 256)


def test_tensor_parallel_shard_whole_prefix_against_the_oracle_loops():
    """The same shard shape with every byte compared: 5000 blocks (1.22 GiB) out of a 6000-block
    pool, the oracle's plain loops run over (layer, K|V) ranges on the host cores."""
    from concurrent.futures import ThreadPoolExecutor
    shape = wl.KVShape(L=32, P=2, B=16, H=1, D=128, e=2)
    NB, n, bpc = 6000, 5000, 16
    g = orc.Dims(shape.L, shape.P, NB, shape.B, shape.H, shape.D, shape.e)
    pool = wl.random_bits(wl.BASE_SEED + 77, g.pool_bytes)
    src, dst = wl.block_ids(wl.BASE_SEED + 78, NB, n), wl.block_ids(wl.BASE_SEED + 79, NB, n)
    pool_t = torch.from_numpy(pool).to(DEV)
    lay = kvc.kvc_layout_create_dense(pool_t, g.L, g.P, NB, g.B, g.H, g.D, g.e, 256)
    one_way = n * g.bytes_per_block
    staging = torch.full((one_way + 4096,), 0x77, dtype=torch.uint8, device=DEV)
    ops, keep, nbytes, on_dev = kvc.request_chunk_ops(lay, src, staging)
    kvc.kvc_pack_batch(lay, ops, on_dev)
    ops2, keep2, _, _ = kvc.request_chunk_ops(lay, dst, staging)
    kvc.kvc_unpack_batch(lay, ops2, on_dev)
    torch.cuda.synchronize()
    ranges = orc.chunk_ranges(n, bpc)
    want = np.zeros(one_way, dtype=np.uint8)
    want_pool = pool.copy()
    lp = g.L * g.P
    cuts = [(a, min(lp, a + 8)) for a in range(0, lp, 8)]

    def pack_part(r):
        for first, nb in ranges:
            lo = first * g.bytes_per_block
            orc.pack_chunk_into(g, pool, src[first:first + nb], want[lo:lo + nb * g.bytes_per_block], r)

    def unpack_part(r):
        for first, nb in ranges:
            lo = first * g.bytes_per_block
            orc.unpack_chunk(g, want_pool, want[lo:lo + nb * g.bytes_per_block], dst[first:first + nb], r)

    with ThreadPoolExecutor(len(cuts)) as ex:
        list(ex.map(pack_part, cuts))
        list(ex.map(unpack_part, cuts))
    host = staging.cpu().numpy()
    assert np.array_equal(host[:one_way], want), "pack"
    assert (host[one_way:] == 0x77).all()
    assert np.array_equal(pool_t.cpu().numpy(), want_pool), "unpack"
    assert kvc.kvc_poll_device_status(lay) == (0, 0)
