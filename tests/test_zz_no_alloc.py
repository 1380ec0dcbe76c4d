"""kvc_pack_batch_static -- the batched pack for callers that must not allocate.

A serving engine that has given all spare device memory to its KV pool, or a thread that may
not stall on an allocation, offloads blocks through this entry point: its id table lives in a
fixed array inside the library instead of memory allocated per call.  Here it is called through
the C ABI twice in a row (the second call is smaller, so stale table entries of the first are
still present behind it) and each result must equal, byte for byte, what the allocating
kvc_pack_batch produces for the same ops; then twice back to back on one stream with nothing
between the calls, against the CPU oracle.  This file is collected last on purpose."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")

from oracle import oracle as orc
from paper_2609_11744_b200 import kvc
import workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _ops(lay, ids, staging):
    ops, keep, nbytes, on_dev = kvc.request_chunk_ops(lay, ids, staging)
    assert on_dev == 0
    return ops, keep, nbytes


@pytest.mark.parametrize("separate_planes", [False, True])
def test_static_pack_matches_allocating_pack_twice_in_a_row(separate_planes):
    s = wl.LLAMA_8B
    L, NB = 6, 160                                   # 6 layers of the 8B shape, 160-block pool
    slab = s.slab_bytes
    plane_bytes = NB * slab
    pool = wl.random_bits_cuda(wl.BASE_SEED + 900, L * s.P * plane_bytes, DEV)
    if separate_planes:
        planes = [pool[i * plane_bytes:(i + 1) * plane_bytes] for i in range(L * s.P)]
        lay = kvc.kvc_layout_create(L, s.P, NB, s.B, s.H, s.D, s.e, 256, plane_ptrs=planes)
    else:
        lay = kvc.kvc_layout_create_dense(pool, L, s.P, NB, s.B, s.H, s.D, s.e, 256)
    bytes_per_block = L * s.P * slab
    for call, n in enumerate((120, 37)):             # second call: fewer blocks, ragged last chunk
        ids = wl.block_ids(wl.BASE_SEED + 901 + call, NB, n)
        want = torch.full((n * bytes_per_block + 4096,), 0x3C, dtype=torch.uint8, device=DEV)
        got = torch.full_like(want, 0x3C)
        ops_a, keep_a, nbytes = _ops(lay, ids, want)
        kvc.kvc_pack_batch(lay, ops_a, 0)
        ops_b, keep_b, _ = _ops(lay, ids, got)
        kvc.kvc_pack_batch_static(lay, ops_b)
        torch.cuda.synchronize()
        assert nbytes == n * bytes_per_block
        assert torch.equal(got, want), "call %d: static and allocating pack differ" % call
        assert bool((got[nbytes:] == 0x3C).all())
        assert bool((got[:nbytes] != 0x3C).any())
    assert kvc.kvc_poll_device_status(lay) == (0, 0)
    assert kvc.kvc_poll_static_status() == (0, 0)


@pytest.mark.parametrize("separate_planes", [False, True])
def test_two_static_packs_back_to_back_without_sync_match_the_oracle(separate_planes):
    """Two calls on ONE stream, different tables and sizes, nothing between them: the second call
    refills the host-side staging of the tables while the first call's kernels may not even have
    started.  Each result is compared with the CPU oracle (layer-major chunks)."""
    s = wl.LLAMA_8B
    g = orc.Dims(5, s.P, 144, s.B, s.H, s.D, s.e)
    pool = wl.random_bits(wl.BASE_SEED + 910, g.pool_bytes)
    pool_t = torch.from_numpy(pool).to(DEV)
    if separate_planes:
        pb = g.NB * g.slab_bytes
        lay = kvc.kvc_layout_create(g.L, g.P, g.NB, g.B, g.H, g.D, g.e, 256,
                                    plane_ptrs=[pool_t[i * pb:(i + 1) * pb] for i in range(g.L * g.P)])
    else:
        lay = kvc.kvc_layout_create_dense(pool_t, g.L, g.P, g.NB, g.B, g.H, g.D, g.e, 256)
    ids_a = wl.block_ids(wl.BASE_SEED + 911, g.NB, 131)   # 8 full chunks and one of 3 blocks
    ids_b = wl.block_ids(wl.BASE_SEED + 912, g.NB, 23)
    out_a = torch.full((131 * g.bytes_per_block + 4096,), 0xE1, dtype=torch.uint8, device=DEV)
    out_b = torch.full((23 * g.bytes_per_block + 4096,), 0xE2, dtype=torch.uint8, device=DEV)
    ops_a, keep_a, n_a = _ops(lay, ids_a, out_a)
    ops_b, keep_b, n_b = _ops(lay, ids_b, out_b)
    torch.cuda.synchronize()
    kvc.kvc_pack_batch_static(lay, ops_a)
    kvc.kvc_pack_batch_static(lay, ops_b)                 # no synchronisation in between
    torch.cuda.synchronize()
    for out, ids, n, fill in ((out_a, ids_a, n_a, 0xE1), (out_b, ids_b, n_b, 0xE2)):
        want = np.concatenate(orc.pack_request(g, pool, ids, 256))
        host = out.cpu().numpy()
        assert want.size == n
        assert np.array_equal(host[:n], want)
        assert (host[n:] == fill).all()
    assert kvc.kvc_poll_static_status() == (0, 0)
    assert kvc.kvc_poll_device_status(lay) == (0, 0)


def test_static_pack_rejects_what_it_cannot_hold():
    s = wl.TINY
    NB = kvc.KVC_STATIC_MAX_BLOCKS + 8
    g = orc.Dims(s.L, s.P, NB, s.B, s.H, s.D, s.e)
    pool_np = wl.random_bits(wl.BASE_SEED + 920, g.pool_bytes)
    pool = torch.from_numpy(pool_np).to(DEV)
    lay = kvc.kvc_layout_create_dense(pool, s.L, s.P, NB, s.B, s.H, s.D, s.e, 16 * NB)
    ids = np.arange(NB, dtype=np.int32)[::-1].copy()
    staging = torch.zeros(NB * s.bytes_per_block, dtype=torch.uint8, device=DEV)
    ops = kvc.make_chunk_ops([staging.data_ptr()], [ids.ctypes.data], [NB])
    with pytest.raises(kvc.KvcError) as e:
        kvc.kvc_pack_batch_static(lay, ops)
    assert e.value.status == kvc.KVC_ERR_TOO_LARGE
    bad = np.array([0, NB], dtype=np.int32)
    ops = kvc.make_chunk_ops([staging.data_ptr()], [bad.ctypes.data], [2])
    with pytest.raises(kvc.KvcError) as e:
        kvc.kvc_pack_batch_static(lay, ops)
    assert e.value.status == kvc.KVC_ERR_OUT_OF_RANGE
    torch.cuda.synchronize()
    assert bool((staging == 0).all())
    # exactly the maximum is accepted -- on a handle that has never launched anything, so the
    # static path also has to supply the device limits the planner needs; checked with the oracle
    n = kvc.KVC_STATIC_MAX_BLOCKS
    ops = kvc.make_chunk_ops([staging.data_ptr()], [ids.ctypes.data], [n])
    kvc.kvc_pack_batch_static(lay, ops)
    torch.cuda.synchronize()
    want = orc.pack_chunk(g, pool_np, ids[:n])
    host = staging.cpu().numpy()
    assert np.array_equal(host[:want.size], want)
    assert (host[want.size:] == 0).all()
    assert kvc.kvc_poll_static_status() == (0, 0)


def test_static_pack_of_thousands_of_small_chunks_with_empty_ops_between():
    """The table travels as chunk records plus ids and is expanded on the device; thousands of
    one-to-five-block chunks need several such launches, and empty ops sit between them and at
    both ends.  Every chunk against the oracle, the gaps between chunks untouched."""
    s = wl.TINY
    NB = 1500
    g = orc.Dims(s.L, s.P, NB, s.B, s.H, s.D, s.e)
    pool_np = wl.random_bits(wl.BASE_SEED + 930, g.pool_bytes)
    pool = torch.from_numpy(pool_np).to(DEV)
    lay = kvc.kvc_layout_create_dense(pool, s.L, s.P, NB, s.B, s.H, s.D, s.e, 16 * 8)
    rng = np.random.default_rng(wl.BASE_SEED + 931)
    sizes, total = [0], 0
    while total + 5 <= kvc.KVC_STATIC_MAX_BLOCKS - 3:
        n = int(rng.integers(1, 6)) if rng.random() > 0.05 else 0
        sizes.append(n)
        total += n
    sizes += [3, 0]
    total += 3
    assert sum(1 for n in sizes if n) > 2400
    stride = 5 * s.bytes_per_block + 64                    # a gap behind every chunk
    staging = torch.full((len(sizes) * stride,), 0x77, dtype=torch.uint8, device=DEV)
    ids = [rng.integers(0, NB, size=max(n, 1)).astype(np.int32) for n in sizes]   # repeats allowed
    ops = kvc.make_chunk_ops([staging.data_ptr() + i * stride for i in range(len(sizes))],
                             [a.ctypes.data for a in ids], sizes)
    kvc.kvc_pack_batch_static(lay, ops)
    torch.cuda.synchronize()
    host = staging.cpu().numpy()
    for i, n in enumerate(sizes):
        lo = i * stride
        if n:
            want = orc.pack_chunk(g, pool_np, ids[i][:n])
            assert np.array_equal(host[lo:lo + want.size], want), i
            lo += want.size
        assert (host[lo:(i + 1) * stride] == 0x77).all(), i
    assert kvc.kvc_poll_static_status() == (0, 0)
