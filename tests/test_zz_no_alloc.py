"""kvc_pack_batch_static -- the batched pack for callers that must not allocate.

A serving engine that has given all spare device memory to its KV pool, or a thread that may
not stall on an allocation, offloads blocks through this entry point: its id table lives in a
fixed array inside the library instead of memory allocated per call.  Here it is called through
the C ABI twice in a row (the second call is smaller, so stale table entries of the first are
still present behind it) and each result must equal, byte for byte, what the allocating
kvc_pack_batch produces for the same ops.  This file is collected last on purpose."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")

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


def test_static_pack_rejects_what_it_cannot_hold():
    s = wl.TINY
    NB = kvc.KVC_STATIC_MAX_BLOCKS + 8
    pool = torch.zeros(s.L * s.P * NB * s.slab_bytes, dtype=torch.uint8, device=DEV)
    lay = kvc.kvc_layout_create_dense(pool, s.L, s.P, NB, s.B, s.H, s.D, s.e, 16 * NB)
    ids = np.arange(NB, dtype=np.int32)
    staging = torch.zeros(NB * s.bytes_per_block, dtype=torch.uint8, device=DEV)
    ops = kvc.make_chunk_ops([staging.data_ptr()], [ids.ctypes.data], [NB])
    with pytest.raises(kvc.KvcError) as e:
        kvc.kvc_pack_batch_static(lay, ops)
    assert e.value.status == kvc.KVC_ERR_TOO_LARGE
    ops = kvc.make_chunk_ops([staging.data_ptr()], [ids.ctypes.data], [kvc.KVC_STATIC_MAX_BLOCKS])
    kvc.kvc_pack_batch_static(lay, ops)               # exactly the maximum is accepted
    bad = np.array([0, NB], dtype=np.int32)
    ops = kvc.make_chunk_ops([staging.data_ptr()], [bad.ctypes.data], [2])
    with pytest.raises(kvc.KvcError) as e:
        kvc.kvc_pack_batch_static(lay, ops)
    assert e.value.status == kvc.KVC_ERR_OUT_OF_RANGE
    torch.cuda.synchronize()
    assert bool((staging == 0).all())
