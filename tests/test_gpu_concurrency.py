"""Pack / unpack beside other GPU work: the regime of Sec. 2.3 (stores deferred so that they
overlap the next forward pass) and Sec. 5.1 (a kernel copy shares the GPU with the model).
Default launches carry the programmatic-dependent-launch attribute and run on high-priority
streams here while a low-priority stream keeps the tensor cores busy; every byte is then compared
with the CPU oracle.  Also: kernels of one stream that read what the previous one wrote, and host
threads whose handles make their first launches at the same moment."""
import threading

import numpy as np
import pytest

torch = pytest.importorskip("torch")

from oracle import oracle as orc
from paper_2609_11744_b200 import cuda_rt, kvc
import workloads as wl
from test_gpu_parity import DEV, _pool_8b_384, dense_layout, dims_of, to_dev

pytestmark = pytest.mark.gpu


class _GemmLoad:
    """A bf16 matmul loop on a low-priority stream.  burst() enqueues about `seconds` of it (few
    enough launches that the host is not held up enqueueing them) and returns a 'done' event."""

    def __init__(self, stream, seconds=0.15):
        N = 8192
        self.stream = stream
        with torch.cuda.stream(stream):
            self.a = torch.randn(N, N, device=DEV, dtype=torch.bfloat16)
            self.b = torch.randn(N, N, device=DEV, dtype=torch.bfloat16)
            self.c = torch.empty(N, N, device=DEV, dtype=torch.bfloat16)
            for _ in range(3):      # library set-up and kernel selection happen on the first calls
                torch.matmul(self.a, self.b, out=self.c)
            stream.synchronize()
            t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            t0.record(stream)
            for _ in range(20):
                torch.matmul(self.a, self.b, out=self.c)
            t1.record(stream)
            t1.synchronize()
        self.iters = int(min(400, max(20, seconds * 1e3 / (t0.elapsed_time(t1) / 20))))

    def burst(self):
        with torch.cuda.stream(self.stream):
            for _ in range(self.iters):
                torch.matmul(self.a, self.b, out=self.c)
            done = torch.cuda.Event()
            done.record(self.stream)
        return done


@pytest.mark.parametrize("kind", [kvc.KVC_RING_DEVICE, kvc.KVC_RING_HOST_MAPPED])
@pytest.mark.parametrize("variant", [kvc.KVC_VARIANT_AUTO, kvc.KVC_VARIANT_VEC, "beside-compute preset"])
def test_ring_streaming_stays_exact_beside_a_compute_stream(kind, variant):
    """A 2048-token prefix (8 chunks) through a 3-slot ring, offload then load, on high-priority
    streams with default (programmatic dependent) launches, while a low-priority stream runs a
    matmul loop for the whole time."""
    w = wl.WORKLOADS["8b_ring"]
    g = dims_of(w.shape, 384)
    pool = _pool_8b_384()
    pool_t = to_dev(pool)
    lay = dense_layout(pool_t, g, 256)
    if isinstance(variant, str):
        kvc.kvc_layout_set_tuning(lay, **kvc.kvc_tuning_preset(kvc.KVC_PRESET_BESIDE_COMPUTE))
    else:
        kvc.kvc_layout_set_tuning(lay, variant=variant)
    src = wl.block_ids(w.seed, g.NB, 128)
    dst = wl.block_ids(w.dst_seed, g.NB, 128)
    descs = kvc.kvc_map_request(lay, len(src))
    cb = kvc.kvc_layout_chunk_bytes(lay, 16)
    ring = kvc.kvc_staging_ring_create(cb, 3, kind)
    host_out = torch.empty(len(descs) * cb, dtype=torch.uint8).pin_memory()
    lo, hi = torch.cuda.Stream.priority_range()
    s_gemm = torch.cuda.Stream(priority=lo)
    s_k, s_c = torch.cuda.Stream(priority=hi), torch.cuda.Stream(priority=hi)
    want_chunks = orc.pack_request(g, pool, src, 256)
    want_pool = pool.copy()
    orc.unpack_request(g, want_pool, want_chunks, dst, 256)
    gemm = _GemmLoad(s_gemm)
    torch.cuda.synchronize()
    overlapped = 0
    for rep in range(4):
        pool_t.copy_(torch.from_numpy(pool))
        torch.cuda.synchronize()
        gemm_done = gemm.burst()    # ~150 ms of matmuls; the 8 chunks below take ~10 ms
        for (_, c, first, nb, nbytes) in descs:
            slot, dptr, hptr = kvc.kvc_staging_ring_acquire(ring, timeout_us=10_000_000)
            kvc.kvc_pack(lay, src[first:first + nb], dptr, cb, stream=s_k)
            kvc.kvc_staging_ring_commit(ring, slot, s_k)
            kvc.kvc_staging_ring_wait_filled(ring, slot, s_c)
            if kind == kvc.KVC_RING_DEVICE:
                cuda_rt.memcpy_async(host_out.data_ptr() + c * cb, dptr, nbytes, cuda_rt.D2H, s_c)
            else:
                cuda_rt.memcpy_async(host_out.data_ptr() + c * cb, hptr, nbytes, cuda_rt.H2H, s_c)
            kvc.kvc_staging_ring_release(ring, slot, s_c)
        s_c.synchronize()
        overlapped += not gemm_done.query()
        assert np.array_equal(host_out.numpy(), np.concatenate(want_chunks)), "offload pass %d" % rep
        torch.cuda.synchronize()
        gemm_done = gemm.burst()
        for (_, c, first, nb, nbytes) in descs:
            slot, dptr, hptr = kvc.kvc_staging_ring_acquire(ring, timeout_us=10_000_000)
            if kind == kvc.KVC_RING_DEVICE:
                cuda_rt.memcpy_async(dptr, host_out.data_ptr() + c * cb, nbytes, cuda_rt.H2D, s_c)
            else:
                cuda_rt.memcpy_async(hptr, host_out.data_ptr() + c * cb, nbytes, cuda_rt.H2H, s_c)
            kvc.kvc_staging_ring_commit(ring, slot, s_c)
            kvc.kvc_staging_ring_wait_filled(ring, slot, s_k)
            kvc.kvc_unpack(lay, dptr, dst[first:first + nb], cb, stream=s_k)
            kvc.kvc_staging_ring_release(ring, slot, s_k)
        s_k.synchronize()
        overlapped += not gemm_done.query()
        assert np.array_equal(pool_t.cpu().numpy(), want_pool), "load pass %d" % rep
    assert overlapped >= 6, "the matmul bursts ended before the transfers that should run beside them"
    torch.cuda.synchronize()
    kvc.kvc_staging_ring_destroy(ring)
    assert kvc.kvc_poll_device_status(lay) == (0, 0)


@pytest.mark.parametrize("variant", [kvc.KVC_VARIANT_VEC, kvc.KVC_VARIANT_BULK])
def test_pack_right_after_unpack_on_one_stream_sees_the_new_data(variant):
    """unpack(new chunk) -> pack of the same blocks, alternating many times on one stream with
    programmatic dependent launch: the pack grid may be resident while the unpack grid still
    writes the pool, and must read the written bytes, never stale ones."""
    g = orc.Dims(4, 2, 64, 16, 8, 128, 2)
    pool = wl.random_bits(2024, g.pool_bytes)
    pool_t = to_dev(pool)
    lay = dense_layout(pool_t, g, 16 * g.B)
    kvc.kvc_layout_set_tuning(lay, variant=variant, pdl=2)
    ids = wl.block_ids(5, g.NB, 16)
    cb = kvc.kvc_layout_chunk_bytes(lay, 16)
    reps = 24
    fresh = [to_dev(wl.random_bits(3000 + i, cb)) for i in range(reps)]
    outs = [torch.zeros(cb, dtype=torch.uint8, device=DEV) for _ in range(reps)]
    torch.cuda.synchronize()
    for i in range(reps):
        kvc.kvc_unpack(lay, fresh[i], ids)
        kvc.kvc_pack(lay, ids, outs[i])
    torch.cuda.synchronize()
    for i in range(reps):
        # pack(unpack(chunk)) of the same ids is the chunk itself (round-trip identity of the oracle)
        assert torch.equal(outs[i], fresh[i]), "round %d read stale pool bytes" % i
    want_pool = pool.copy()
    orc.unpack_chunk(g, want_pool, fresh[-1].cpu().numpy(), ids)
    assert np.array_equal(pool_t.cpu().numpy(), want_pool)
    assert kvc.kvc_poll_device_status(lay) == (0, 0)


def test_first_launches_of_two_handles_race_on_two_threads():
    """Two host threads, each with its own handle and a different shared-memory footprint, make
    their first bulk launches at the same time (the opt-in shared-memory size of a kernel is
    process-wide state).  Both must succeed and be exact; repeated with fresh handles."""
    g = orc.Dims(2, 2, 48, 16, 8, 128, 2)
    pool = wl.random_bits(77, g.pool_bytes)
    ids = wl.block_ids(6, g.NB, 20)
    want = np.concatenate(orc.pack_request(g, pool, ids, 64))
    pool_t = to_dev(pool)
    tunings = [dict(max_ctas=8, stages=2), dict(max_ctas=8, stages=6), dict(stages=3, group=kvc.KVC_GROUP_FORCE_KERNEL),
               dict(max_ctas=4, stages=5, group=kvc.KVC_GROUP_FORCE_KERNEL)]
    errors = []

    def worker(tuning, barrier, out):
        try:
            torch.cuda.set_device(0)
            st = torch.cuda.Stream()
            lay = dense_layout(pool_t, g, 64)
            kvc.kvc_layout_set_tuning(lay, variant=kvc.KVC_VARIANT_BULK, **tuning)
            ops, keep, nbytes, dev = kvc.request_chunk_ops(lay, ids, out)
            barrier.wait()
            for _ in range(5):
                kvc.kvc_pack_batch(lay, ops, dev, stream=st)
            st.synchronize()
            assert kvc.kvc_poll_device_status(lay, stream=st) == (0, 0)
        except Exception as e:  # reported by the main thread
            errors.append(repr(e))

    for rnd in range(3):
        outs = [torch.zeros(want.size, dtype=torch.uint8, device=DEV) for _ in tunings]
        barrier = threading.Barrier(len(tunings))
        ts = [threading.Thread(target=worker, args=(t, barrier, o)) for t, o in zip(tunings, outs)]
        for t in ts:
            t.start()
        for t in ts:
            t.join(timeout=120)
        assert errors == []
        torch.cuda.synchronize()
        for o in outs:
            assert np.array_equal(o.cpu().numpy(), want)


@pytest.mark.parametrize("kind", [kvc.KVC_RING_DEVICE, kvc.KVC_RING_HOST_MAPPED])
def test_offload_and_load_share_one_staging_pool_at_the_same_time(kind):
    """Sec. 6.4: loads and stores draw from the same pool.  Request A is offloaded (pack -> slot ->
    host) while request B is loaded (host -> slot -> unpack) through ONE 4-slot pool, chunk by
    chunk in alternation, each direction on its own pair of streams.  Host bytes of A and the
    blocks of B must equal the oracle's."""
    w = wl.WORKLOADS["8b_ring"]
    g = dims_of(w.shape, 384)
    pool = _pool_8b_384()
    pool_t = to_dev(pool)
    lay = dense_layout(pool_t, g, 256)
    ids_a = wl.block_ids(31, g.NB, 150)                     # offloaded: 9 full chunks + 6 blocks
    perm = wl.block_ids(32, g.NB, g.NB)
    rest = np.array([b for b in perm if b not in set(ids_a.tolist())], dtype=np.int32)
    ids_b = np.ascontiguousarray(rest[:120])                # loaded into blocks A does not read
    src_b = wl.block_ids(33, g.NB, 120)                     # what B's chunks hold (packed by the oracle)
    chunks_b = orc.pack_request(g, pool, src_b, 256)
    host_b = torch.from_numpy(np.concatenate(chunks_b)).pin_memory()
    want_a = np.concatenate(orc.pack_request(g, pool, ids_a, 256))
    want_pool = pool.copy()
    orc.unpack_request(g, want_pool, chunks_b, ids_b, 256)
    host_a = torch.zeros(want_a.size, dtype=torch.uint8).pin_memory()
    cb = kvc.kvc_layout_chunk_bytes(lay, 16)
    ring = kvc.kvc_staging_ring_create(cb, 4, kind)
    kvc.kvc_staging_ring_set_policy(ring, foreground_reserve=0)
    s_pack, s_d2h, s_h2d, s_unpack = (torch.cuda.Stream() for _ in range(4))
    da, db = kvc.kvc_map_request(lay, len(ids_a)), kvc.kvc_map_request(lay, len(ids_b))
    TO = 10_000_000
    off_a = off_b = 0
    for i in range(max(len(da), len(db))):
        if i < len(da):
            _, c, first, nb, nbytes = da[i]
            slot, dptr, hptr, joined = kvc.kvc_staging_ring_acquire_for(ring, kvc.KVC_CLASS_STORE, 1000 + c, TO)
            assert not joined
            kvc.kvc_pack(lay, ids_a[first:first + nb], dptr, nbytes, stream=s_pack)
            kvc.kvc_staging_ring_commit(ring, slot, s_pack)
            kvc.kvc_staging_ring_wait_filled(ring, slot, s_d2h)
            if kind == kvc.KVC_RING_DEVICE:
                cuda_rt.memcpy_async(host_a.data_ptr() + off_a, dptr, nbytes, cuda_rt.D2H, s_d2h)
            else:
                cuda_rt.memcpy_async(host_a.data_ptr() + off_a, hptr, nbytes, cuda_rt.H2H, s_d2h)
            kvc.kvc_staging_ring_release(ring, slot, s_d2h)
            off_a += nbytes
        if i < len(db):
            _, c, first, nb, nbytes = db[i]
            slot, dptr, hptr, joined = kvc.kvc_staging_ring_acquire_for(ring, kvc.KVC_CLASS_DEMAND_LOAD,
                                                                        2000 + c, TO)
            assert not joined
            if kind == kvc.KVC_RING_DEVICE:
                cuda_rt.memcpy_async(dptr, host_b.data_ptr() + off_b, nbytes, cuda_rt.H2D, s_h2d)
            else:
                cuda_rt.memcpy_async(hptr, host_b.data_ptr() + off_b, nbytes, cuda_rt.H2H, s_h2d)
            kvc.kvc_staging_ring_commit(ring, slot, s_h2d)
            kvc.kvc_staging_ring_wait_filled(ring, slot, s_unpack)
            kvc.kvc_unpack(lay, dptr, ids_b[first:first + nb], nbytes, stream=s_unpack)
            kvc.kvc_staging_ring_release(ring, slot, s_unpack)
            off_b += nbytes
    torch.cuda.synchronize()
    assert np.array_equal(host_a.numpy(), want_a)
    assert np.array_equal(pool_t.cpu().numpy(), want_pool)
    c = kvc.kvc_staging_ring_policy_counters(ring)
    assert (c["n_free"], c["acquires"]) == (4, len(da) + len(db))
    kvc.kvc_staging_ring_destroy(ring)
    assert kvc.kvc_poll_device_status(lay) == (0, 0)


@pytest.mark.parametrize("variant", [kvc.KVC_VARIANT_BULK, kvc.KVC_VARIANT_VEC])
def test_independent_launches_may_overlap_and_stay_exact(variant):
    """pdl = 3: consecutive per-chunk calls on one stream whose kernels do not depend on each other
    (the chunks of a request packed into different places; then unpacked into different blocks)
    skip the wait for the previous kernel.  Many small chunks, so that kernels really run beside
    their predecessors' last blocks; bytes against the oracle."""
    g = orc.Dims(8, 2, 600, 16, 8, 128, 2)
    pool = wl.random_bits(4242, g.pool_bytes)
    pool_t = to_dev(pool)
    lay = dense_layout(pool_t, g, 32)                     # chunks of 2 blocks: 1 MiB each
    kvc.kvc_layout_set_tuning(lay, variant=variant, pdl=3, slot_memory=1)
    src, dst = wl.block_ids(41, g.NB, 301), wl.block_ids(42, g.NB, 301)
    descs = kvc.kvc_map_request(lay, len(src))
    total = sum(d[4] for d in descs)
    staging = torch.full((total + 4096,), 0x3E, dtype=torch.uint8, device=DEV)
    want_chunks = orc.pack_request(g, pool, src, 32)
    want_pool = pool.copy()
    orc.unpack_request(g, want_pool, want_chunks, dst, 32)
    torch.cuda.synchronize()
    for rep in range(3):
        staging.fill_(0x3E)
        pool_t.copy_(torch.from_numpy(pool))
        torch.cuda.synchronize()
        off = 0
        for (_, _, first, nb, nbytes) in descs:
            kvc.kvc_pack(lay, src[first:first + nb], staging[off:off + nbytes])
            off += nbytes
        done = torch.cuda.Event()
        done.record()                                      # an event after the calls covers all of them
        done.synchronize()
        host = staging.cpu().numpy()
        assert np.array_equal(host[:total], np.concatenate(want_chunks)), "pack, pass %d" % rep
        assert (host[total:] == 0x3E).all()
        off = 0
        for (_, _, first, nb, nbytes) in descs:
            kvc.kvc_unpack(lay, staging[off:off + nbytes], dst[first:first + nb])
            off += nbytes
        torch.cuda.synchronize()
        assert np.array_equal(pool_t.cpu().numpy(), want_pool), "unpack, pass %d" % rep
    assert kvc.kvc_poll_device_status(lay) == (0, 0)
