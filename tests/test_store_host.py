"""Chunk files behind the ring (host only): hash-addressed paths, first-writer-wins publication
through a temporary file and a hard link, complete-or-absent reads (Sec. 6.3), and the prefix
hash chain (Sec. 2.1)."""
import multiprocessing as mp
import os

import numpy as np
import pytest

from paper_2609_11744_b200 import kvc


def _aligned(nbytes, fill=None, seed=0):
    raw = np.zeros(nbytes + 4096, dtype=np.uint8)
    off = (-raw.ctypes.data) % 4096
    buf = raw[off:off + nbytes]
    if seed:
        buf[:] = np.random.default_rng(seed).integers(0, 256, nbytes, dtype=np.uint8)
    return buf


def test_fnv1a64_published_vectors():
    # test vectors of the FNV-1a 64-bit hash as published with the algorithm
    assert kvc.kvc_fnv1a64(b"") == 0xcbf29ce484222325
    assert kvc.kvc_fnv1a64(b"a") == 0xaf63dc4c8601ec8c
    assert kvc.kvc_fnv1a64(b"foobar") == 0x85944171f73967e8


def test_chain_hash_is_fnv_over_prev_and_tokens_and_chains_prefixes():
    toks = np.arange(100, 132, dtype=np.int32)
    for prev in (0, 0x0123456789abcdef):
        want = kvc.kvc_fnv1a64(int(prev).to_bytes(8, "little") + toks.tobytes())
        assert kvc.kvc_chain_hash(prev, toks) == want
    # Sec. 2.1: same block tokens after different prefixes hash differently; same prefix -> same chain
    a = [np.arange(0, 16), np.arange(16, 32), np.arange(32, 48)]
    b = [np.arange(0, 16), np.arange(99, 115), np.arange(32, 48)]

    def chain(blocks):
        h, out = 0, []
        for blk in blocks:
            h = kvc.kvc_chain_hash(h, blk)
            out.append(h)
        return out
    ca, cb = chain(a), chain(b)
    assert ca[0] == cb[0] and ca[1] != cb[1] and ca[2] != cb[2]
    assert chain(a) == ca and len(set(ca)) == 3


def test_publish_read_round_trip_and_layout(tmp_path):
    st = kvc.kvc_store_open(str(tmp_path), "llama-8b-bf16-b16", direct_io=True)
    h = 0xAB12CD34EF567890
    path = kvc.kvc_store_path(st, h)
    assert path == os.path.join(str(tmp_path), "llama-8b-bf16-b16", "ab", "12", "ab12cd34ef567890.kv")
    assert kvc.kvc_store_lookup(st, h) is None
    data = _aligned(1 << 20, seed=5)
    assert kvc.kvc_store_publish(st, h, data) is True
    assert kvc.kvc_store_lookup(st, h) == 1 << 20
    assert os.listdir(os.path.dirname(path)) == ["ab12cd34ef567890.kv"]     # no temporary left behind
    back = _aligned(1 << 20)
    kvc.kvc_store_read(st, h, back)
    assert np.array_equal(back, data)
    # a second publication of the same hash keeps the first entry
    other = _aligned(1 << 20, seed=6)
    assert kvc.kvc_store_publish(st, h, other) is False
    kvc.kvc_store_read(st, h, back)
    assert np.array_equal(back, data)
    # unaligned buffers and odd sizes work too (buffered I/O)
    odd = np.arange(1000, dtype=np.uint8)[1:]
    assert kvc.kvc_store_publish(st, 7, odd) is True
    got = np.zeros(999, dtype=np.uint8)
    kvc.kvc_store_read(st, 7, got)
    assert np.array_equal(got, odd)
    # errors
    with pytest.raises(kvc.KvcError) as e:
        kvc.kvc_store_read(st, 0xdead, back)
    assert e.value.status == kvc.KVC_ERR_NOT_FOUND
    with pytest.raises(kvc.KvcError) as e:
        kvc.kvc_store_read(st, h, back[:4096])           # entry has another size
    assert e.value.status == kvc.KVC_ERR_INVALID_ARG
    with pytest.raises(kvc.KvcError):
        kvc.kvc_store_open(str(tmp_path), "bad/tag")
    assert kvc.kvc_store_direct_io_refused(st) >= 0
    kvc.kvc_store_close(st)


def _racer(root, seed, barrier, q):
    from paper_2609_11744_b200 import kvc as k
    st = k.kvc_store_open(root, "m", direct_io=False)
    data = np.full(1 << 18, seed, dtype=np.uint8)
    barrier.wait()
    wins = [k.kvc_store_publish(st, 1000 + i, data) for i in range(40)]
    q.put((seed, wins))


def test_first_writer_wins_between_processes(tmp_path):
    """Four processes publish the same 40 hashes at once: every entry ends up complete, written by
    exactly one of them, and every publish call reports truthfully whether it was the winner."""
    ctx = mp.get_context("fork")
    n = 4
    barrier, q = ctx.Barrier(n), ctx.Queue()
    procs = [ctx.Process(target=_racer, args=(str(tmp_path), s + 1, barrier, q)) for s in range(n)]
    for p in procs:
        p.start()
    results = dict(q.get(timeout=120) for _ in range(n))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    st = kvc.kvc_store_open(str(tmp_path), "m", direct_io=False)
    buf = np.zeros(1 << 18, dtype=np.uint8)
    for i in range(40):
        winners = [s for s, wins in results.items() if wins[i]]
        assert len(winners) == 1, (i, winners)
        kvc.kvc_store_read(st, 1000 + i, buf)
        assert (buf == winners[0]).all()                # complete, and the winner's bytes
    leftovers = [f for _, _, fs in os.walk(str(tmp_path)) for f in fs if f.startswith(".tmp")]
    assert leftovers == []


def test_file_system_that_refuses_direct_io_falls_back_and_leaves_no_litter(tmp_path):
    """Linux creates the file before it refuses O_DIRECT on a file system without it.  The store
    must remove that empty file, retry with buffered I/O, count the refusal, publish the entry
    and leave no temporary name behind.  The refusal is played by an open() stand-in."""
    import ctypes
    libc = ctypes.CDLL(None, use_errno=True)
    libc.open.restype = ctypes.c_int
    libc.open.argtypes = [ctypes.c_char_p, ctypes.c_int, ctypes.c_uint]
    refused = []

    def refusing_open(path, flags, mode):
        if flags & os.O_DIRECT:
            if flags & os.O_CREAT:                       # what the kernel does: create, then refuse
                fd = libc.open(path, flags & ~os.O_DIRECT, mode)
                if fd >= 0:
                    os.close(fd)
            refused.append(path)
            ctypes.set_errno(22)                         # EINVAL
            return -1
        fd = libc.open(path, flags, mode)
        if fd < 0:
            ctypes.set_errno(ctypes.get_errno())
        return fd

    st = kvc.kvc_store_open(str(tmp_path), "m", direct_io=True)
    try:
        kvc.kvc_store_set_open_fn(refusing_open)
        data = _aligned(1 << 20, seed=11)
        assert kvc.kvc_store_publish(st, 0xabcdef, data) is True
        assert kvc.kvc_store_direct_io_refused(st) == 1 and len(refused) == 1
        back = _aligned(1 << 20, seed=12)
        kvc.kvc_store_read(st, 0xabcdef, back)           # the read is refused once too, then buffered
        assert np.array_equal(back, data)
        assert kvc.kvc_store_direct_io_refused(st) == 2
        assert kvc.kvc_store_publish(st, 0xabcdef, data) is False
    finally:
        kvc.kvc_store_set_open_fn(None)
        kvc.kvc_store_close(st)
    leftovers = [f for _, _, fs in os.walk(str(tmp_path)) for f in fs if f.startswith(".tmp")]
    assert leftovers == []
