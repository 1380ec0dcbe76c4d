"""Pins for the CPU oracle: each test ties the oracle to something that is not the
oracle -- printed sizes, hand-worked indices, numpy's own index routines, closed
forms and invariants -- so that a dropped term, a swapped axis or a wrong sign in
the oracle fails at least one of them.  No GPU needed."""
import itertools
import os

import numpy as np
import pytest

from oracle import oracle as orc
from oracle.oracle import Dims

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _read_kv(path):
    out = {}
    with open(path) as f:
        for line in f:
            line = line.split("#", 1)[0].strip()
            if line:
                k, v = [s.strip() for s in line.split("=")]
                out[k] = float(v) if "." in v else int(v)
    return out


# ---------------------------------------------------------------- printed sizes (Sec. 2.1, 4.1, 6.4)
def test_paper_sizes():
    g = _read_kv(os.path.join(GOLDEN, "kv_sizes.txt"))
    d = Dims(L=g["layers"], P=g["planes"], NB=1, B=16, H=g["kv_heads"], D=g["head_dim"],
             e=g["elem_bytes"])
    assert d.bytes_per_token == g["bytes_per_token"] == 112 * 1024
    assert d.bytes_per_token * g["tokens_80k"] == int(g["gib_80k"] * 2**30)
    nb = g["chunk_tokens"] // d.B
    assert orc.chunk_bytes(d, nb) == int(g["chunk_mib"] * 2**20)
    assert orc.blocks_per_chunk(d, g["chunk_tokens"]) == 16
    # the 8B shape of the benchmark configs: 128 KiB per token, 2 MiB per block, 32 MiB per chunk
    d8 = Dims(32, 2, 1, 16, 8, 128, 2)
    assert d8.bytes_per_token == 128 * 1024 and d8.slab_bytes == 32 * 1024
    assert orc.chunk_bytes(d8, 16) == 32 * 2**20


# ---------------------------------------------------------------- hand-worked indices
def test_worked_example():
    w = _read_kv(os.path.join(GOLDEN, "worked_example.txt"))
    g = Dims(w["L"], w["P"], w["NB"], w["B"], w["H"], w["D"], w["e"])
    c = (w["l"], w["p"], w["j"], w["t"], w["h"], w["d"])
    assert orc.pool_elem(g, w["l"], w["p"], w["block_id"], w["t"], w["h"], w["d"]) == w["pool_elem"]
    assert orc.chunk_elem(g, w["nb_c"], *c) == w["chunk_elem"]
    assert w["pool_elem"] * g.e == w["pool_byte"] and w["chunk_elem"] * g.e == w["chunk_byte"]
    assert orc.chunk_bytes(g, w["nb_c"]) == w["chunk_bytes"]
    # the C copies of the two formulas agree with the hand-worked numbers too
    lib, cd = orc._clib(), orc._cd(g)
    import ctypes
    assert lib.kvc_oracle_pool_elem(ctypes.byref(cd), w["l"], w["p"], w["block_id"], w["t"],
                                    w["h"], w["d"]) == w["pool_elem"]
    assert lib.kvc_oracle_chunk_elem(ctypes.byref(cd), w["nb_c"], *c) == w["chunk_elem"]
    # and the byte really moves there: put a marker at the pool byte, find it at the chunk byte
    pool = np.zeros(g.pool_bytes, dtype=np.uint8)
    pool[w["pool_byte"]] = 0xA5
    pool[w["pool_byte"] + 1] = 0x5A
    ids = np.arange(w["nb_c"], dtype=np.int32) + 7
    ids[w["j"]] = w["block_id"]
    ch = orc.pack_chunk(g, pool, ids)
    nz = np.flatnonzero(ch)
    assert nz.tolist() == [w["chunk_byte"], w["chunk_byte"] + 1]
    assert ch[w["chunk_byte"]] == 0xA5 and ch[w["chunk_byte"] + 1] == 0x5A


# ---------------------------------------------------------------- formulas vs numpy's own index routines
@pytest.mark.parametrize("shape", [(2, 2, 8, 2, 3, 4), (3, 2, 5, 4, 2, 6), (1, 1, 7, 3, 5, 2)])
def test_index_formulas_match_ravel(shape):
    L, P, NB, B, H, D = shape
    g = Dims(L, P, NB, B, H, D, 2)
    rng = np.random.default_rng(1)
    for _ in range(200):
        c = tuple(int(rng.integers(0, s)) for s in shape)
        assert orc.pool_elem(g, *c) == np.ravel_multi_index(c, shape)
        nb_c = int(rng.integers(1, NB + 1))
        cj = (c[0], c[1], int(rng.integers(0, nb_c)), c[3], c[4], c[5])
        assert orc.chunk_elem(g, nb_c, *cj) == np.ravel_multi_index(cj, (L, P, nb_c, B, H, D))


# ---------------------------------------------------------------- unique tags + brute force over all id lists
def _tag_pool(g):
    """4-byte elements whose value is their own flat pool index."""
    assert g.e == 4
    return np.arange(g.pool_bytes // 4, dtype=np.uint32).view(np.uint8).copy()


def test_tags_all_small_id_lists():
    g = Dims(L=2, P=2, NB=8, B=2, H=2, D=4, e=4)   # every axis length distinct from its neighbour's role
    pool = _tag_pool(g)
    for n in range(1, 5):
        for ids in itertools.permutations(range(g.NB), n):
            ch = orc.pack_chunk(g, pool, ids).view(np.uint32)
            # decode every chunk position with numpy, not with the oracle's formula
            l, p, j, t, h, d = np.unravel_index(np.arange(ch.size), (g.L, g.P, n, g.B, g.H, g.D))
            b = np.asarray(ids)[j]
            want = np.ravel_multi_index((l, p, b, t, h, d), (g.L, g.P, g.NB, g.B, g.H, g.D))
            assert np.array_equal(ch, want.astype(np.uint32)), ids
            if n <= 2:   # the pure-Python loops state the same thing
                assert np.array_equal(orc.pack_chunk_loops(g, pool, ids).view(np.uint32), ch)


def test_tags_unpack_all_small_id_lists():
    g = Dims(L=2, P=2, NB=6, B=2, H=3, D=2, e=4)
    sentinel = np.uint32(0xFFFFFFFF)
    for n in range(1, 4):
        for ids in itertools.permutations(range(g.NB), n):
            nel = orc.chunk_bytes(g, n) // 4
            chunk = np.arange(nel, dtype=np.uint32)             # value = own chunk index
            pool = np.full(g.pool_bytes // 4, sentinel, dtype=np.uint32)
            orc.unpack_chunk(g, pool.view(np.uint8), chunk.view(np.uint8), ids)
            p6 = pool.reshape(g.L, g.P, g.NB, g.B, g.H, g.D)
            for j, b in enumerate(ids):
                l, p, t, h, d = np.meshgrid(*[np.arange(s) for s in (g.L, g.P, g.B, g.H, g.D)],
                                            indexing="ij")
                want = np.ravel_multi_index((l, p, np.full_like(l, j), t, h, d),
                                            (g.L, g.P, n, g.B, g.H, g.D))
                assert np.array_equal(p6[:, :, b], want)
            untouched = [b for b in range(g.NB) if b not in ids]
            assert (p6[:, :, untouched] == sentinel).all()
            if n == 1:
                pool2 = np.full(g.pool_bytes // 4, sentinel, dtype=np.uint32)
                orc.unpack_chunk_loops(g, pool2.view(np.uint8), chunk.view(np.uint8), ids)
                assert np.array_equal(pool, pool2)


# ---------------------------------------------------------------- reduces to library routines
@pytest.mark.parametrize("e", [1, 2, 4])
def test_pack_is_numpy_take(e):
    g = Dims(L=3, P=2, NB=37, B=4, H=2, D=8, e=e)
    rng = np.random.default_rng(7)
    pool = rng.integers(0, 256, g.pool_bytes, dtype=np.uint8)
    ids = rng.permutation(g.NB)[:11].astype(np.int32)
    want = np.take(pool.reshape(g.L, g.P, g.NB, g.B, g.H, g.D * e), ids, axis=2).reshape(-1)
    assert np.array_equal(orc.pack_chunk(g, pool, ids), want)
    # duplicates are legal for pack (the block is read twice)
    ids2 = np.array([5, 5, 0, 36, 5], dtype=np.int32)
    want2 = np.take(pool.reshape(g.L, g.P, g.NB, -1), ids2, axis=2).reshape(-1)
    assert np.array_equal(orc.pack_chunk(g, pool, ids2), want2)


def test_identity_table_is_memcpy():
    g = Dims(L=2, P=2, NB=9, B=4, H=2, D=8, e=2)
    pool = np.random.default_rng(3).integers(0, 256, g.pool_bytes, dtype=np.uint8)
    ch = orc.pack_chunk(g, pool, np.arange(g.NB))
    assert ch.tobytes() == pool.tobytes()
    out = np.zeros_like(pool)
    orc.unpack_chunk(g, out, ch, np.arange(g.NB))
    assert out.tobytes() == pool.tobytes()


def test_unpack_is_numpy_fancy_assign():
    g = Dims(L=2, P=2, NB=21, B=4, H=3, D=4, e=2)
    rng = np.random.default_rng(11)
    ids = rng.permutation(g.NB)[:6].astype(np.int32)
    chunk = rng.integers(0, 256, orc.chunk_bytes(g, 6), dtype=np.uint8)
    pool = rng.integers(0, 256, g.pool_bytes, dtype=np.uint8)
    want = pool.copy().reshape(g.L, g.P, g.NB, -1)
    want[:, :, ids] = chunk.reshape(g.L, g.P, 6, -1)
    orc.unpack_chunk(g, pool, chunk, ids)
    assert np.array_equal(pool, want.reshape(-1))


# ---------------------------------------------------------------- invariants
def test_round_trip_and_sentinels():
    g = Dims(L=2, P=2, NB=64, B=16, H=4, D=64, e=2)
    rng = np.random.default_rng(5)
    pool = rng.integers(0, 256, g.pool_bytes, dtype=np.uint8)
    ids = rng.permutation(g.NB)[:24].astype(np.int32)
    chunks = orc.pack_request(g, pool, ids, 128)            # 8 blocks per chunk -> 3 chunks
    assert [c.size for c in chunks] == [orc.chunk_bytes(g, 8)] * 3
    fresh = np.full(g.pool_bytes, 0xEE, dtype=np.uint8)
    orc.unpack_request(g, fresh, chunks, ids, 128)
    a = pool.reshape(g.L, g.P, g.NB, -1)
    b = fresh.reshape(g.L, g.P, g.NB, -1)
    assert np.array_equal(a[:, :, ids], b[:, :, ids])
    rest = np.setdiff1d(np.arange(g.NB), ids)
    assert (b[:, :, rest] == 0xEE).all()
    # pack(unpack(chunks, ids'), ids') == chunks for another table
    ids2 = rng.permutation(g.NB)[:24].astype(np.int32)
    other = np.zeros(g.pool_bytes, dtype=np.uint8)
    orc.unpack_request(g, other, chunks, ids2, 128)
    again = orc.pack_request(g, other, ids2, 128)
    assert all(np.array_equal(x, y) for x, y in zip(chunks, again))


def test_chunk_size_invariance_and_tail():
    g = Dims(L=2, P=2, NB=50, B=4, H=2, D=8, e=2)
    rng = np.random.default_rng(9)
    pool = rng.integers(0, 256, g.pool_bytes, dtype=np.uint8)
    src = rng.permutation(g.NB)[:19].astype(np.int32)       # 19 blocks: ragged for 8 and 16
    dst = rng.permutation(g.NB)[:19].astype(np.int32)
    results = []
    for chunk_tokens in (4, 32, 64, 128):
        chunks = orc.pack_request(g, pool, src, chunk_tokens)
        bpc = chunk_tokens // g.B
        assert len(chunks) == -(-19 // bpc)
        assert sum(c.size for c in chunks) == 19 * g.bytes_per_block   # compact tail: no padding
        out = np.zeros(g.pool_bytes, dtype=np.uint8)
        orc.unpack_request(g, out, chunks, dst, chunk_tokens)
        results.append(out)
    for r in results[1:]:
        assert np.array_equal(results[0], r)
    # with one block per chunk the chunk stream is just the blocks' slabs in request order
    one = orc.pack_request(g, pool, src, g.B)
    p4 = pool.reshape(g.L, g.P, g.NB, -1)
    for j, b in enumerate(src):
        assert np.array_equal(one[j], p4[:, :, b].reshape(-1))


def test_chunk_ranges():
    assert orc.chunk_ranges(64, 16) == [(0, 16), (16, 16), (32, 16), (48, 16)]
    r = orc.chunk_ranges(5000, 16)
    assert len(r) == 313 and r[-1] == (4992, 8)
    r = orc.chunk_ranges(5000, 128)
    assert len(r) == 40 and r[-1] == (4992, 8)
    assert len(orc.chunk_ranges(5000, 1)) == 5000
    assert orc.chunk_ranges(0, 16) == []
    assert orc.chunk_ranges(3, 16) == [(0, 3)]
    for n, bpc in [(1, 1), (17, 4), (128, 128), (129, 128)]:
        rr = orc.chunk_ranges(n, bpc)
        assert sum(nb for _, nb in rr) == n and all(f == i * bpc for i, (f, _) in enumerate(rr))


def test_planes_equal_monolithic_and_padded_stride():
    g = Dims(L=3, P=2, NB=16, B=4, H=2, D=8, e=2)
    rng = np.random.default_rng(13)
    pool = rng.integers(0, 256, g.pool_bytes, dtype=np.uint8)
    ids = rng.permutation(g.NB)[:7].astype(np.int32)
    plane_bytes = g.NB * g.slab_bytes
    planes = [pool[i * plane_bytes:(i + 1) * plane_bytes].copy() for i in range(g.L * g.P)]
    assert np.array_equal(orc.pack_chunk_planes(g, planes, ids), orc.pack_chunk(g, pool, ids))
    # padded blocks: stride 1.5 slabs; padding bytes must never be read or written
    bs = g.slab_bytes * 3 // 2
    padded = []
    for pl in planes:
        q = np.full(g.NB * bs, 0xCC, dtype=np.uint8)
        q.reshape(g.NB, bs)[:, :g.slab_bytes] = pl.reshape(g.NB, g.slab_bytes)
        padded.append(q)
    ch = orc.pack_chunk_planes(g, padded, ids, bs)
    assert np.array_equal(ch, orc.pack_chunk(g, pool, ids))
    dst = [np.full(g.NB * bs, 0xCC, dtype=np.uint8) for _ in planes]
    orc.unpack_chunk_planes(g, dst, ch, ids, bs)
    mono = np.full(g.pool_bytes, 0xCC, dtype=np.uint8)
    orc.unpack_chunk(g, mono, ch, ids)
    for i, q in enumerate(dst):
        q2 = q.reshape(g.NB, bs)
        assert (q2[:, g.slab_bytes:] == 0xCC).all()
        assert np.array_equal(q2[:, :g.slab_bytes].reshape(-1),
                              mono[i * plane_bytes:(i + 1) * plane_bytes])


def test_lp_range_partition_is_the_whole():
    g = Dims(L=4, P=2, NB=12, B=4, H=2, D=8, e=2)
    rng = np.random.default_rng(17)
    pool = rng.integers(0, 256, g.pool_bytes, dtype=np.uint8)
    ids = rng.permutation(g.NB)[:5].astype(np.int32)
    whole = orc.pack_chunk(g, pool, ids)
    parts = np.zeros_like(whole)
    for lo, hi in [(0, 3), (3, 4), (4, 8)]:
        orc.pack_chunk_into(g, pool, ids, parts, (lo, hi))
    assert np.array_equal(whole, parts)
    # unpack side: scattering the chunk plane range by plane range equals scattering it whole,
    # and a single range touches only its own planes
    before = rng.integers(0, 256, g.pool_bytes, dtype=np.uint8)
    dst = rng.permutation(g.NB)[:5].astype(np.int32)
    want = before.copy()
    orc.unpack_chunk(g, want, whole, dst)
    only = before.copy()
    orc.unpack_chunk(g, only, whole, dst, (3, 4))
    pb = g.NB * g.slab_bytes
    assert np.array_equal(only[:3 * pb], before[:3 * pb]) and np.array_equal(only[4 * pb:], before[4 * pb:])
    assert np.array_equal(only[3 * pb:4 * pb], want[3 * pb:4 * pb])
    assert not np.array_equal(only[3 * pb:4 * pb], before[3 * pb:4 * pb])
    pieces = before.copy()
    for lo, hi in [(0, 3), (3, 4), (4, 8)]:
        orc.unpack_chunk(g, pieces, whole, dst, (lo, hi))
    assert np.array_equal(pieces, want)


def test_out_of_range_ids_rejected():
    g = Dims(L=1, P=2, NB=4, B=2, H=2, D=2, e=2)
    pool = np.zeros(g.pool_bytes, dtype=np.uint8)
    for bad in ([4], [-1], [0, 1, 99]):
        with pytest.raises(IndexError):
            orc.pack_chunk(g, pool, bad)
        with pytest.raises(IndexError):
            orc.unpack_chunk(g, pool, np.zeros(orc.chunk_bytes(g, len(bad)), np.uint8), bad)


# ---------------------------------------------------------------- shared-prefix dedup (Sec. 6.5)
def test_dedup_ops_small_cases():
    shared = [10, 11, 12, 13]
    tables = [shared + [20, 21, 22], shared + [30], shared[:2], shared + [20, 21, 22]]
    kept = orc.dedup_ops(tables, 2)
    # request 0 keeps all 4 of its chunks; request 1 only its private tail chunk;
    # request 2 (a prefix of the shared list) and request 3 (identical to 0) add nothing
    assert kept == [(0, 0, 0, 2), (0, 1, 2, 2), (0, 2, 4, 2), (0, 3, 6, 1), (1, 2, 4, 1)]
    # every distinct (history, block) pair is staged exactly once
    covered = set()
    for r, c, f, nb in kept:
        for i in range(f, f + nb):
            key = tuple(tables[r][:i + 1])
            assert key not in covered
            covered.add(key)
    every = {tuple(t[:i + 1]) for t in tables for i in range(len(t))}
    assert covered == every
    # same ids at the same position but a different history are NOT shared
    kept2 = orc.dedup_ops([[1, 2, 3, 4], [9, 2, 3, 4]], 2)
    assert len(kept2) == 4
    # a shorter tail chunk that is a prefix of a longer one is dropped
    assert orc.dedup_ops([[1, 2, 3], [1, 2, 3, 4]], 2) == [(0, 0, 0, 2), (1, 1, 2, 2)]


# ---------------------------------------------------------------- block-major chunk order
def test_block_major_chunk_order_pins():
    g = Dims(L=3, P=2, NB=11, B=2, H=3, D=4, e=4)
    pool = _tag_pool(g)                       # value = own dense pool index
    planes = orc.dense_planes(g, pool)
    rng = np.random.default_rng(21)
    for n in (1, 4, 7):
        ids = rng.permutation(g.NB)[:n].astype(np.int32)
        ch = orc.pack_chunk_planes_block_major(g, planes, ids).view(np.uint32)
        # decode each chunk position with numpy over the block-major shape
        j, l, p, t, h, d = np.unravel_index(np.arange(ch.size), (n, g.L, g.P, g.B, g.H, g.D))
        want = np.ravel_multi_index((l, p, ids[j], t, h, d), (g.L, g.P, g.NB, g.B, g.H, g.D))
        assert np.array_equal(ch, want.astype(np.uint32))
        # it is the layer-major chunk with the block axis moved to the front (library routine)
        lm = orc.pack_chunk(g, pool, ids).view(np.uint32).reshape(g.L, g.P, n, -1)
        assert np.array_equal(ch, np.moveaxis(lm, 2, 0).reshape(-1))
        # a shorter chunk is a prefix of a longer one (what makes the order attractive for files)
        if n > 1:
            shorter = orc.pack_chunk_planes_block_major(g, planes, ids[:n - 1])
            assert np.array_equal(shorter, ch.view(np.uint8)[:shorter.size])
        # formula against numpy
        for _ in range(50):
            c = tuple(int(rng.integers(0, s)) for s in (g.L, g.P, n, g.B, g.H, g.D))
            assert orc.chunk_elem_block_major(g, n, *c) == np.ravel_multi_index(
                (c[2], c[0], c[1], c[3], c[4], c[5]), (n, g.L, g.P, g.B, g.H, g.D))
        # round trip into a sentinel pool
        fresh = np.full(g.pool_bytes, 0xEE, dtype=np.uint8)
        orc.unpack_chunk_planes_block_major(g, orc.dense_planes(g, fresh), ch.view(np.uint8), ids)
        a, b = pool.reshape(g.L, g.P, g.NB, -1), fresh.reshape(g.L, g.P, g.NB, -1)
        assert np.array_equal(a[:, :, ids], b[:, :, ids])
        rest = np.setdiff1d(np.arange(g.NB), ids)
        assert (b[:, :, rest] == 0xEE).all()


def test_interleaved_kv_pool_order_is_a_strided_plane_view():
    """A pool laid out [L][NB][P][B][H][D] (K|V inside the block axis) is the same data seen as
    planes with plane stride S and block stride P*S: its chunks equal those of the dense pool."""
    g = Dims(L=2, P=2, NB=9, B=4, H=2, D=8, e=2)
    rng = np.random.default_rng(23)
    dense = rng.integers(0, 256, g.pool_bytes, dtype=np.uint8)
    S = g.slab_bytes
    inter = np.ascontiguousarray(
        dense.reshape(g.L, g.P, g.NB, S).transpose(0, 2, 1, 3)).reshape(-1)   # [L][NB][P][S]
    layer = g.NB * g.P * S
    planes = [inter[l * layer + p * S:] for l in range(g.L) for p in range(g.P)]
    planes = [pl[:(g.NB - 1) * g.P * S + S] for pl in planes]
    ids = rng.permutation(g.NB)[:5].astype(np.int32)
    assert np.array_equal(orc.pack_chunk_planes(g, planes, ids, g.P * S), orc.pack_chunk(g, dense, ids))


# ---------------------------------------------------------------- random layouts (hypothesis)
from hypothesis import given, settings, strategies as st


@settings(max_examples=60, deadline=None)
@given(L=st.integers(1, 4), P=st.integers(1, 3), NB=st.integers(1, 12), B=st.integers(1, 5),
       H=st.integers(1, 4), D=st.integers(1, 9), e=st.sampled_from([1, 2, 4]),
       data=st.data())
def test_random_layouts_against_numpy_and_round_trip(L, P, NB, B, H, D, e, data):
    g = Dims(L, P, NB, B, H, D, e)
    n = data.draw(st.integers(1, NB))
    ids = np.array(data.draw(st.permutations(list(range(NB))))[:n], dtype=np.int32)
    seed = data.draw(st.integers(0, 2**31))
    pool = np.random.default_rng(seed).integers(0, 256, g.pool_bytes, dtype=np.uint8)
    # layer-major chunk = take along the block axis; block-major = the same with that axis first
    lm = orc.pack_chunk(g, pool, ids)
    want = np.take(pool.reshape(L, P, NB, -1), ids, axis=2)
    assert np.array_equal(lm, want.reshape(-1))
    bm = orc.pack_chunk_planes_block_major(g, orc.dense_planes(g, pool), ids)
    assert np.array_equal(bm, np.moveaxis(want, 2, 0).reshape(-1))
    assert np.array_equal(orc.pack_chunk_planes(g, orc.dense_planes(g, pool), ids), lm)
    # unpack into a sentinel pool restores exactly the named blocks
    fresh = np.full(g.pool_bytes, 0xA7, dtype=np.uint8)
    orc.unpack_chunk(g, fresh, lm, ids)
    f4, p4 = fresh.reshape(L, P, NB, -1), pool.reshape(L, P, NB, -1)
    assert np.array_equal(f4[:, :, ids], p4[:, :, ids])
    rest = np.setdiff1d(np.arange(NB), ids)
    assert (f4[:, :, rest] == 0xA7).all()
    fresh2 = np.full(g.pool_bytes, 0xA7, dtype=np.uint8)
    orc.unpack_chunk_planes_block_major(g, orc.dense_planes(g, fresh2), bm, ids)
    assert np.array_equal(fresh2, fresh)
