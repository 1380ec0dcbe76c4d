"""TEST INFRASTRUCTURE -- plain CPU statement of paged-KV pack / unpack.

Notation (paper Sec. 2.1 for the paged pool and the bytes-per-token formula,
Sec. 6.4 for storage blocks = chunks, one staging slot per chunk):

    L layers, P planes per layer (K, V), NB pool blocks, B tokens per block,
    H kv heads, D head dim, e bytes per element.
    pool   [L][P][NB][B][H][D]        chunk of nb_c blocks  [L][P][nb_c][B][H][D]
    pack  : chunk[l,p,j,t,h,d]      = pool[l,p,ids[j],t,h,d]
    unpack: pool[l,p,ids[j],t,h,d]  = chunk[l,p,j,t,h,d]

A request with n block ids and ``chunk_tokens`` tokens per chunk is cut, in
request order, into ceil(n / bpc) chunks (bpc = chunk_tokens / B); the last
one may be short and is stored compactly (its own nb_c in the formula).

Three statements of the same thing live here:
  * ``*_chunk`` / ``*_request`` -- the oracle proper: six nested C loops over
    element coordinates (kvc_oracle.c), called through ctypes;
  * ``*_chunk_loops`` -- the same loops in pure Python, for tiny layouts;
  * the index formulas ``pool_elem`` / ``chunk_elem`` on their own.
Pool data is handed over as bytes (numpy uint8); elements are never
interpreted.  Nothing here imports or calls the CUDA library.
"""
from __future__ import annotations

import ctypes
from dataclasses import dataclass
from typing import List, Sequence, Tuple

import numpy as np

from . import build as _build


@dataclass(frozen=True)
class Dims:
    """Shape of a paged KV pool (Sec. 2.1)."""
    L: int
    P: int
    NB: int
    B: int
    H: int
    D: int
    e: int

    @property
    def row_bytes(self) -> int:      # one token of one plane: H*D elements
        return self.H * self.D * self.e

    @property
    def slab_bytes(self) -> int:     # one block of one plane: B tokens
        return self.B * self.row_bytes

    @property
    def bytes_per_token(self) -> int:
        # Sec. 2.1: layers x 2 x KV heads x head dim x datatype size
        return self.L * self.P * self.H * self.D * self.e

    @property
    def bytes_per_block(self) -> int:
        return self.bytes_per_token * self.B

    @property
    def pool_bytes(self) -> int:
        return self.bytes_per_block * self.NB


# ---------------------------------------------------------------- index formulas
def pool_elem(g: Dims, l: int, p: int, b: int, t: int, h: int, d: int) -> int:
    """Element index in the dense pool [L][P][NB][B][H][D]."""
    return ((((l * g.P + p) * g.NB + b) * g.B + t) * g.H + h) * g.D + d


def chunk_elem(g: Dims, nb_c: int, l: int, p: int, j: int, t: int, h: int, d: int) -> int:
    """Element index in a chunk of nb_c blocks, [L][P][nb_c][B][H][D]."""
    return ((((l * g.P + p) * nb_c + j) * g.B + t) * g.H + h) * g.D + d


def chunk_elem_block_major(g: Dims, nb_c: int, l: int, p: int, j: int, t: int, h: int, d: int) -> int:
    """Element index in a block-major chunk, [nb_c][L][P][B][H][D] (nb_c does not enter)."""
    return ((((j * g.L + l) * g.P + p) * g.B + t) * g.H + h) * g.D + d


def chunk_bytes(g: Dims, nb_c: int) -> int:
    """Exact size of a chunk of nb_c blocks: every byte is useful KV data."""
    return g.L * g.P * nb_c * g.slab_bytes


def blocks_per_chunk(g: Dims, chunk_tokens: int) -> int:
    if chunk_tokens <= 0 or chunk_tokens % g.B:
        raise ValueError("chunk_tokens must be a positive multiple of the block size")
    return chunk_tokens // g.B


def chunk_ranges(n_blocks: int, bpc: int) -> List[Tuple[int, int]]:
    """Sec. 6.4: one job per storage block.  Chunk c covers table entries
    [c*bpc, min((c+1)*bpc, n)); returns (first, nb_c) per chunk."""
    out = []
    c = 0
    while c * bpc < n_blocks:
        first = c * bpc
        out.append((first, min(bpc, n_blocks - first)))
        c += 1
    return out


def dedup_ops(tables: Sequence[Sequence[int]], bpc: int) -> List[Tuple[int, int, int, int]]:
    """Sec. 6.5: requests whose block tables start identically share one
    staged copy of the common chunks.  Brute-force statement: chunk c of
    request r is dropped when some other request r2 has a chunk c whose block
    table, from entry 0 up to that chunk's end, starts with r's table up to
    its chunk's end -- i.e. the other chunk already carries every block of
    this one at the same position with the same history -- and r2's is longer
    there or, on an exact tie, r2 < r.  Returns kept ops (r, c, first, nb_c)
    in (r, c) order."""
    ops = []
    for r, tab in enumerate(tables):
        for c, (first, nb_c) in enumerate(chunk_ranges(len(tab), bpc)):
            ops.append((r, c, first, nb_c))
    kept = []
    for (r, c, first, nb_c) in ops:
        mine = tuple(tables[r][: first + nb_c])
        dropped = False
        for (r2, c2, first2, nb2) in ops:
            if r2 == r or c2 != c:
                continue
            other = tuple(tables[r2][: first2 + nb2])
            if len(other) >= len(mine) and other[: len(mine)] == mine:
                if len(other) > len(mine) or r2 < r:
                    dropped = True
                    break
        if not dropped:
            kept.append((r, c, first, nb_c))
    return kept


# ---------------------------------------------------------------- C loops via ctypes
class _CDims(ctypes.Structure):
    _fields_ = [(k, ctypes.c_uint32) for k in ("L", "P", "NB", "B", "H", "D", "e")]


_lib = None


def _clib():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(_build.build())
        u8p, i32p, u32, u64 = (ctypes.c_void_p, ctypes.c_void_p, ctypes.c_uint32,
                               ctypes.c_uint64)
        dp = ctypes.POINTER(_CDims)
        lib.kvc_oracle_pool_elem.restype = u64
        lib.kvc_oracle_pool_elem.argtypes = [dp] + [u64] * 6
        lib.kvc_oracle_chunk_elem.restype = u64
        lib.kvc_oracle_chunk_elem.argtypes = [dp] + [u64] * 7
        for name in ("kvc_oracle_pack_chunk_mono", "kvc_oracle_unpack_chunk_mono"):
            f = getattr(lib, name)
            f.restype = ctypes.c_int
            f.argtypes = [dp, u8p, i32p, u32, u8p, u32, u32]
        for name in ("kvc_oracle_pack_chunk_planes", "kvc_oracle_unpack_chunk_planes"):
            f = getattr(lib, name)
            f.restype = ctypes.c_int
            f.argtypes = [dp, ctypes.c_void_p, u64, i32p, u32, u8p, u32, u32]
        for name in ("kvc_oracle_pack_chunk_planes_block_major",
                     "kvc_oracle_unpack_chunk_planes_block_major"):
            f = getattr(lib, name)
            f.restype = ctypes.c_int
            f.argtypes = [dp, ctypes.c_void_p, u64, i32p, u32, u8p]
        lib.kvc_oracle_chunk_elem_block_major.restype = u64
        lib.kvc_oracle_chunk_elem_block_major.argtypes = [dp] + [u64] * 7
        _lib = lib
    return _lib


def _cd(g: Dims) -> _CDims:
    return _CDims(g.L, g.P, g.NB, g.B, g.H, g.D, g.e)


def _bytes_view(a: np.ndarray) -> np.ndarray:
    if a.dtype != np.uint8 or not a.flags.c_contiguous or a.ndim != 1:
        raise ValueError("expected a flat contiguous uint8 array")
    return a


def _ids32(ids) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(ids, dtype=np.int32))


def pack_chunk(g: Dims, pool: np.ndarray, ids, lp_range=None) -> np.ndarray:
    """Pack one chunk from a dense monolithic pool (flat uint8 of g.pool_bytes)."""
    pool = _bytes_view(pool)
    assert pool.size == g.pool_bytes
    ids = _ids32(ids)
    out = np.zeros(chunk_bytes(g, len(ids)), dtype=np.uint8)
    lo, hi = lp_range if lp_range else (0, g.L * g.P)
    rc = _clib().kvc_oracle_pack_chunk_mono(ctypes.byref(_cd(g)), pool.ctypes.data,
                                            ids.ctypes.data, len(ids), out.ctypes.data, lo, hi)
    if rc:
        raise IndexError("block id out of range")
    return out


def pack_chunk_into(g: Dims, pool: np.ndarray, ids, out: np.ndarray, lp_range=None) -> None:
    """Same as pack_chunk but writes into a caller buffer (used for timing and threads)."""
    pool, out, ids = _bytes_view(pool), _bytes_view(out), _ids32(ids)
    assert pool.size == g.pool_bytes and out.size == chunk_bytes(g, len(ids))
    lo, hi = lp_range if lp_range else (0, g.L * g.P)
    rc = _clib().kvc_oracle_pack_chunk_mono(ctypes.byref(_cd(g)), pool.ctypes.data,
                                            ids.ctypes.data, len(ids), out.ctypes.data, lo, hi)
    if rc:
        raise IndexError("block id out of range")


def unpack_chunk(g: Dims, pool: np.ndarray, chunk: np.ndarray, ids, lp_range=None) -> None:
    """Unpack one chunk into a dense monolithic pool, in place."""
    pool, chunk, ids = _bytes_view(pool), _bytes_view(chunk), _ids32(ids)
    assert pool.size == g.pool_bytes and chunk.size == chunk_bytes(g, len(ids))
    lo, hi = lp_range if lp_range else (0, g.L * g.P)
    rc = _clib().kvc_oracle_unpack_chunk_mono(ctypes.byref(_cd(g)), pool.ctypes.data,
                                              ids.ctypes.data, len(ids), chunk.ctypes.data, lo, hi)
    if rc:
        raise IndexError("block id out of range")


def _plane_ptrs(g: Dims, planes: Sequence[np.ndarray], block_stride_bytes: int):
    assert len(planes) == g.L * g.P
    assert block_stride_bytes % g.e == 0 and block_stride_bytes >= g.slab_bytes
    need = (g.NB - 1) * block_stride_bytes + g.slab_bytes
    arr = (ctypes.c_void_p * len(planes))()
    for i, pl in enumerate(planes):
        pl = _bytes_view(pl)
        assert pl.size >= need
        arr[i] = pl.ctypes.data
    return arr


def pack_chunk_planes(g: Dims, planes: Sequence[np.ndarray], ids,
                      block_stride_bytes: int | None = None) -> np.ndarray:
    """Pack one chunk when every (layer, K|V) plane is its own allocation."""
    bs = block_stride_bytes or g.slab_bytes
    arr = _plane_ptrs(g, planes, bs)
    ids = _ids32(ids)
    out = np.zeros(chunk_bytes(g, len(ids)), dtype=np.uint8)
    rc = _clib().kvc_oracle_pack_chunk_planes(ctypes.byref(_cd(g)), arr, bs // g.e,
                                              ids.ctypes.data, len(ids), out.ctypes.data,
                                              0, g.L * g.P)
    if rc:
        raise IndexError("block id out of range")
    return out


def unpack_chunk_planes(g: Dims, planes: Sequence[np.ndarray], chunk: np.ndarray, ids,
                        block_stride_bytes: int | None = None) -> None:
    bs = block_stride_bytes or g.slab_bytes
    arr = _plane_ptrs(g, planes, bs)
    chunk, ids = _bytes_view(chunk), _ids32(ids)
    assert chunk.size == chunk_bytes(g, len(ids))
    rc = _clib().kvc_oracle_unpack_chunk_planes(ctypes.byref(_cd(g)), arr, bs // g.e,
                                                ids.ctypes.data, len(ids), chunk.ctypes.data,
                                                0, g.L * g.P)
    if rc:
        raise IndexError("block id out of range")


def pack_chunk_planes_block_major(g: Dims, planes: Sequence[np.ndarray], ids,
                                  block_stride_bytes: int | None = None) -> np.ndarray:
    """Pack one chunk in block-major order [nb_c][L][P][B][H][D]."""
    bs = block_stride_bytes or g.slab_bytes
    arr = _plane_ptrs(g, planes, bs)
    ids = _ids32(ids)
    out = np.zeros(chunk_bytes(g, len(ids)), dtype=np.uint8)
    rc = _clib().kvc_oracle_pack_chunk_planes_block_major(ctypes.byref(_cd(g)), arr, bs // g.e,
                                                          ids.ctypes.data, len(ids), out.ctypes.data)
    if rc:
        raise IndexError("block id out of range")
    return out


def unpack_chunk_planes_block_major(g: Dims, planes: Sequence[np.ndarray], chunk: np.ndarray, ids,
                                    block_stride_bytes: int | None = None) -> None:
    bs = block_stride_bytes or g.slab_bytes
    arr = _plane_ptrs(g, planes, bs)
    chunk, ids = _bytes_view(chunk), _ids32(ids)
    assert chunk.size == chunk_bytes(g, len(ids))
    rc = _clib().kvc_oracle_unpack_chunk_planes_block_major(ctypes.byref(_cd(g)), arr, bs // g.e,
                                                            ids.ctypes.data, len(ids),
                                                            chunk.ctypes.data)
    if rc:
        raise IndexError("block id out of range")


def dense_planes(g: Dims, pool: np.ndarray) -> List[np.ndarray]:
    """The L*P planes of a dense pool [L][P][NB][B][H][D] as views (plane l*P+p)."""
    pool = _bytes_view(pool)
    pb = g.NB * g.slab_bytes
    return [pool[i * pb:(i + 1) * pb] for i in range(g.L * g.P)]


def pack_request(g: Dims, pool: np.ndarray, ids, chunk_tokens: int) -> List[np.ndarray]:
    """Sec. 6.4: the whole prefix of a request, one chunk per storage block, in order."""
    ids = _ids32(ids)
    bpc = blocks_per_chunk(g, chunk_tokens)
    return [pack_chunk(g, pool, ids[f:f + nb]) for f, nb in chunk_ranges(len(ids), bpc)]


def unpack_request(g: Dims, pool: np.ndarray, chunks: Sequence[np.ndarray], ids,
                   chunk_tokens: int) -> None:
    ids = _ids32(ids)
    bpc = blocks_per_chunk(g, chunk_tokens)
    ranges = chunk_ranges(len(ids), bpc)
    assert len(ranges) == len(chunks)
    for (f, nb), ch in zip(ranges, chunks):
        unpack_chunk(g, pool, ch, ids[f:f + nb])


# ---------------------------------------------------------------- pure-Python loops
def pack_chunk_loops(g: Dims, pool: np.ndarray, ids) -> np.ndarray:
    """The definition in pure Python loops over element coordinates (tiny layouts only)."""
    pool = _bytes_view(pool)
    nb_c = len(ids)
    out = np.zeros(chunk_bytes(g, nb_c), dtype=np.uint8)
    for l in range(g.L):
        for p in range(g.P):
            for j in range(nb_c):
                b = int(ids[j])
                if not 0 <= b < g.NB:
                    raise IndexError("block id out of range")
                for t in range(g.B):
                    for h in range(g.H):
                        for d in range(g.D):
                            s = pool_elem(g, l, p, b, t, h, d) * g.e
                            q = chunk_elem(g, nb_c, l, p, j, t, h, d) * g.e
                            for k in range(g.e):
                                out[q + k] = pool[s + k]
    return out


def unpack_chunk_loops(g: Dims, pool: np.ndarray, chunk: np.ndarray, ids) -> None:
    pool, chunk = _bytes_view(pool), _bytes_view(chunk)
    nb_c = len(ids)
    for l in range(g.L):
        for p in range(g.P):
            for j in range(nb_c):
                b = int(ids[j])
                if not 0 <= b < g.NB:
                    raise IndexError("block id out of range")
                for t in range(g.B):
                    for h in range(g.H):
                        for d in range(g.D):
                            q = pool_elem(g, l, p, b, t, h, d) * g.e
                            s = chunk_elem(g, nb_c, l, p, j, t, h, d) * g.e
                            for k in range(g.e):
                                pool[q + k] = chunk[s + k]
