"""Seeded synthetic inputs shared by the tests, the smoke check and the benchmark.

This module only draws shapes, random bits and block tables.  It holds none of
the pack/unpack arithmetic, so both the CUDA path and the CPU oracle can be fed
from it without sharing any code of the method.

The workloads stand in for the paper's (Sec. 4.1 long-document prefixes up to
80k tokens; Sec. 6.4 storage blocks of 256 tokens built from 16-token GPU
blocks; Sec. 5.1 2048-token offload transfers and sub-chunk transfers; Sec. 6.4
loads of many concurrent requests fused into one launch; Sec. 6.5 requests that
share a prefix).  The paper's datasets are not available; lengths are lognormal.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Tuple

import numpy as np

BASE_SEED = 260911744
DST_SEED_OFFSET = 1000


@dataclass(frozen=True)
class KVShape:
    """Paged-KV geometry: layers, planes (K,V), tokens per block, kv heads, head dim, element bytes."""
    L: int
    P: int
    B: int
    H: int
    D: int
    e: int

    @property
    def slab_bytes(self) -> int:
        return self.B * self.H * self.D * self.e

    @property
    def bytes_per_token(self) -> int:
        return self.L * self.P * self.H * self.D * self.e

    @property
    def bytes_per_block(self) -> int:
        return self.bytes_per_token * self.B


TINY = KVShape(L=2, P=2, B=16, H=4, D=64, e=2)
LLAMA_8B = KVShape(L=32, P=2, B=16, H=8, D=128, e=2)
LLAMA_70B = KVShape(L=80, P=2, B=16, H=8, D=128, e=2)


@dataclass(frozen=True)
class Workload:
    name: str
    index: int                 # position in the benchmark's config list
    shape: KVShape
    pool_blocks: int
    request_tokens: int        # single-request configs; 0 for the batch config
    chunk_tokens: Tuple[int, ...]
    separate_planes: bool = False
    extra: Dict[str, float] = field(default_factory=dict)

    @property
    def seed(self) -> int:
        return BASE_SEED + self.index

    @property
    def dst_seed(self) -> int:
        return self.seed + DST_SEED_OFFSET

    @property
    def request_blocks(self) -> int:
        return self.request_tokens // self.shape.B


WORKLOADS: Dict[str, Workload] = {
    w.name: w for w in [
        Workload("tiny", 0, TINY, 256, 1024, (256,), separate_planes=True),
        Workload("8b_8k", 1, LLAMA_8B, 4096, 8192, (256,)),
        Workload("8b_80k", 2, LLAMA_8B, 20000, 80000, (16, 256, 2048)),
        Workload("70b_batch", 3, LLAMA_70B, 0, 0, (256,),
                 extra={"requests": 64, "median_tokens": 2048, "sigma": 1.0,
                        "min_tokens": 128, "max_tokens": 32768, "shared_tokens": 1024,
                        "pool_slack": 1.25}),
        Workload("8b_ring", 4, LLAMA_8B, 4096, 32768, (256,),
                 extra={"ring_slots": 8}),
    ]
}


def block_ids(seed: int, pool_blocks: int, n: int) -> np.ndarray:
    """First n entries of a seeded permutation of the pool's block ids (int32)."""
    perm = np.random.Generator(np.random.PCG64(seed)).permutation(pool_blocks)
    return np.ascontiguousarray(perm[:n].astype(np.int32))


def random_bits(seed: int, nbytes: int) -> np.ndarray:
    """nbytes of uniform random bits as a flat uint8 array (every 16-bit pattern occurs,
    NaN/Inf/denormal encodings included: values must be compared as integers)."""
    assert nbytes % 2 == 0
    rng = np.random.Generator(np.random.PCG64(seed))
    return rng.integers(0, 65536, size=nbytes // 2, dtype=np.uint16).view(np.uint8)


def random_bits_cuda(seed: int, nbytes: int, device="cuda:0"):
    """nbytes of uniform random bits in device memory (flat torch.uint8), drawn on
    the device in pieces so that no host copy of a multi-GiB pool is ever needed."""
    import torch
    assert nbytes % 2 == 0
    gen = torch.Generator(device=device)
    gen.manual_seed(seed)
    out = torch.empty(nbytes // 2, dtype=torch.int16, device=device)
    piece = 1 << 28
    for lo in range(0, out.numel(), piece):
        hi = min(out.numel(), lo + piece)
        out[lo:hi].random_(-32768, 32768, generator=gen)
    return out.view(torch.uint8)


def lognormal_tokens(seed: int, n_requests: int, median: float, sigma: float,
                     lo: int, hi: int, block_size: int) -> np.ndarray:
    """Prefix lengths in tokens: lognormal, clipped, rounded UP to whole blocks
    (only full blocks are cached, Sec. 2.1)."""
    rng = np.random.Generator(np.random.PCG64(seed))
    x = rng.lognormal(mean=np.log(median), sigma=sigma, size=n_requests)
    x = np.clip(x, lo, hi)
    return (np.ceil(x / block_size) * block_size).astype(np.int64)


def shared_prefix_tables(seed: int, lengths_tokens: np.ndarray, shared_tokens: int,
                         block_size: int, pool_slack: float
                         ) -> Tuple[int, List[np.ndarray]]:
    """Block tables of concurrent requests whose first ``shared_tokens`` tokens use
    one common list of blocks; the rest of every table is private.  Returns
    (pool_blocks, tables).  A request shorter than the shared prefix uses a
    prefix of the shared list."""
    shared_blocks = shared_tokens // block_size
    lens = [int(t) // block_size for t in lengths_tokens]
    private = [max(0, n - shared_blocks) for n in lens]
    unique = shared_blocks + sum(private)
    pool_blocks = int(np.ceil(unique * pool_slack))
    perm = np.random.Generator(np.random.PCG64(seed)).permutation(pool_blocks).astype(np.int32)
    shared = perm[:shared_blocks]
    tables, cur = [], shared_blocks
    for n, k in zip(lens, private):
        tables.append(np.ascontiguousarray(
            np.concatenate([shared[:min(n, shared_blocks)], perm[cur:cur + k]])))
        cur += k
    return pool_blocks, tables


def batch_workload(w: Workload, scale: float = 1.0):
    """Tables of the many-requests config; ``scale`` < 1 shrinks every length for the
    parity tests (same structure, fewer tokens)."""
    x = w.extra
    toks = lognormal_tokens(w.seed, int(x["requests"]), x["median_tokens"] * scale, x["sigma"],
                            max(w.shape.B, int(x["min_tokens"] * scale)),
                            max(w.shape.B, int(x["max_tokens"] * scale)), w.shape.B)
    shared = max(w.shape.B, int(x["shared_tokens"] * scale) // w.shape.B * w.shape.B)
    return shared_prefix_tables(w.seed + 7, toks, shared, w.shape.B, x["pool_slack"])
