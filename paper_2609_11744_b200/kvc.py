"""ctypes binding of libkvc: one Python function per C entry point, same names.

Only argument marshalling happens here.  Every copy runs in the library's CUDA
kernels; if ``libkvc.so`` has not been built the import of the library fails
with an error -- there is no fallback path of any kind.

Pointers may be given as ints, as torch tensors (their ``data_ptr()``) or as
numpy arrays (host memory).  Streams may be ``None`` (torch's current stream
when torch has a CUDA context, else the default stream), a ``torch.cuda.Stream``
or a raw ``cudaStream_t`` value.
"""
from __future__ import annotations

import ctypes
import os
from typing import List, Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libkvc.so")

KVC_OK, KVC_ERR_INVALID_ARG, KVC_ERR_OUT_OF_RANGE, KVC_ERR_ALIGNMENT, KVC_ERR_CONFLICT, \
    KVC_ERR_NOMEM, KVC_ERR_CUDA, KVC_ERR_WOULD_BLOCK, KVC_ERR_TIMEOUT, KVC_ERR_STATE, \
    KVC_ERR_TOO_LARGE, KVC_ERR_EXISTS, KVC_ERR_NOT_FOUND, KVC_ERR_IO = range(14)
KVC_VARIANT_AUTO, KVC_VARIANT_VEC, KVC_VARIANT_BULK = 0, 1, 2
KVC_ORDER_AUTO, KVC_ORDER_PLANE_MAJOR, KVC_ORDER_BLOCK_MAJOR, KVC_ORDER_CHUNK_MAJOR = 0, 1, 2, 3
KVC_RING_DEVICE, KVC_RING_HOST_MAPPED, KVC_RING_DEVICE_STAGED = 0, 1, 2
KVC_CHUNK_LAYER_MAJOR, KVC_CHUNK_BLOCK_MAJOR = 0, 1
KVC_MAP_FULL_CHUNKS_ONLY = 1
KVC_GROUP_FORCE_KERNEL = 0x100


class KvcError(RuntimeError):
    """A libkvc call returned a status other than KVC_OK."""

    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s: %s (status %d)" % (where, kvc_status_str(status), status))


class kvc_layout_desc(ctypes.Structure):
    _fields_ = [("num_layers", ctypes.c_uint32), ("kv_planes", ctypes.c_uint32),
                ("num_blocks", ctypes.c_uint32), ("block_size", ctypes.c_uint32),
                ("num_kv_heads", ctypes.c_uint32), ("head_dim", ctypes.c_uint32),
                ("elem_bytes", ctypes.c_uint32), ("chunk_tokens", ctypes.c_uint32),
                ("plane_ptrs", ctypes.POINTER(ctypes.c_void_p)), ("base", ctypes.c_void_p),
                ("layer_stride", ctypes.c_uint64), ("plane_stride", ctypes.c_uint64),
                ("block_stride", ctypes.c_uint64), ("chunk_order", ctypes.c_uint32),
                ("reserved", ctypes.c_uint32)]


class kvc_tuning(ctypes.Structure):
    _fields_ = [("variant", ctypes.c_uint32), ("order", ctypes.c_uint32),
                ("max_ctas", ctypes.c_uint32), ("tile_bytes", ctypes.c_uint32),
                ("stages", ctypes.c_uint32), ("ctas_per_sm", ctypes.c_uint32),
                ("l2_hint", ctypes.c_uint32), ("lag", ctypes.c_uint32),
                ("items_per_cta", ctypes.c_uint32), ("pdl", ctypes.c_uint32),
                ("group", ctypes.c_uint32), ("slot_memory", ctypes.c_uint32),
                ("vec_threads", ctypes.c_uint32)]


class kvc_chunk_desc(ctypes.Structure):
    _fields_ = [("request", ctypes.c_uint32), ("chunk", ctypes.c_uint32),
                ("first", ctypes.c_uint32), ("n_blocks", ctypes.c_uint32),
                ("bytes", ctypes.c_uint64)]


class kvc_host_transfer_stats(ctypes.Structure):
    _fields_ = [("bytes", ctypes.c_uint64), ("ring_stalls", ctypes.c_uint64), ("chunks", ctypes.c_uint32),
                ("total_chunks", ctypes.c_uint32)]


class kvc_pipeline_stats(ctypes.Structure):
    _fields_ = [("bytes", ctypes.c_uint64), ("seconds", ctypes.c_double), ("chunks", ctypes.c_uint32),
                ("published", ctypes.c_uint32), ("already_present", ctypes.c_uint32),
                ("ring_stalls", ctypes.c_uint32)]


class kvc_load_request(ctypes.Structure):
    _fields_ = [("ids", ctypes.c_void_p), ("n_blocks", ctypes.c_uint32), ("hashes", ctypes.c_void_p),
                ("n_hashes", ctypes.c_uint32), ("cls", ctypes.c_uint32),
                ("loaded_chunks", ctypes.c_uint32), ("ready_seconds", ctypes.c_double)]


class kvc_load_many_stats(ctypes.Structure):
    _fields_ = [("bytes_read", ctypes.c_uint64), ("seconds", ctypes.c_double)] + \
               [(k, ctypes.c_uint32) for k in ("chunks", "reads", "joins", "claims", "unpack_launches",
                                               "ring_stalls", "preloads_refused")]


class kvc_store_counters(ctypes.Structure):
    _fields_ = [(k, ctypes.c_uint64) for k in ("reads", "read_bytes", "publishes", "publish_bytes")]


class kvc_slot_pool_counters(ctypes.Structure):
    _fields_ = [(k, ctypes.c_uint32) for k in ("n_free", "n_in_flight", "n_staged", "n_retained")] + \
               [(k, ctypes.c_uint64) for k in ("acquires", "joins", "claims", "reclaims", "cancels",
                                               "preload_refusals", "foreground_refusals")]


KVC_CLASS_DEMAND_LOAD, KVC_CLASS_STORE, KVC_CLASS_PRELOAD = 0, 1, 2


# kvc_chunk_op as a numpy record so that thousands of ops can be filled without a Python loop
CHUNK_OP_DTYPE = np.dtype([("slot", np.uint64), ("ids", np.uint64), ("n_blocks", np.uint32),
                           ("reserved", np.uint32)])
assert CHUNK_OP_DTYPE.itemsize == 24

_EVENT_FN = {
    "create": ctypes.CFUNCTYPE(ctypes.c_int, ctypes.c_void_p, ctypes.POINTER(ctypes.c_void_p)),
    "destroy": ctypes.CFUNCTYPE(ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p),
    "record": ctypes.CFUNCTYPE(ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p),
    "query": ctypes.CFUNCTYPE(ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p),
    "stream_wait": ctypes.CFUNCTYPE(ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p),
    "synchronize": ctypes.CFUNCTYPE(ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p),
}


class kvc_event_provider(ctypes.Structure):
    _fields_ = [("ctx", ctypes.c_void_p)] + [(k, v) for k, v in _EVENT_FN.items()]


_lib = None


def lib() -> ctypes.CDLL:
    """The loaded C-ABI library.  Raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            "libkvc.so is missing (%s). Build it with `python -m paper_2609_11744_b200.build`; "
            "there is no fallback implementation." % LIB_PATH)
    L = ctypes.CDLL(LIB_PATH)
    vp, u32, u64, i64, ci = ctypes.c_void_p, ctypes.c_uint32, ctypes.c_uint64, ctypes.c_int64, ctypes.c_int
    P = ctypes.POINTER
    sig = {
        "kvc_status_str": (ctypes.c_char_p, [ci]),
        "kvc_layout_create": (ci, [P(kvc_layout_desc), P(vp)]),
        "kvc_layout_desc_init_dense": (ci, [P(kvc_layout_desc), vp] + [u32] * 9),
        "kvc_layout_destroy": (ci, [vp]),
        "kvc_layout_slab_bytes": (u64, [vp]),
        "kvc_layout_bytes_per_token": (u64, [vp]),
        "kvc_layout_blocks_per_chunk": (u32, [vp]),
        "kvc_layout_chunk_bytes": (u64, [vp, u32]),
        "kvc_layout_num_chunks": (u32, [vp, u32]),
        "kvc_layout_num_blocks": (u32, [vp]),
        "kvc_offload_to_host": (ci, [vp, vp, vp, u32, vp, u64, vp, vp, ctypes.c_int64,
                                     P(kvc_host_transfer_stats)]),
        "kvc_load_from_host": (ci, [vp, vp, vp, u64, vp, u32, vp, vp, ctypes.c_int64,
                                    P(kvc_host_transfer_stats)]),
        "kvc_layout_set_tuning": (ci, [vp, P(kvc_tuning)]),
        "kvc_tuning_preset": (ci, [ci, P(kvc_tuning)]),
        "kvc_map_request": (ci, [vp, u32, u32, P(kvc_chunk_desc), u32, P(u32)]),
        "kvc_map_requests_shared": (ci, [vp, P(vp), P(u32), u32, u32, P(kvc_chunk_desc), u32, P(u32),
                                         P(u64)]),
        "kvc_pack": (ci, [vp, vp, u32, ci, vp, u64, vp]),
        "kvc_unpack": (ci, [vp, vp, u64, vp, u32, ci, vp]),
        "kvc_pack_batch": (ci, [vp, vp, u32, ci, vp]),
        "kvc_unpack_batch": (ci, [vp, vp, u32, ci, vp]),
        "kvc_pack_batch_static": (ci, [vp, vp, u32, vp]),
        "kvc_poll_static_status": (ci, [vp, P(u32), P(u32)]),
        "kvc_pack_copy_engine": (ci, [vp, vp, u32, vp, u64, vp]),
        "kvc_unpack_copy_engine": (ci, [vp, vp, u64, vp, u32, vp]),
        "kvc_poll_device_status": (ci, [vp, vp, P(u32), P(u32)]),
        "kvc_layout_launch_count": (u64, [vp]),
        "kvc_layout_set_kernel_timing": (ci, [vp, ci]),
        "kvc_layout_kernel_time": (ci, [vp, P(u32), P(ctypes.c_double), P(ctypes.c_double),
                                        P(ctypes.c_double)]),
        "kvc_staging_ring_create": (ci, [u64, u32, ci, vp, u64, P(vp)]),
        "kvc_staging_ring_destroy": (ci, [vp]),
        "kvc_staging_ring_acquire": (ci, [vp, i64, P(u32), P(vp), P(vp)]),
        "kvc_staging_ring_commit": (ci, [vp, u32, vp]),
        "kvc_staging_ring_wait_filled": (ci, [vp, u32, vp]),
        "kvc_staging_ring_release": (ci, [vp, u32, vp]),
        "kvc_staging_ring_stats": (ci, [vp, P(u32), P(u64), P(u64)]),
        "kvc_staging_ring_slot_bytes": (u64, [vp]),
        "kvc_staging_ring_num_slots": (u32, [vp]),
        "kvc_staging_ring_set_event_provider": (ci, [P(kvc_event_provider)]),
        "kvc_staging_ring_set_trace": (ci, [vp, vp, u32]),
        "kvc_staging_ring_trace_count": (u32, [vp]),
        "kvc_staging_ring_commit_host": (ci, [vp, u32]),
        "kvc_staging_ring_sync_filled": (ci, [vp, u32]),
        "kvc_staging_ring_release_host": (ci, [vp, u32]),
        "kvc_pipeline_store": (ci, [vp, vp, vp, vp, u32, vp, u32, u32, ci, vp, P(kvc_pipeline_stats)]),
        "kvc_pipeline_load": (ci, [vp, vp, vp, vp, u32, vp, u32, u32, ci, vp, P(kvc_pipeline_stats)]),
        "kvc_pipeline_load_many": (ci, [vp, vp, vp, P(kvc_load_request), u32, u32, vp,
                                        P(kvc_load_many_stats)]),
        "kvc_store_get_counters": (ci, [vp, P(kvc_store_counters)]),
        "kvc_staging_ring_pool_mode": (ci, [vp]),
        "kvc_staging_ring_kind": (ci, [vp]),
        "kvc_slot_pool_create": (ci, [u32, u32, u32, ci, P(vp)]),
        "kvc_slot_pool_destroy": (ci, [vp]),
        "kvc_slot_pool_acquire": (ci, [vp, ci, u64, P(u32), P(ci)]),
        "kvc_slot_pool_mark_staged": (ci, [vp, u32]),
        "kvc_slot_pool_release": (ci, [vp, u32]),
        "kvc_slot_pool_cancel": (ci, [vp, u32]),
        "kvc_slot_pool_get_counters": (ci, [vp, P(kvc_slot_pool_counters)]),
        "kvc_slot_pool_slot_info": (ci, [vp, u32, P(u32), P(u32), P(u64), P(ci)]),
        "kvc_staging_ring_set_policy": (ci, [vp, u32, u32, ci]),
        "kvc_staging_ring_acquire_for": (ci, [vp, ci, u64, i64, P(u32), P(vp), P(vp), P(ci)]),
        "kvc_staging_ring_slot_filled": (ci, [vp, u32, P(ci)]),
        "kvc_staging_ring_cancel": (ci, [vp, u32]),
        "kvc_staging_ring_abandon": (ci, [vp, u32]),
        "kvc_staging_ring_policy_counters": (ci, [vp, P(kvc_slot_pool_counters)]),
        "kvc_store_open": (ci, [ctypes.c_char_p, ctypes.c_char_p, ci, P(vp)]),
        "kvc_store_close": (ci, [vp]),
        "kvc_store_path": (ci, [vp, u64, ctypes.c_char_p, u32]),
        "kvc_store_lookup": (ci, [vp, u64, P(u64)]),
        "kvc_store_publish": (ci, [vp, u64, vp, u64]),
        "kvc_store_read": (ci, [vp, u64, vp, u64]),
        "kvc_store_direct_io_refused": (ci, [vp]),
        "kvc_chain_hash": (u64, [u64, vp, u32]),
        "kvc_fnv1a64": (u64, [vp, u64]),
    }
    for name, (res, args) in sig.items():
        f = getattr(L, name)
        f.restype, f.argtypes = res, args
    _lib = L
    return L


# ------------------------------------------------------------------ marshalling helpers
def _ptr(x) -> int:
    """Address of a torch tensor, numpy array, ctypes object or a plain int."""
    if x is None:
        return 0
    if isinstance(x, int):
        return x
    if hasattr(x, "data_ptr"):
        return int(x.data_ptr())
    if isinstance(x, np.ndarray):
        return int(x.ctypes.data)
    if isinstance(x, ctypes.c_void_p):
        return int(x.value or 0)
    raise TypeError("cannot take the address of %r" % type(x))


def _nbytes(x) -> int:
    if hasattr(x, "data_ptr"):
        return int(x.numel() * x.element_size())
    if isinstance(x, np.ndarray):
        return int(x.nbytes)
    raise TypeError("need an explicit size for %r" % type(x))


_torch_cuda = None  # torch.cuda once it is known to be initialised (per-chunk callers call this a lot)


def _stream(s) -> int:
    global _torch_cuda
    if s is None:
        if _torch_cuda is not None:
            return _torch_cuda.current_stream().cuda_stream
        try:
            import torch
            if torch.cuda.is_available() and torch.cuda.is_initialized():
                _torch_cuda = torch.cuda
                return int(torch.cuda.current_stream().cuda_stream)
        except ImportError:
            pass
        return 0
    if isinstance(s, int):
        return s
    return int(s.cuda_stream)


def _ids(ids) -> Tuple[object, int, int, int]:
    """(keep-alive object, address, count, on_device) of a block-id list.
    Host ids are converted to a contiguous int32 array; a CUDA tensor must already be int32."""
    if type(ids) is np.ndarray and ids.dtype == np.int32 and ids.flags.c_contiguous:
        return ids, ids.ctypes.data, ids.size, 0   # the common case, without a conversion
    if hasattr(ids, "data_ptr"):
        import torch
        if ids.is_cuda:
            if ids.dtype != torch.int32 or not ids.is_contiguous():
                raise TypeError("device-resident block ids must be a contiguous int32 tensor")
            return ids, int(ids.data_ptr()), int(ids.numel()), 1
        ids = ids.numpy()
    a = np.ascontiguousarray(np.asarray(ids, dtype=np.int32))
    return a, int(a.ctypes.data), int(a.size), 0


def _check(status: int, where: str) -> None:
    if status != KVC_OK:
        raise KvcError(status, where)


def kvc_status_str(status: int) -> str:
    return lib().kvc_status_str(int(status)).decode()


# ------------------------------------------------------------------ layout
class LayoutHandle:
    """Owns a ``kvc_layout*``."""

    def __init__(self, handle: int, keep):
        self.handle = handle
        self._keep = keep

    def __del__(self):
        try:
            if self.handle and _lib is not None:
                _lib.kvc_layout_destroy(self.handle)
        except Exception:
            pass
        self.handle = 0


def kvc_layout_create(num_layers: int, kv_planes: int, num_blocks: int, block_size: int,
                      num_kv_heads: int, head_dim: int, elem_bytes: int, chunk_tokens: int,
                      base=None, layer_stride: int = 0, plane_stride: int = 0,
                      block_stride: int = 0, plane_ptrs: Optional[Sequence] = None,
                      chunk_order: int = 0) -> LayoutHandle:
    d = kvc_layout_desc(num_layers, kv_planes, num_blocks, block_size, num_kv_heads, head_dim,
                        elem_bytes, chunk_tokens)
    keep = [base, plane_ptrs]
    if plane_ptrs is not None:
        arr = (ctypes.c_void_p * len(plane_ptrs))(*[_ptr(p) for p in plane_ptrs])
        if len(plane_ptrs) != num_layers * kv_planes:
            raise ValueError("plane_ptrs needs num_layers*kv_planes entries")
        d.plane_ptrs = ctypes.cast(arr, ctypes.POINTER(ctypes.c_void_p))
    else:
        d.base = _ptr(base)
        d.layer_stride, d.plane_stride = layer_stride, plane_stride
    d.block_stride = block_stride
    d.chunk_order = chunk_order
    out = ctypes.c_void_p()
    _check(lib().kvc_layout_create(ctypes.byref(d), ctypes.byref(out)), "kvc_layout_create")
    return LayoutHandle(out.value, keep)


def kvc_layout_create_dense(pool, num_layers, kv_planes, num_blocks, block_size, num_kv_heads,
                            head_dim, elem_bytes, chunk_tokens, chunk_order: int = 0) -> LayoutHandle:
    """Layout over one dense allocation [L][P][NB][B][H][D] (a tensor or a device address):
    kvc_layout_desc_init_dense followed by kvc_layout_create."""
    d = kvc_layout_desc()
    _check(lib().kvc_layout_desc_init_dense(ctypes.byref(d), _ptr(pool), num_layers, kv_planes,
                                            num_blocks, block_size, num_kv_heads, head_dim,
                                            elem_bytes, chunk_tokens, chunk_order),
           "kvc_layout_desc_init_dense")
    out = ctypes.c_void_p()
    _check(lib().kvc_layout_create(ctypes.byref(d), ctypes.byref(out)), "kvc_layout_create")
    return LayoutHandle(out.value, [pool])


def kvc_layout_destroy(layout: LayoutHandle) -> None:
    h, layout.handle = layout.handle, 0
    if h:
        _check(lib().kvc_layout_destroy(h), "kvc_layout_destroy")


def kvc_layout_slab_bytes(layout) -> int:
    return lib().kvc_layout_slab_bytes(layout.handle)


def kvc_layout_bytes_per_token(layout) -> int:
    return lib().kvc_layout_bytes_per_token(layout.handle)


def kvc_layout_blocks_per_chunk(layout) -> int:
    return lib().kvc_layout_blocks_per_chunk(layout.handle)


def kvc_layout_chunk_bytes(layout, n_blocks: int) -> int:
    return lib().kvc_layout_chunk_bytes(layout.handle, n_blocks)


def kvc_layout_num_chunks(layout, n_blocks: int) -> int:
    return lib().kvc_layout_num_chunks(layout.handle, n_blocks)


def kvc_layout_num_blocks(layout) -> int:
    return lib().kvc_layout_num_blocks(layout.handle)


def kvc_layout_set_tuning(layout, variant=0, order=0, max_ctas=0, tile_bytes=0, stages=0,
                          ctas_per_sm=0, l2_hint=0, lag=0, items_per_cta=0, pdl=0, group=0,
                          slot_memory=0, vec_threads=0) -> None:
    t = kvc_tuning(variant, order, max_ctas, tile_bytes, stages, ctas_per_sm, l2_hint, lag,
                   items_per_cta, pdl, group, slot_memory, vec_threads)
    _check(lib().kvc_layout_set_tuning(layout.handle, ctypes.byref(t)), "kvc_layout_set_tuning")


KVC_PRESET_DEFAULT, KVC_PRESET_BESIDE_COMPUTE = 0, 1


def kvc_tuning_preset(which: int) -> dict:
    """The fields of a ready-made tuning, as keyword arguments for kvc_layout_set_tuning."""
    t = kvc_tuning()
    _check(lib().kvc_tuning_preset(which, ctypes.byref(t)), "kvc_tuning_preset")
    return {k: getattr(t, k) for k, _ in kvc_tuning._fields_}


def kvc_layout_launch_count(layout) -> int:
    return lib().kvc_layout_launch_count(layout.handle)


def kvc_layout_set_kernel_timing(layout, on: bool) -> None:
    _check(lib().kvc_layout_set_kernel_timing(layout.handle, int(on)), "kvc_layout_set_kernel_timing")


def kvc_layout_kernel_time(layout) -> Tuple[int, float, float, float]:
    """(launches, total ms, shortest ms, longest ms) of the kernels timed since the last call."""
    n = ctypes.c_uint32()
    t, lo, hi = ctypes.c_double(), ctypes.c_double(), ctypes.c_double()
    _check(lib().kvc_layout_kernel_time(layout.handle, ctypes.byref(n), ctypes.byref(t),
                                        ctypes.byref(lo), ctypes.byref(hi)), "kvc_layout_kernel_time")
    return n.value, t.value, lo.value, hi.value


# ------------------------------------------------------------------ mapper
def _descs(arr, n) -> List[Tuple[int, int, int, int, int]]:
    return [(d.request, d.chunk, d.first, d.n_blocks, d.bytes) for d in arr[:n]]


def kvc_map_request(layout, n_blocks: int, flags: int = 0):
    """[(request, chunk, first, n_blocks, bytes)] for one request."""
    n = ctypes.c_uint32()
    _check(lib().kvc_map_request(layout.handle, n_blocks, flags, None, 0, ctypes.byref(n)),
           "kvc_map_request")
    arr = (kvc_chunk_desc * max(1, n.value))()
    _check(lib().kvc_map_request(layout.handle, n_blocks, flags, arr, n.value, ctypes.byref(n)),
           "kvc_map_request")
    return _descs(arr, n.value)


def kvc_map_requests_shared(layout, tables: Sequence, flags: int = 0):
    """([(request, chunk, first, n_blocks, bytes)], unique_blocks) with shared chunks staged once."""
    tabs = [np.ascontiguousarray(np.asarray(t, dtype=np.int32)) for t in tables]
    nreq = len(tabs)
    ptrs = (ctypes.c_void_p * max(1, nreq))(*[t.ctypes.data for t in tabs])
    lens = (ctypes.c_uint32 * max(1, nreq))(*[t.size for t in tabs])
    n, uniq = ctypes.c_uint32(), ctypes.c_uint64()
    L = lib()
    _check(L.kvc_map_requests_shared(layout.handle, ptrs, lens, nreq, flags, None, 0,
                                     ctypes.byref(n), ctypes.byref(uniq)), "kvc_map_requests_shared")
    arr = (kvc_chunk_desc * max(1, n.value))()
    _check(L.kvc_map_requests_shared(layout.handle, ptrs, lens, nreq, flags, arr, n.value,
                                     ctypes.byref(n), ctypes.byref(uniq)), "kvc_map_requests_shared")
    return _descs(arr, n.value), uniq.value


# ------------------------------------------------------------------ pack / unpack
def kvc_pack(layout, ids, dst_slot, slot_bytes: Optional[int] = None, stream=None) -> None:
    keep, p, n, dev = _ids(ids)
    nb = _nbytes(dst_slot) if slot_bytes is None else slot_bytes
    _check(lib().kvc_pack(layout.handle, p, n, dev, _ptr(dst_slot), nb, _stream(stream)), "kvc_pack")


def kvc_unpack(layout, src_slot, ids, slot_bytes: Optional[int] = None, stream=None) -> None:
    keep, p, n, dev = _ids(ids)
    nb = _nbytes(src_slot) if slot_bytes is None else slot_bytes
    _check(lib().kvc_unpack(layout.handle, _ptr(src_slot), nb, p, n, dev, _stream(stream)),
           "kvc_unpack")


def kvc_pack_copy_engine(layout, ids, dst, dst_bytes: Optional[int] = None, stream=None) -> None:
    """kvc_pack done by the DMA engines (strided async copies); dst may be pinned host memory."""
    keep, p, n, dev = _ids(ids)
    if dev:
        raise TypeError("the copy-engine variants take host-resident ids")
    nb = _nbytes(dst) if dst_bytes is None else dst_bytes
    _check(lib().kvc_pack_copy_engine(layout.handle, p, n, _ptr(dst), nb, _stream(stream)),
           "kvc_pack_copy_engine")


def kvc_unpack_copy_engine(layout, src, ids, src_bytes: Optional[int] = None, stream=None) -> None:
    keep, p, n, dev = _ids(ids)
    if dev:
        raise TypeError("the copy-engine variants take host-resident ids")
    nb = _nbytes(src) if src_bytes is None else src_bytes
    _check(lib().kvc_unpack_copy_engine(layout.handle, _ptr(src), nb, p, n, _stream(stream)),
           "kvc_unpack_copy_engine")


def make_chunk_ops(slot_addrs, ids_addrs, n_blocks) -> np.ndarray:
    """Array of kvc_chunk_op records from three equally long sequences."""
    ops = np.zeros(len(n_blocks), dtype=CHUNK_OP_DTYPE)
    ops["slot"] = np.asarray(slot_addrs, dtype=np.uint64)
    ops["ids"] = np.asarray(ids_addrs, dtype=np.uint64)
    ops["n_blocks"] = np.asarray(n_blocks, dtype=np.uint32)
    return ops


def request_chunk_ops(layout, ids, staging, flags: int = 0):
    """Ops that move one request's chunks to/from a staging area where the chunks lie back to
    back in request order.  Returns (ops, keep_alive, total_bytes, ids_on_device)."""
    keep, p, n, dev = _ids(ids)
    descs = kvc_map_request(layout, n, flags)
    nb = np.array([d[3] for d in descs], dtype=np.uint64)
    first = np.array([d[2] for d in descs], dtype=np.uint64)
    sizes = np.array([d[4] for d in descs], dtype=np.uint64)
    offs = np.concatenate([[0], np.cumsum(sizes)[:-1]]).astype(np.uint64) if len(descs) else sizes
    ops = make_chunk_ops(np.uint64(_ptr(staging)) + offs, np.uint64(p) + first * np.uint64(4), nb)
    return ops, keep, int(sizes.sum()), dev


def _batch(fn_name: str, layout, ops: np.ndarray, ids_on_device: int, stream) -> None:
    if ops.dtype != CHUNK_OP_DTYPE or not ops.flags.c_contiguous:
        raise TypeError("ops must be a contiguous array of CHUNK_OP_DTYPE")
    fn = getattr(lib(), fn_name)
    _check(fn(layout.handle, ops.ctypes.data, len(ops), int(ids_on_device), _stream(stream)), fn_name)


def kvc_pack_batch(layout, ops: np.ndarray, ids_on_device: int = 0, stream=None) -> None:
    _batch("kvc_pack_batch", layout, ops, ids_on_device, stream)


def kvc_unpack_batch(layout, ops: np.ndarray, ids_on_device: int = 0, stream=None) -> None:
    _batch("kvc_unpack_batch", layout, ops, ids_on_device, stream)


KVC_STATIC_MAX_BLOCKS, KVC_STATIC_MAX_PLANES = 8192, 1024


def kvc_pack_batch_static(layout, ops: np.ndarray, stream=None) -> None:
    """kvc_pack_batch for callers that must not allocate device memory (an engine whose KV pool
    already owns all of it, a thread that cannot tolerate an allocation's stall).  Host-resident
    ids only, at most KVC_STATIC_MAX_BLOCKS blocks per call; calls share one fixed scratch area
    inside the library, so keep them on one stream."""
    if ops.dtype != CHUNK_OP_DTYPE or not ops.flags.c_contiguous:
        raise TypeError("ops must be a contiguous array of CHUNK_OP_DTYPE")
    _check(lib().kvc_pack_batch_static(layout.handle, ops.ctypes.data, len(ops), _stream(stream)),
           "kvc_pack_batch_static")


def kvc_poll_static_status(stream=None) -> Tuple[int, int]:
    """kvc_poll_device_status for the kvc_pack_batch_static path of the current device."""
    a, b = ctypes.c_uint32(), ctypes.c_uint32()
    _check(lib().kvc_poll_static_status(_stream(stream), ctypes.byref(a), ctypes.byref(b)),
           "kvc_poll_static_status")
    return a.value, b.value


def kvc_poll_device_status(layout, stream=None) -> Tuple[int, int]:
    """(blocks skipped for a bad device-resident id, in-kernel waits that gave up), then clears."""
    a, b = ctypes.c_uint32(), ctypes.c_uint32()
    _check(lib().kvc_poll_device_status(layout.handle, _stream(stream), ctypes.byref(a),
                                        ctypes.byref(b)), "kvc_poll_device_status")
    return a.value, b.value


# ------------------------------------------------------------------ staging ring
class RingHandle:
    """Owns a ``kvc_ring*``."""

    def __init__(self, handle: int, keep):
        self.handle = handle
        self._keep = keep

    def __del__(self):
        try:
            if self.handle and _lib is not None:
                _lib.kvc_staging_ring_destroy(self.handle)
        except Exception:
            pass
        self.handle = 0


def kvc_staging_ring_create(slot_bytes: int, n_slots: int, kind: int = KVC_RING_DEVICE, mem=None,
                            mem_bytes: Optional[int] = None) -> RingHandle:
    out = ctypes.c_void_p()
    mb = 0 if mem is None else (_nbytes(mem) if mem_bytes is None else mem_bytes)
    _check(lib().kvc_staging_ring_create(slot_bytes, n_slots, kind, _ptr(mem), mb, ctypes.byref(out)),
           "kvc_staging_ring_create")
    return RingHandle(out.value, mem)


def kvc_staging_ring_destroy(ring: RingHandle) -> None:
    h, ring.handle = ring.handle, 0
    if h:
        _check(lib().kvc_staging_ring_destroy(h), "kvc_staging_ring_destroy")


def kvc_staging_ring_acquire(ring, timeout_us: int = 0) -> Tuple[int, int, int]:
    """(slot index, device address, host address or 0).  Raises KvcError(WOULD_BLOCK/TIMEOUT)."""
    slot, dp, hp = ctypes.c_uint32(), ctypes.c_void_p(), ctypes.c_void_p()
    _check(lib().kvc_staging_ring_acquire(ring.handle, timeout_us, ctypes.byref(slot),
                                          ctypes.byref(dp), ctypes.byref(hp)),
           "kvc_staging_ring_acquire")
    return slot.value, int(dp.value or 0), int(hp.value or 0)


def kvc_staging_ring_commit(ring, slot: int, producer_stream=None) -> None:
    _check(lib().kvc_staging_ring_commit(ring.handle, slot, _stream(producer_stream)),
           "kvc_staging_ring_commit")


def kvc_staging_ring_wait_filled(ring, slot: int, consumer_stream=None) -> None:
    _check(lib().kvc_staging_ring_wait_filled(ring.handle, slot, _stream(consumer_stream)),
           "kvc_staging_ring_wait_filled")


def kvc_staging_ring_release(ring, slot: int, consumer_stream=None) -> None:
    _check(lib().kvc_staging_ring_release(ring.handle, slot, _stream(consumer_stream)),
           "kvc_staging_ring_release")


def kvc_staging_ring_stats(ring) -> Tuple[int, int, int]:
    """(in_flight, acquires, stalls)."""
    a, b, c = ctypes.c_uint32(), ctypes.c_uint64(), ctypes.c_uint64()
    _check(lib().kvc_staging_ring_stats(ring.handle, ctypes.byref(a), ctypes.byref(b),
                                        ctypes.byref(c)), "kvc_staging_ring_stats")
    return a.value, b.value, c.value


def kvc_staging_ring_slot_bytes(ring) -> int:
    return lib().kvc_staging_ring_slot_bytes(ring.handle)


def kvc_staging_ring_num_slots(ring) -> int:
    return lib().kvc_staging_ring_num_slots(ring.handle)


_provider_keep = []   # rings copy the provider when they are created: its callbacks must outlive them


def kvc_staging_ring_set_event_provider(provider: Optional[dict]) -> None:
    """Install callables {create, destroy, record, query, stream_wait, synchronize} (each
    taking the C callback's arguments, ctx first), or None for CUDA events.  Used by
    host-only tests."""
    global _provider_keep
    if provider is None:
        _check(lib().kvc_staging_ring_set_event_provider(None), "kvc_staging_ring_set_event_provider")
        _provider_keep = []   # rings copy the provider when they are created: its callbacks must outlive them
        return
    p = kvc_event_provider()
    fns = {}
    for name, ftype in _EVENT_FN.items():
        fns[name] = ftype(provider[name])
        setattr(p, name, fns[name])
    _check(lib().kvc_staging_ring_set_event_provider(ctypes.byref(p)),
           "kvc_staging_ring_set_event_provider")
    _provider_keep.append((p, fns))


# ------------------------------------------------------------------ chunk files
class StoreHandle:
    """Owns a ``kvc_store*``."""

    def __init__(self, handle: int):
        self.handle = handle

    def __del__(self):
        try:
            if self.handle and _lib is not None:
                _lib.kvc_store_close(self.handle)
        except Exception:
            pass
        self.handle = 0


def kvc_store_open(root: str, model_tag: str, direct_io: bool = True) -> StoreHandle:
    out = ctypes.c_void_p()
    _check(lib().kvc_store_open(root.encode(), model_tag.encode(), int(direct_io), ctypes.byref(out)),
           "kvc_store_open")
    return StoreHandle(out.value)


def kvc_store_close(store: StoreHandle) -> None:
    h, store.handle = store.handle, 0
    if h:
        _check(lib().kvc_store_close(h), "kvc_store_close")


def kvc_store_path(store, hash64: int) -> str:
    buf = ctypes.create_string_buffer(4096)
    _check(lib().kvc_store_path(store.handle, hash64, buf, 4096), "kvc_store_path")
    return buf.value.decode()


def kvc_store_lookup(store, hash64: int) -> Optional[int]:
    """Size of the entry in bytes, or None if it is not published."""
    n = ctypes.c_uint64()
    st = lib().kvc_store_lookup(store.handle, hash64, ctypes.byref(n))
    if st == KVC_ERR_NOT_FOUND:
        return None
    _check(st, "kvc_store_lookup")
    return n.value


def kvc_store_publish(store, hash64: int, host_buf, nbytes: Optional[int] = None) -> bool:
    """True if this call published the entry, False if another writer already had."""
    nb = _nbytes(host_buf) if nbytes is None else nbytes
    st = lib().kvc_store_publish(store.handle, hash64, _ptr(host_buf), nb)
    if st == KVC_ERR_EXISTS:
        return False
    _check(st, "kvc_store_publish")
    return True


def kvc_store_read(store, hash64: int, host_buf, nbytes: Optional[int] = None) -> None:
    nb = _nbytes(host_buf) if nbytes is None else nbytes
    _check(lib().kvc_store_read(store.handle, hash64, _ptr(host_buf), nb), "kvc_store_read")


def kvc_store_direct_io_refused(store) -> int:
    return lib().kvc_store_direct_io_refused(store.handle)


_OPEN_FN = ctypes.CFUNCTYPE(ctypes.c_int, ctypes.c_char_p, ctypes.c_int, ctypes.c_uint, use_errno=True)
_open_keep = None


def kvc_store_set_open_fn(fn) -> None:
    """Test seam: route every open() of the store through fn(path: bytes, flags, mode) -> fd or -1
    (set errno with ctypes.set_errno before returning -1); None restores open(2)."""
    global _open_keep
    L = lib()
    L.kvc_store_set_open_fn.argtypes = [_OPEN_FN]
    L.kvc_store_set_open_fn.restype = ctypes.c_int
    cb = ctypes.cast(None, _OPEN_FN) if fn is None else _OPEN_FN(fn)
    _check(L.kvc_store_set_open_fn(cb), "kvc_store_set_open_fn")
    _open_keep = None if fn is None else cb


def kvc_chain_hash(prev: int, tokens) -> int:
    t = np.ascontiguousarray(np.asarray(tokens, dtype=np.int32))
    return lib().kvc_chain_hash(prev, t.ctypes.data, t.size)


def kvc_fnv1a64(data: bytes) -> int:
    return lib().kvc_fnv1a64(ctypes.c_char_p(data), len(data))


def kvc_staging_ring_commit_host(ring, slot: int) -> None:
    _check(lib().kvc_staging_ring_commit_host(ring.handle, slot), "kvc_staging_ring_commit_host")


def kvc_staging_ring_sync_filled(ring, slot: int) -> None:
    _check(lib().kvc_staging_ring_sync_filled(ring.handle, slot), "kvc_staging_ring_sync_filled")


def kvc_staging_ring_release_host(ring, slot: int) -> None:
    _check(lib().kvc_staging_ring_release_host(ring.handle, slot), "kvc_staging_ring_release_host")


def _pipeline(fn_name, layout, ring, store, ids, hashes, io_threads, use_copy_engine, stream):
    keep, p, n, dev = _ids(ids)
    if dev:
        raise TypeError("the pipelines take host-resident ids")
    hs = np.ascontiguousarray(np.asarray(hashes, dtype=np.uint64))
    stats = kvc_pipeline_stats()
    st = getattr(lib(), fn_name)(layout.handle, ring.handle, store.handle, p, n, hs.ctypes.data,
                                 hs.size, io_threads, int(use_copy_engine), _stream(stream),
                                 ctypes.byref(stats))
    _check(st, fn_name)
    return {k: getattr(stats, k) for k, _ in kvc_pipeline_stats._fields_}


def _host_transfer(fn_name: str, layout, ring, ids, host, host_bytes, kernel_stream, copy_stream,
                   slot_timeout_us: int) -> dict:
    keep, p, n, dev = _ids(ids)
    if dev:
        raise TypeError("the host transfers take host-resident ids")
    nb = _nbytes(host) if host_bytes is None else host_bytes
    ks = _stream(kernel_stream)
    cs = ks if copy_stream is None else _stream(copy_stream)
    stats = kvc_host_transfer_stats()
    if fn_name == "kvc_offload_to_host":
        st = lib().kvc_offload_to_host(layout.handle, ring.handle, p, n, _ptr(host), nb, ks, cs,
                                       int(slot_timeout_us), ctypes.byref(stats))
    else:
        st = lib().kvc_load_from_host(layout.handle, ring.handle, _ptr(host), nb, p, n, ks, cs,
                                      int(slot_timeout_us), ctypes.byref(stats))
    _check(st, fn_name)
    return {k: getattr(stats, k) for k, _ in kvc_host_transfer_stats._fields_}


def kvc_offload_to_host(layout, ring, ids, host_dst, host_bytes: Optional[int] = None, kernel_stream=None,
                        copy_stream=None, slot_timeout_us: int = 10_000_000) -> dict:
    """Pack a request chunk by chunk through the ring into a (pinned) host buffer; returns the stats.
    copy_stream None = the kernel stream.  Synchronise the copy stream before reading the buffer."""
    return _host_transfer("kvc_offload_to_host", layout, ring, ids, host_dst, host_bytes, kernel_stream,
                          copy_stream, slot_timeout_us)


def kvc_load_from_host(layout, ring, host_src, ids, host_bytes: Optional[int] = None, kernel_stream=None,
                       copy_stream=None, slot_timeout_us: int = 10_000_000) -> dict:
    """The reverse: host buffer -> ring slots -> unpack into ids.  Synchronise the kernel stream."""
    return _host_transfer("kvc_load_from_host", layout, ring, ids, host_src, host_bytes, kernel_stream,
                          copy_stream, slot_timeout_us)


def kvc_pipeline_store(layout, ring, store, ids, hashes, io_threads: int = 0,
                       use_copy_engine: bool = False, stream=None) -> dict:
    """Offload a request to chunk files through a mapped-host ring; returns the stats as a dict."""
    return _pipeline("kvc_pipeline_store", layout, ring, store, ids, hashes, io_threads,
                     use_copy_engine, stream)


def kvc_pipeline_load(layout, ring, store, ids, hashes, io_threads: int = 0,
                      use_copy_engine: bool = False, stream=None) -> dict:
    """Load the present prefix of a request's chunks from files; synchronise the stream afterwards."""
    return _pipeline("kvc_pipeline_load", layout, ring, store, ids, hashes, io_threads,
                     use_copy_engine, stream)


def kvc_pipeline_load_many(layout, ring, store, requests: Sequence[dict], io_threads: int = 0,
                           stream=None) -> Tuple[dict, List[dict]]:
    """Serve several requests at once from a ring in pool mode.  Each request is a dict with
    'hashes', 'cls' (KVC_CLASS_DEMAND_LOAD / KVC_CLASS_PRELOAD) and, for demand loads, 'ids'
    (a preload gives 'n_blocks' instead).  Returns (stats, [{'loaded_chunks', 'ready_seconds'}])."""
    n = len(requests)
    arr = (kvc_load_request * max(1, n))()
    keep = []
    for i, q in enumerate(requests):
        hs = np.ascontiguousarray(np.asarray(q["hashes"], dtype=np.uint64))
        keep.append(hs)
        arr[i].hashes, arr[i].n_hashes, arr[i].cls = hs.ctypes.data, hs.size, int(q["cls"])
        if q.get("ids") is not None:
            k, p, cnt, dev = _ids(q["ids"])
            if dev:
                raise TypeError("the pipelines take host-resident ids")
            keep.append(k)
            arr[i].ids, arr[i].n_blocks = p, cnt
        else:
            arr[i].ids, arr[i].n_blocks = None, int(q["n_blocks"])
    stats = kvc_load_many_stats()
    st = lib().kvc_pipeline_load_many(layout.handle, ring.handle, store.handle, arr, n, io_threads,
                                      _stream(stream), ctypes.byref(stats))
    _check(st, "kvc_pipeline_load_many")
    return ({k: getattr(stats, k) for k, _ in kvc_load_many_stats._fields_},
            [{"loaded_chunks": arr[i].loaded_chunks, "ready_seconds": arr[i].ready_seconds}
             for i in range(n)])


def kvc_store_get_counters(store) -> dict:
    c = kvc_store_counters()
    _check(lib().kvc_store_get_counters(store.handle, ctypes.byref(c)), "kvc_store_get_counters")
    return {k: getattr(c, k) for k, _ in kvc_store_counters._fields_}


def kvc_staging_ring_pool_mode(ring) -> bool:
    return bool(lib().kvc_staging_ring_pool_mode(ring.handle))


def kvc_staging_ring_kind(ring) -> int:
    return lib().kvc_staging_ring_kind(ring.handle)


# ------------------------------------------------------------------ slot policy
class SlotPoolHandle:
    """Owns a ``kvc_slot_pool*``."""

    def __init__(self, handle: int):
        self.handle = handle

    def __del__(self):
        try:
            if self.handle and _lib is not None:
                _lib.kvc_slot_pool_destroy(self.handle)
        except Exception:
            pass
        self.handle = 0


def kvc_slot_pool_create(n_slots: int, foreground_reserve: int, max_speculative: int = 1,
                         retain_completed: bool = False) -> SlotPoolHandle:
    out = ctypes.c_void_p()
    _check(lib().kvc_slot_pool_create(n_slots, foreground_reserve, max_speculative,
                                      int(retain_completed), ctypes.byref(out)), "kvc_slot_pool_create")
    return SlotPoolHandle(out.value)


def kvc_slot_pool_destroy(pool: SlotPoolHandle) -> None:
    h, pool.handle = pool.handle, 0
    if h:
        _check(lib().kvc_slot_pool_destroy(h), "kvc_slot_pool_destroy")


def kvc_slot_pool_acquire(pool, cls: int, key: int) -> Optional[Tuple[int, bool]]:
    """(slot, joined), or None when nothing is available for this class right now."""
    slot, joined = ctypes.c_uint32(), ctypes.c_int()
    st = lib().kvc_slot_pool_acquire(pool.handle, cls, key, ctypes.byref(slot), ctypes.byref(joined))
    if st == KVC_ERR_WOULD_BLOCK:
        return None
    _check(st, "kvc_slot_pool_acquire")
    return slot.value, bool(joined.value)


def kvc_slot_pool_mark_staged(pool, slot: int) -> None:
    _check(lib().kvc_slot_pool_mark_staged(pool.handle, slot), "kvc_slot_pool_mark_staged")


def kvc_slot_pool_release(pool, slot: int) -> None:
    _check(lib().kvc_slot_pool_release(pool.handle, slot), "kvc_slot_pool_release")


def kvc_slot_pool_cancel(pool, slot: int) -> None:
    _check(lib().kvc_slot_pool_cancel(pool.handle, slot), "kvc_slot_pool_cancel")


def kvc_slot_pool_get_counters(pool) -> dict:
    c = kvc_slot_pool_counters()
    _check(lib().kvc_slot_pool_get_counters(pool.handle, ctypes.byref(c)), "kvc_slot_pool_get_counters")
    return {k: getattr(c, k) for k, _ in kvc_slot_pool_counters._fields_}


KVC_SLOT_FREE, KVC_SLOT_IN_FLIGHT, KVC_SLOT_STAGED, KVC_SLOT_RETAINED = 0, 1, 2, 3


def kvc_slot_pool_slot_info(pool, slot: int) -> Tuple[int, int, int, bool]:
    """(state, references, key, unclaimed preload?) of one slot."""
    st, refs, key, spec = ctypes.c_uint32(), ctypes.c_uint32(), ctypes.c_uint64(), ctypes.c_int()
    _check(lib().kvc_slot_pool_slot_info(pool.handle, slot, ctypes.byref(st), ctypes.byref(refs),
                                         ctypes.byref(key), ctypes.byref(spec)), "kvc_slot_pool_slot_info")
    return st.value, refs.value, key.value, bool(spec.value)


# ------------------------------------------------------------------ staging pool mode
def kvc_staging_ring_set_policy(ring, foreground_reserve: int, max_speculative: int = 1,
                                retain_completed: bool = False) -> None:
    _check(lib().kvc_staging_ring_set_policy(ring.handle, foreground_reserve, max_speculative,
                                             int(retain_completed)), "kvc_staging_ring_set_policy")


def kvc_staging_ring_acquire_for(ring, cls: int, key: int, timeout_us: int = 0):
    """(slot, device address, host address or 0, joined), or None when nothing is available for
    this class (timeout_us == 0).  Raises KvcError(TIMEOUT) after a positive timeout."""
    slot, dp, hp, j = ctypes.c_uint32(), ctypes.c_void_p(), ctypes.c_void_p(), ctypes.c_int()
    st = lib().kvc_staging_ring_acquire_for(ring.handle, cls, key, timeout_us, ctypes.byref(slot),
                                            ctypes.byref(dp), ctypes.byref(hp), ctypes.byref(j))
    if st == KVC_ERR_WOULD_BLOCK:
        return None
    _check(st, "kvc_staging_ring_acquire_for")
    return slot.value, int(dp.value or 0), int(hp.value or 0), bool(j.value)


def kvc_staging_ring_slot_filled(ring, slot: int) -> bool:
    f = ctypes.c_int()
    _check(lib().kvc_staging_ring_slot_filled(ring.handle, slot, ctypes.byref(f)),
           "kvc_staging_ring_slot_filled")
    return bool(f.value)


def kvc_staging_ring_cancel(ring, slot: int) -> None:
    _check(lib().kvc_staging_ring_cancel(ring.handle, slot), "kvc_staging_ring_cancel")


def kvc_staging_ring_abandon(ring, slot: int) -> None:
    _check(lib().kvc_staging_ring_abandon(ring.handle, slot), "kvc_staging_ring_abandon")


def kvc_staging_ring_policy_counters(ring) -> dict:
    c = kvc_slot_pool_counters()
    _check(lib().kvc_staging_ring_policy_counters(ring.handle, ctypes.byref(c)),
           "kvc_staging_ring_policy_counters")
    return {k: getattr(c, k) for k, _ in kvc_slot_pool_counters._fields_}


RING_TRACE_DTYPE = np.dtype([("t_ns", np.uint64), ("slot", np.uint32), ("what", np.uint32)])
KVC_TRACE_ACQUIRE, KVC_TRACE_COMMIT, KVC_TRACE_RELEASE, KVC_TRACE_STALL = 0, 1, 2, 3


def kvc_staging_ring_set_trace(ring, capacity: int) -> Optional[np.ndarray]:
    """Start logging slot transitions into a new array of RING_TRACE_DTYPE (returned; it is kept
    alive by the ring handle), or stop logging with capacity 0."""
    if capacity <= 0:
        _check(lib().kvc_staging_ring_set_trace(ring.handle, None, 0), "kvc_staging_ring_set_trace")
        ring._trace = None
        return None
    buf = np.zeros(capacity, dtype=RING_TRACE_DTYPE)
    _check(lib().kvc_staging_ring_set_trace(ring.handle, buf.ctypes.data, capacity),
           "kvc_staging_ring_set_trace")
    ring._trace = buf
    return buf


def kvc_staging_ring_trace_count(ring) -> int:
    return lib().kvc_staging_ring_trace_count(ring.handle)
