"""Host-side checks that need no GPU: the library loads, exports what the header declares,
validates arguments before any CUDA call, and the mapper / ring state machine behave."""
import ctypes
import os
import re

import numpy as np
import pytest

from oracle import oracle as orc
from paper_2609_11744_b200 import kvc
import workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _layout(chunk_tokens=64, NB=32, base=0x10000, **kw):
    args = dict(num_layers=2, kv_planes=2, num_blocks=NB, block_size=16, num_kv_heads=4,
                head_dim=64, elem_bytes=2, chunk_tokens=chunk_tokens)
    args.update(kw)
    if "plane_ptrs" in args:
        return kvc.kvc_layout_create(**args)
    return kvc.kvc_layout_create_dense(base, *[args[k] for k in (
        "num_layers", "kv_planes", "num_blocks", "block_size", "num_kv_heads", "head_dim",
        "elem_bytes", "chunk_tokens")])


def test_library_exports_every_declared_symbol():
    text = open(os.path.join(ROOT, "include", "kvc.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    declared = set(re.findall(r"\b(kvc_[a-z0-9_]+)\s*\(", text))
    declared -= {"kvc_status"}
    assert len(declared) >= 25
    L = kvc.lib()
    for name in sorted(declared):
        assert hasattr(L, name), name
    assert kvc.kvc_status_str(kvc.KVC_OK) == "ok"
    assert all(kvc.kvc_status_str(i) for i in range(10))


def test_layout_sizes_and_mapper_match_paper_numbers():
    # Llama-3.2-3B shape (Sec. 2.1: 112 KiB per token; Sec. 6.4: ~28 MiB per 256-token block)
    lay = kvc.kvc_layout_create_dense(0x100000, 28, 2, 1000, 16, 8, 128, 2, 256)
    assert kvc.kvc_layout_bytes_per_token(lay) == 114688
    assert kvc.kvc_layout_slab_bytes(lay) == 32768
    assert kvc.kvc_layout_blocks_per_chunk(lay) == 16
    assert kvc.kvc_layout_chunk_bytes(lay, 16) == 28 * 2**20
    assert kvc.kvc_layout_bytes_per_token(lay) * 81920 == int(8.75 * 2**30)
    assert kvc.kvc_layout_num_chunks(lay, 5000) == 313
    d = kvc.kvc_map_request(lay, 5000)
    assert len(d) == 313 and d[-1] == (0, 312, 4992, 8, 8 * 28 * 2 * 32768)
    assert len(kvc.kvc_map_request(lay, 5000, kvc.KVC_MAP_FULL_CHUNKS_ONLY)) == 312
    assert kvc.kvc_map_request(lay, 0) == []
    kvc.kvc_layout_destroy(lay)


@pytest.mark.parametrize("n,chunk_tokens", [(64, 256), (5000, 16), (5000, 2048), (3, 256), (129, 2048)])
def test_mapper_matches_oracle_ranges(n, chunk_tokens):
    lay = _layout(chunk_tokens=chunk_tokens, NB=8192)
    g = orc.Dims(2, 2, 8192, 16, 4, 64, 2)
    want = orc.chunk_ranges(n, chunk_tokens // 16)
    got = kvc.kvc_map_request(lay, n)
    assert [(f, nb) for _, _, f, nb, _ in got] == want
    assert [b for *_, b in got] == [orc.chunk_bytes(g, nb) for _, nb in want]
    assert [c for _, c, *_ in got] == list(range(len(want)))


def test_shared_prefix_mapper_matches_bruteforce():
    lay = _layout(chunk_tokens=32, NB=4096)   # 2 blocks per chunk
    shared = [10, 11, 12, 13]
    cases = [
        [shared + [20, 21, 22], shared + [30], shared[:2], shared + [20, 21, 22]],
        [[1, 2, 3, 4], [9, 2, 3, 4]],
        [[1, 2, 3], [1, 2, 3, 4]],
        [[5], [5], [5, 6], []],
        [[1, 2, 3, 4, 5], [1, 2, 3, 9, 9], [1, 2, 3]],
    ]
    rng = np.random.default_rng(0)
    for _ in range(30):   # random forests of tables with common prefixes
        root = rng.permutation(200)[:12].tolist()
        tabs = []
        for _ in range(int(rng.integers(1, 7))):
            k = int(rng.integers(0, 13))
            tabs.append(root[:k] + rng.integers(200, 400, int(rng.integers(0, 6))).tolist())
        cases.append(tabs)
    for tabs in cases:
        got, uniq = kvc.kvc_map_requests_shared(lay, tabs)
        want = orc.dedup_ops(tabs, 2)
        assert [(r, c, f, nb) for r, c, f, nb, _ in got] == want, tabs
        keys = {tuple(t[:i + 1]) for t in tabs for i in range(len(t))}
        assert uniq == len(keys)


def test_shared_prefix_mapper_on_batch_workload():
    w = wl.WORKLOADS["70b_batch"]
    nb_pool, tables = wl.batch_workload(w, scale=1 / 16)
    lay = kvc.kvc_layout_create_dense(0x100000, 80, 2, nb_pool, 16, 8, 128, 2, 256 // 16 * 16 // 16 * 16)
    got, uniq = kvc.kvc_map_requests_shared(lay, tables)
    want = orc.dedup_ops([t.tolist() for t in tables], kvc.kvc_layout_blocks_per_chunk(lay))
    assert [(r, c, f, nb) for r, c, f, nb, _ in got] == want
    assert uniq == len({int(b) for t in tables for b in t})
    assert uniq < sum(len(t) for t in tables)


def test_create_rejects_bad_descriptors():
    def status(**kw):
        with pytest.raises(kvc.KvcError) as e:
            _layout(**kw)
        return e.value.status
    assert status(chunk_tokens=24) == kvc.KVC_ERR_INVALID_ARG          # not a multiple of block_size
    assert status(elem_bytes=3) == kvc.KVC_ERR_INVALID_ARG
    assert status(num_layers=0) == kvc.KVC_ERR_INVALID_ARG
    assert status(base=0) == kvc.KVC_ERR_INVALID_ARG
    assert status(base=0x10008) == kvc.KVC_ERR_ALIGNMENT
    assert status(num_kv_heads=1, head_dim=1, block_size=4, chunk_tokens=4) == kvc.KVC_ERR_ALIGNMENT
    with pytest.raises(kvc.KvcError) as e:   # block stride smaller than a slab
        kvc.kvc_layout_create(2, 2, 8, 16, 4, 64, 2, 64, base=0x10000, layer_stride=1 << 20,
                              plane_stride=1 << 19, block_stride=4096)
    assert e.value.status == kvc.KVC_ERR_INVALID_ARG
    with pytest.raises(kvc.KvcError) as e:   # planes overlap
        kvc.kvc_layout_create(2, 2, 8, 16, 4, 64, 2, 64, base=0x10000, layer_stride=1 << 20,
                              plane_stride=4096)
    assert e.value.status == kvc.KVC_ERR_INVALID_ARG
    with pytest.raises(kvc.KvcError) as e:
        kvc.kvc_layout_create(1, 2, 8, 16, 4, 64, 2, 64, plane_ptrs=[0x10000, 0x20004])
    assert e.value.status == kvc.KVC_ERR_ALIGNMENT


def test_pack_unpack_validate_before_any_launch():
    """Bad arguments are refused on the host; nothing reaches CUDA (there is no GPU here anyway)."""
    lay = _layout(chunk_tokens=64, NB=32)
    chunk = kvc.kvc_layout_chunk_bytes(lay, 4)
    slot = 0x7f0000000000
    def st(fn, *a, **k):
        with pytest.raises(kvc.KvcError) as e:
            fn(*a, **k)
        return e.value.status
    assert st(kvc.kvc_pack, lay, [0, 1, 32, 3], slot, chunk) == kvc.KVC_ERR_OUT_OF_RANGE
    assert st(kvc.kvc_pack, lay, [0, -1], slot, chunk) == kvc.KVC_ERR_OUT_OF_RANGE
    assert st(kvc.kvc_pack, lay, [0, 1, 2, 3], slot, chunk - 1) == kvc.KVC_ERR_INVALID_ARG
    assert st(kvc.kvc_pack, lay, [0, 1, 2, 3], slot + 8, chunk) == kvc.KVC_ERR_ALIGNMENT
    assert st(kvc.kvc_unpack, lay, slot, [5, 6, 5], chunk) == kvc.KVC_ERR_CONFLICT
    assert st(kvc.kvc_unpack, lay, slot, [99], chunk) == kvc.KVC_ERR_OUT_OF_RANGE
    kvc.kvc_pack(lay, [], slot, 0)            # empty chunk: a no-op that succeeds
    kvc.kvc_unpack(lay, slot, [], 0)
    ids = np.array([1, 2, 3, 4, 2], dtype=np.int32)
    ops = kvc.make_chunk_ops([slot, slot + chunk], [ids.ctypes.data, ids.ctypes.data + 12], [3, 2])
    assert st(kvc.kvc_unpack_batch, lay, ops) == kvc.KVC_ERR_CONFLICT      # id 2 in two ops
    ops["reserved"][0] = 1
    assert st(kvc.kvc_pack_batch, lay, ops) == kvc.KVC_ERR_INVALID_ARG
    kvc.kvc_pack_batch(lay, ops[:0])          # no ops: no-op
    assert kvc.kvc_layout_launch_count(lay) == 0
    assert kvc.kvc_poll_device_status(lay) == (0, 0)


def test_set_tuning_validation():
    lay = _layout()
    kvc.kvc_layout_set_tuning(lay, variant=kvc.KVC_VARIANT_VEC, max_ctas=8, tile_bytes=8192)
    for bad in (dict(variant=3), dict(order=4), dict(tile_bytes=24), dict(stages=1), dict(stages=99)):
        with pytest.raises(kvc.KvcError):
            kvc.kvc_layout_set_tuning(lay, **bad)


def test_tuning_presets():
    assert not any(kvc.kvc_tuning_preset(kvc.KVC_PRESET_DEFAULT).values())
    p = kvc.kvc_tuning_preset(kvc.KVC_PRESET_BESIDE_COMPUTE)
    assert (p["max_ctas"], p["tile_bytes"], p["stages"]) == (16, 8192, 2)
    lay = _layout()
    kvc.kvc_layout_set_tuning(lay, **p)              # a preset is a valid tuning
    with pytest.raises(kvc.KvcError):
        kvc.kvc_tuning_preset(7)


def test_product_never_imports_the_oracle():
    pkg = os.path.join(ROOT, "paper_2609_11744_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".h", ".cpp")):
                assert "oracle" not in open(os.path.join(dirpath, f)).read().lower(), f


# ------------------------------------------------------------------ ring state machine with fake events
class FakeEvents:
    """Events that complete only when the test says so."""

    def __init__(self):
        self.done = {}
        self.recorded = []
        self.next = 1

    def provider(self):
        def create(ctx, out):
            out[0] = self.next
            self.done[self.next] = True
            self.next += 1
            return 0
        def destroy(ctx, ev):
            self.done.pop(ev, None)
            return 0
        def record(ctx, ev, stream):
            self.done[ev] = False
            self.recorded.append((ev, stream))
            return 0
        def query(ctx, ev):
            return 0 if self.done[ev] else 1
        def stream_wait(ctx, stream, ev):
            return 0
        def synchronize(ctx, ev):
            self.done[ev] = True
            return 0
        return dict(create=create, destroy=destroy, record=record, query=query,
                    stream_wait=stream_wait, synchronize=synchronize)

    def complete_all(self):
        for k in self.done:
            self.done[k] = True


@pytest.fixture
def fake_events():
    fe = FakeEvents()
    kvc.kvc_staging_ring_set_event_provider(fe.provider())
    yield fe
    kvc.kvc_staging_ring_set_event_provider(None)


def test_ring_state_machine(fake_events):
    n, sb = 4, 8192
    mem = np.zeros(n * sb + 64, dtype=np.uint8)
    base = (mem.ctypes.data + 15) // 16 * 16
    ring = kvc.kvc_staging_ring_create(sb, n, kvc.KVC_RING_DEVICE, base, n * sb)
    assert kvc.kvc_staging_ring_num_slots(ring) == n and kvc.kvc_staging_ring_slot_bytes(ring) == sb
    got = [kvc.kvc_staging_ring_acquire(ring) for _ in range(n)]
    assert [g[0] for g in got] == [0, 1, 2, 3]                       # FIFO
    assert [g[1] for g in got] == [base + i * sb for i in range(n)]
    with pytest.raises(kvc.KvcError) as e:                           # N+1-th: all slots held
        kvc.kvc_staging_ring_acquire(ring)
    assert e.value.status == kvc.KVC_ERR_WOULD_BLOCK
    with pytest.raises(kvc.KvcError) as e:
        kvc.kvc_staging_ring_acquire(ring, timeout_us=2000)
    assert e.value.status == kvc.KVC_ERR_TIMEOUT
    with pytest.raises(kvc.KvcError) as e:
        kvc.kvc_staging_ring_acquire(ring, timeout_us=-1)
    assert e.value.status == kvc.KVC_ERR_INVALID_ARG
    # wrong-order calls are refused
    for fn in (kvc.kvc_staging_ring_wait_filled, kvc.kvc_staging_ring_release):
        with pytest.raises(kvc.KvcError) as e:
            fn(ring, 0, 0)
        assert e.value.status == kvc.KVC_ERR_STATE
    kvc.kvc_staging_ring_commit(ring, 0, 11)
    with pytest.raises(kvc.KvcError) as e:
        kvc.kvc_staging_ring_commit(ring, 0, 11)
    assert e.value.status == kvc.KVC_ERR_STATE
    kvc.kvc_staging_ring_wait_filled(ring, 0, 22)
    kvc.kvc_staging_ring_release(ring, 0, 22)
    assert [s for _, s in fake_events.recorded] == [11, 22]
    # released but its event has not completed: still not reusable (Sec. 6.4)
    with pytest.raises(kvc.KvcError) as e:
        kvc.kvc_staging_ring_acquire(ring)
    assert e.value.status == kvc.KVC_ERR_WOULD_BLOCK
    assert kvc.kvc_staging_ring_stats(ring)[0] == 4
    fake_events.complete_all()
    assert kvc.kvc_staging_ring_acquire(ring)[0] == 0                # exactly one more succeeds
    with pytest.raises(kvc.KvcError):
        kvc.kvc_staging_ring_acquire(ring)
    in_flight, acquires, stalls = kvc.kvc_staging_ring_stats(ring)
    assert (in_flight, acquires) == (4, 5) and stalls >= 4
    with pytest.raises(kvc.KvcError) as e:
        kvc.kvc_staging_ring_commit(ring, 9, 0)
    assert e.value.status == kvc.KVC_ERR_INVALID_ARG
    kvc.kvc_staging_ring_destroy(ring)


def test_ring_streams_a_request_larger_than_itself(fake_events):
    """A prefix of many chunks passes through a few slots; every slot is reused only after the
    test has let its release event complete, and chunks come out in order."""
    n, sb, chunks = 3, 4096, 17
    mem = np.zeros(n * sb + 64, dtype=np.uint8)
    base = (mem.ctypes.data + 15) // 16 * 16
    view = mem[base - mem.ctypes.data:][:n * sb].reshape(n, sb)
    ring = kvc.kvc_staging_ring_create(sb, n, kvc.KVC_RING_DEVICE, base, n * sb)
    out, pending = [], []
    for c in range(chunks):
        try:
            slot, dp, _ = kvc.kvc_staging_ring_acquire(ring)
        except kvc.KvcError as e:
            assert e.status == kvc.KVC_ERR_WOULD_BLOCK and len(pending) == n
            fake_events.complete_all()          # "the copies finished"
            pending.clear()
            slot, dp, _ = kvc.kvc_staging_ring_acquire(ring)
        assert slot == c % n and dp == base + slot * sb
        view[slot, :] = c                        # producer fills the slot
        kvc.kvc_staging_ring_commit(ring, slot, 1)
        kvc.kvc_staging_ring_wait_filled(ring, slot, 2)
        out.append(int(view[slot, 0]))           # consumer drains it
        kvc.kvc_staging_ring_release(ring, slot, 2)
        pending.append(slot)
    assert out == list(range(chunks))
    assert kvc.kvc_staging_ring_stats(ring)[1] == chunks
    kvc.kvc_staging_ring_destroy(ring)


def _pool_ring(n, sb, reserve, max_spec=1, retain=False):
    mem = np.zeros(n * sb + 64, dtype=np.uint8)
    base = (mem.ctypes.data + 15) // 16 * 16
    ring = kvc.kvc_staging_ring_create(sb, n, kvc.KVC_RING_DEVICE, base, n * sb)
    kvc.kvc_staging_ring_set_policy(ring, reserve, max_spec, retain)
    ring._mem = mem
    return ring, base


def test_pool_mode_any_free_slot_and_events_gate_reuse(fake_events):
    """Pool mode (Sec. 6.4 / 6.5): slots leave in any order, a slow slot holds up nobody, and a
    slot goes back to the policy only once the event behind its last consumer has completed."""
    D, S, P = kvc.KVC_CLASS_DEMAND_LOAD, kvc.KVC_CLASS_STORE, kvc.KVC_CLASS_PRELOAD
    ring, base = _pool_ring(4, 4096, reserve=1)
    with pytest.raises(kvc.KvcError) as e:                          # FIFO acquisition is off
        kvc.kvc_staging_ring_acquire(ring)
    assert e.value.status == kvc.KVC_ERR_STATE
    a = kvc.kvc_staging_ring_acquire_for(ring, D, 100)
    b = kvc.kvc_staging_ring_acquire_for(ring, S, 101)
    c = kvc.kvc_staging_ring_acquire_for(ring, D, 102)
    assert [x[0] for x in (a, b, c)] == [0, 1, 2] and not any(x[3] for x in (a, b, c))
    assert a[1] == base and c[1] == base + 2 * 4096
    # slot 0 is slow (its read never finishes in this test); slots 1 and 2 complete and are reused
    for slot in (1, 2):
        kvc.kvc_staging_ring_commit(ring, slot, 7)
        kvc.kvc_staging_ring_wait_filled(ring, slot, 8)
        kvc.kvc_staging_ring_release(ring, slot, 8)
    d = kvc.kvc_staging_ring_acquire_for(ring, D, 103)
    assert d[0] == 3                                                 # the last free slot
    # released slots are not reusable before their events complete: nothing is left
    assert kvc.kvc_staging_ring_acquire_for(ring, D, 104) is None
    with pytest.raises(kvc.KvcError) as e:
        kvc.kvc_staging_ring_acquire_for(ring, D, 104, timeout_us=2000)
    assert e.value.status == kvc.KVC_ERR_TIMEOUT
    fake_events.complete_all()
    e1 = kvc.kvc_staging_ring_acquire_for(ring, D, 104)
    e2 = kvc.kvc_staging_ring_acquire_for(ring, S, 105)
    assert sorted([e1[0], e2[0]]) == [1, 2]                          # while slot 0 is still held
    c = kvc.kvc_staging_ring_policy_counters(ring)
    assert (c["n_free"], c["n_in_flight"], c["acquires"]) == (0, 4, 6)
    # more releases than references are refused
    kvc.kvc_staging_ring_commit_host(ring, 0)
    kvc.kvc_staging_ring_release(ring, 0, 8)
    with pytest.raises(kvc.KvcError) as e:
        kvc.kvc_staging_ring_release(ring, 0, 8)
    assert e.value.status == kvc.KVC_ERR_STATE
    kvc.kvc_staging_ring_destroy(ring)


def test_pool_mode_reserve_join_claim_and_shared_release(fake_events):
    D, S, P = kvc.KVC_CLASS_DEMAND_LOAD, kvc.KVC_CLASS_STORE, kvc.KVC_CLASS_PRELOAD
    ring, base = _pool_ring(4, 4096, reserve=2, max_spec=2)
    p1 = kvc.kvc_staging_ring_acquire_for(ring, P, 1)
    p2 = kvc.kvc_staging_ring_acquire_for(ring, P, 2)
    assert p1[0] == 0 and p2[0] == 1
    assert kvc.kvc_staging_ring_acquire_for(ring, P, 3) is None      # the reserve is for foreground work
    # a demand load for key 1 joins the preload that is still being read, and claims it
    j = kvc.kvc_staging_ring_acquire_for(ring, D, 1)
    assert j[0] == 0 and j[3] is True
    assert kvc.kvc_staging_ring_slot_filled(ring, 0) is False
    with pytest.raises(kvc.KvcError) as e:                           # claimed: no longer cancellable
        kvc.kvc_staging_ring_cancel(ring, 0)
    assert e.value.status == kvc.KVC_ERR_STATE
    kvc.kvc_staging_ring_cancel(ring, 1)                             # the unclaimed one is
    assert kvc.kvc_staging_ring_policy_counters(ring)["cancels"] == 1
    kvc.kvc_staging_ring_commit_host(ring, 0)                        # the read finished
    assert kvc.kvc_staging_ring_slot_filled(ring, 0) is True
    kvc.kvc_staging_ring_release_host(ring, 0)                       # the preloader's reference
    kvc.kvc_staging_ring_wait_filled(ring, 0, 5)
    kvc.kvc_staging_ring_release(ring, 0, 5)                         # the demand load's, after its unpack
    c = kvc.kvc_staging_ring_policy_counters(ring)
    assert (c["joins"], c["claims"], c["n_staged"], c["n_free"]) == (1, 1, 1, 3)   # event not complete yet
    fake_events.complete_all()
    c = kvc.kvc_staging_ring_policy_counters(ring)
    assert (c["n_staged"], c["n_free"]) == (0, 4)
    # two consumers on different streams share a slot: the event is re-recorded behind each
    a = kvc.kvc_staging_ring_acquire_for(ring, D, 9)
    b = kvc.kvc_staging_ring_acquire_for(ring, D, 9)
    assert b[0] == a[0] and b[3]
    kvc.kvc_staging_ring_commit(ring, a[0], 3)
    n0 = len(fake_events.recorded)
    kvc.kvc_staging_ring_release(ring, a[0], 5)
    kvc.kvc_staging_ring_release(ring, a[0], 6)
    assert [s for _, s in fake_events.recorded[n0:]] == [5, 6]
    assert kvc.kvc_staging_ring_policy_counters(ring)["n_free"] == 3
    fake_events.complete_all()
    assert kvc.kvc_staging_ring_policy_counters(ring)["n_free"] == 4
    # abandon: an acquired slot that will not be filled goes back at once
    x = kvc.kvc_staging_ring_acquire_for(ring, S, 77)
    kvc.kvc_staging_ring_abandon(ring, x[0])
    assert kvc.kvc_staging_ring_policy_counters(ring)["n_free"] == 4
    kvc.kvc_staging_ring_destroy(ring)


def test_pool_mode_finished_preload_is_kept_then_claimed_or_taken_over(fake_events):
    D, S, P = kvc.KVC_CLASS_DEMAND_LOAD, kvc.KVC_CLASS_STORE, kvc.KVC_CLASS_PRELOAD
    ring, base = _pool_ring(3, 4096, reserve=1, max_spec=2)
    for key in (1, 2):
        s, dp, hp, j = kvc.kvc_staging_ring_acquire_for(ring, P, key)
        kvc.kvc_staging_ring_commit_host(ring, s)
        kvc.kvc_staging_ring_release_host(ring, s)                   # finished preloads wait unclaimed
    c = kvc.kvc_staging_ring_policy_counters(ring)
    assert (c["n_staged"], c["n_free"]) == (2, 1)
    s, dp, hp, j = kvc.kvc_staging_ring_acquire_for(ring, D, 2)      # the request arrives: no read
    assert j and kvc.kvc_staging_ring_slot_filled(ring, s)
    d1 = kvc.kvc_staging_ring_acquire_for(ring, D, 50)               # last free slot
    d2 = kvc.kvc_staging_ring_acquire_for(ring, D, 51)               # takes over the unclaimed preload (key 1)
    assert d1[0] == 2 and d2[0] == 0 and not d2[3]
    assert kvc.kvc_staging_ring_slot_filled(ring, 0) is False        # to be filled anew
    c = kvc.kvc_staging_ring_policy_counters(ring)
    assert (c["claims"], c["reclaims"]) == (1, 1)
    # policy can only be replaced while everything is free
    with pytest.raises(kvc.KvcError) as e:
        kvc.kvc_staging_ring_set_policy(ring, 0)
    assert e.value.status == kvc.KVC_ERR_STATE
    kvc.kvc_staging_ring_destroy(ring)


def test_rings_created_on_several_threads_while_the_provider_is_replaced(fake_events):
    """The event provider is process-wide state copied into a ring at creation.  Threads create,
    use and destroy rings while another thread keeps re-installing the provider: every ring must
    see one complete provider (never a half-written one) and work."""
    import threading
    errors = []
    stop = threading.Event()

    def churn():
        import time
        p = fake_events.provider()
        for _ in range(400):                      # (every installation keeps its callbacks alive)
            if stop.is_set():
                break
            kvc.kvc_staging_ring_set_event_provider(p)
            time.sleep(0.0005)

    def worker(seed):
        try:
            for it in range(40):
                mem = np.zeros(3 * 4096 + 64, dtype=np.uint8)
                base = (mem.ctypes.data + 15) // 16 * 16
                ring = kvc.kvc_staging_ring_create(4096, 3, kvc.KVC_RING_DEVICE, base, 3 * 4096)
                for _ in range(3):
                    slot, dp, _h = kvc.kvc_staging_ring_acquire(ring)
                    kvc.kvc_staging_ring_commit(ring, slot, seed)
                    kvc.kvc_staging_ring_wait_filled(ring, slot, seed + 1)
                    kvc.kvc_staging_ring_release(ring, slot, seed + 1)
                assert kvc.kvc_staging_ring_stats(ring)[1] == 3
                kvc.kvc_staging_ring_destroy(ring)
        except Exception as e:
            errors.append(repr(e))

    c = threading.Thread(target=churn)
    ws = [threading.Thread(target=worker, args=(10 * i,)) for i in range(4)]
    c.start()
    for t in ws:
        t.start()
    for t in ws:
        t.join(timeout=120)
    stop.set()
    c.join(timeout=30)
    assert errors == []


@pytest.mark.parametrize("seed", [1, 2, 3, 4])
def test_pool_mode_random_walk_keeps_its_invariants(fake_events, seed):
    """Random acquire / commit / release / cancel / abandon / event-completion sequences against a
    small model of who holds what.  Whatever the policy decides, these must hold: a slot handed
    out for a new operation has no holder left and no unfinished release event; a join lands on
    the slot that holds the key; counters add up; releases beyond the references are refused."""
    D, S, P = kvc.KVC_CLASS_DEMAND_LOAD, kvc.KVC_CLASS_STORE, kvc.KVC_CLASS_PRELOAD
    rng = np.random.default_rng(seed)
    n = 5
    ring, base = _pool_ring(n, 4096, reserve=int(rng.integers(0, 3)), max_spec=int(rng.integers(0, 3)),
                            retain=bool(rng.integers(0, 2)))
    drained_ev = {i: 2 * i + 2 for i in range(n)}     # events are created slot by slot: filled, drained
    held = {i: 0 for i in range(n)}                   # references this test holds per slot
    key_of, filled, filler = {}, {}, {}
    for step in range(600):
        op = rng.integers(0, 7)
        if op <= 1:
            cls, key = [D, S, P][rng.integers(0, 3)], int(rng.integers(0, 7))
            got = kvc.kvc_staging_ring_acquire_for(ring, cls, key)
            if got is None:
                continue
            slot, dp, hp, joined = got
            assert dp == base + slot * 4096
            if joined:
                assert key_of.get(slot) == key
            else:
                assert held[slot] == 0, "slot %d handed out while references remain" % slot
                assert fake_events.done[drained_ev[slot]], "slot %d reused before its event" % slot
                key_of[slot], filled[slot], filler[slot] = key, False, True
            held[slot] += 1
        elif op == 2:
            cands = [i for i in range(n) if held[i] and not filled.get(i, True) and filler.get(i)]
            if cands:
                i = int(rng.choice(cands))
                (kvc.kvc_staging_ring_commit_host(ring, i) if rng.integers(0, 2)
                 else kvc.kvc_staging_ring_commit(ring, i, 3))
                filled[i] = True
        elif op == 3:
            cands = [i for i in range(n) if held[i] and filled.get(i)]
            if cands:
                i = int(rng.choice(cands))
                (kvc.kvc_staging_ring_release(ring, i, int(rng.integers(4, 9))) if rng.integers(0, 2)
                 else kvc.kvc_staging_ring_release_host(ring, i))
                held[i] -= 1
        elif op == 4:
            for ev in list(fake_events.done):
                if rng.integers(0, 2):
                    fake_events.done[ev] = True
        elif op == 5:
            cands = [i for i in range(n) if held[i] == 1 and not filled.get(i, True) and filler.get(i)]
            if cands:
                i = int(rng.choice(cands))
                try:
                    kvc.kvc_staging_ring_abandon(ring, i)
                    held[i] -= 1
                    filler[i] = False
                except kvc.KvcError as e:
                    assert e.status == kvc.KVC_ERR_STATE
        else:
            i = int(rng.integers(0, n))
            if held[i] == 0 and filled.get(i):
                with pytest.raises(kvc.KvcError) as e:      # nothing left to release
                    kvc.kvc_staging_ring_release_host(ring, i)
                assert e.value.status == kvc.KVC_ERR_STATE
        c = kvc.kvc_staging_ring_policy_counters(ring)
        assert c["n_free"] + c["n_in_flight"] + c["n_staged"] + c["n_retained"] == n
    # wind down: fill what is being filled, let go of everything, finish every event
    for i in range(n):
        if held[i] and not filled.get(i, True):
            kvc.kvc_staging_ring_commit_host(ring, i)
            filled[i] = True
        while held[i]:
            kvc.kvc_staging_ring_release(ring, i, 9)
            held[i] -= 1
    fake_events.complete_all()
    c = kvc.kvc_staging_ring_policy_counters(ring)
    assert c["n_in_flight"] == 0
    assert c["n_free"] + c["n_staged"] + c["n_retained"] == n
    kvc.kvc_staging_ring_destroy(ring)


def test_staged_ring_has_a_device_half_and_a_host_half(fake_events):
    n, sb = 3, 8192
    mem = np.zeros(n * sb + 64, dtype=np.uint8)
    base = (mem.ctypes.data + 15) // 16 * 16
    ring = kvc.kvc_staging_ring_create(sb, n, kvc.KVC_RING_DEVICE_STAGED, base, n * sb)
    assert kvc.kvc_staging_ring_kind(ring) == kvc.KVC_RING_DEVICE_STAGED
    seen = []
    for i in range(n):
        slot, dp, hp = kvc.kvc_staging_ring_acquire(ring)
        assert dp == base + slot * sb and hp != 0 and hp % 4096 == 0
        assert not (base <= hp < base + n * sb)              # a separate buffer, not an alias
        ctypes.memset(hp, 0x40 + i, sb)                      # the whole host half is writable
        seen.append(hp)
    assert sorted(seen) == [seen[0] + i * sb for i in range(n)]
    kvc.kvc_staging_ring_destroy(ring)


def test_load_many_argument_checks_need_no_gpu(fake_events, tmp_path):
    """What kvc_pipeline_load_many decides before it touches the GPU: the ring must be in pool mode,
    classes must be demand load or preload, hashes must cover the chunks, and a request none of whose
    chunks is in the store is simply empty."""
    lay = _layout(chunk_tokens=64, NB=64)
    store = kvc.kvc_store_open(str(tmp_path), "m", direct_io=False)
    sb = kvc.kvc_layout_chunk_bytes(lay, 4)                               # a whole chunk fits a slot
    mem = np.zeros(4 * sb + 64, dtype=np.uint8)
    base = (mem.ctypes.data + 15) // 16 * 16
    fifo = kvc.kvc_staging_ring_create(sb, 4, kvc.KVC_RING_DEVICE, base, 4 * sb)
    ids = np.arange(10, dtype=np.int32)
    req = dict(ids=ids, hashes=[1, 2, 3], cls=kvc.KVC_CLASS_DEMAND_LOAD)
    with pytest.raises(kvc.KvcError) as e:
        kvc.kvc_pipeline_load_many(lay, fifo, store, [req])
    assert e.value.status == kvc.KVC_ERR_STATE
    kvc.kvc_staging_ring_set_policy(fifo, 1)
    stats, res = kvc.kvc_pipeline_load_many(lay, fifo, store, [req])      # nothing stored: nothing to do
    assert (stats["chunks"], stats["reads"], stats["unpack_launches"]) == (0, 0, 0)
    assert res[0]["loaded_chunks"] == 0
    with pytest.raises(kvc.KvcError) as e:                                # 10 blocks = 3 chunks, 2 hashes
        kvc.kvc_pipeline_load_many(lay, fifo, store, [dict(ids=ids, hashes=[1, 2], cls=0)])
    assert e.value.status == kvc.KVC_ERR_INVALID_ARG
    with pytest.raises(kvc.KvcError) as e:                                # stores are not loads
        kvc.kvc_pipeline_load_many(lay, fifo, store, [dict(ids=ids, hashes=[1, 2, 3], cls=kvc.KVC_CLASS_STORE)])
    assert e.value.status == kvc.KVC_ERR_INVALID_ARG
    stats, res = kvc.kvc_pipeline_load_many(lay, fifo, store, [])
    assert stats["chunks"] == 0 and res == []
    c = kvc.kvc_staging_ring_policy_counters(fifo)
    assert c["n_free"] == 4 and c["acquires"] == 0
    kvc.kvc_staging_ring_destroy(fifo)
    kvc.kvc_store_close(store)


def test_host_transfer_argument_checks_need_no_gpu(fake_events):
    """What kvc_offload_to_host / kvc_load_from_host decide before anything is enqueued: FIFO ring
    only, a positive slot timeout, a host buffer that covers every chunk, slots that hold a chunk,
    and the WHOLE block table in range (load: without repeats, also across chunks)."""
    lay = _layout(chunk_tokens=64, NB=64)
    assert kvc.kvc_layout_num_blocks(lay) == 64
    sb = kvc.kvc_layout_chunk_bytes(lay, 4)
    mem = np.zeros(4 * sb + 64, dtype=np.uint8)
    base = (mem.ctypes.data + 15) // 16 * 16
    ring = kvc.kvc_staging_ring_create(sb, 4, kvc.KVC_RING_DEVICE, base, 4 * sb)
    ids = np.arange(10, dtype=np.int32)
    need = kvc.kvc_layout_chunk_bytes(lay, 10)
    host = np.zeros(need, dtype=np.uint8)

    def both(want, ids=ids, host=host, host_bytes=None, ring=ring, **kw):
        for fn, args in ((kvc.kvc_offload_to_host, (lay, ring, ids, host)),
                         (kvc.kvc_load_from_host, (lay, ring, host, ids))):
            with pytest.raises(kvc.KvcError) as e:
                fn(*args, host_bytes=host_bytes, kernel_stream=0, copy_stream=0, **kw)
            assert e.value.status == want, fn.__name__

    both(kvc.KVC_ERR_INVALID_ARG, host_bytes=need - 1)                    # buffer one byte short
    both(kvc.KVC_ERR_INVALID_ARG, slot_timeout_us=0)                      # every wait must be bounded
    bad = ids.copy()
    bad[9] = 64
    both(kvc.KVC_ERR_OUT_OF_RANGE, ids=bad)                               # last id of the last chunk
    bad[9] = -1
    both(kvc.KVC_ERR_OUT_OF_RANGE, ids=bad)
    dup = ids.copy()
    dup[9] = dup[0]                                                       # same block in chunks 0 and 2
    with pytest.raises(kvc.KvcError) as e:
        kvc.kvc_load_from_host(lay, ring, host, dup, kernel_stream=0, copy_stream=0)
    assert e.value.status == kvc.KVC_ERR_CONFLICT
    small = kvc.kvc_staging_ring_create(4096, 4, kvc.KVC_RING_DEVICE, base, 4 * sb)
    both(kvc.KVC_ERR_INVALID_ARG, ring=small)                             # a chunk does not fit a slot
    kvc.kvc_staging_ring_destroy(small)
    in_flight, acquires, _ = kvc.kvc_staging_ring_stats(ring)
    assert (in_flight, acquires) == (0, 0)                                # nothing was taken
    kvc.kvc_staging_ring_set_policy(ring, 1)
    both(kvc.KVC_ERR_STATE)                                               # pool mode: slots are keyed by hash
    # an empty request is a no-op
    fifo = kvc.kvc_staging_ring_create(sb, 2, kvc.KVC_RING_DEVICE, base, 4 * sb)
    st = kvc.kvc_offload_to_host(lay, fifo, ids[:0], host, kernel_stream=0, copy_stream=0)
    assert (st["chunks"], st["total_chunks"], st["bytes"]) == (0, 0, 0)
    kvc.kvc_staging_ring_destroy(fifo)
    kvc.kvc_staging_ring_destroy(ring)


def test_ring_create_validation(fake_events):
    for args, want in [((4096, 0, 0, 0x1000, 1 << 20), kvc.KVC_ERR_INVALID_ARG),
                       ((0, 2, 0, 0x1000, 1 << 20), kvc.KVC_ERR_INVALID_ARG),
                       ((4100, 2, 0, 0x1000, 1 << 20), kvc.KVC_ERR_ALIGNMENT),
                       ((4096, 2, 7, 0x1000, 1 << 20), kvc.KVC_ERR_INVALID_ARG),
                       ((4096, 4, 0, 0x1000, 8192), kvc.KVC_ERR_INVALID_ARG),
                       ((4096, 2, 0, 0x1008, 1 << 20), kvc.KVC_ERR_ALIGNMENT)]:
        with pytest.raises(kvc.KvcError) as e:
            kvc.kvc_staging_ring_create(*args)
        assert e.value.status == want, args


def test_ring_host_side_transitions(fake_events):
    """Slots filled or drained by the host (file reads and writes) need no event."""
    n, sb = 2, 4096
    mem = np.zeros(n * sb + 64, dtype=np.uint8)
    base = (mem.ctypes.data + 15) // 16 * 16
    ring = kvc.kvc_staging_ring_create(sb, n, kvc.KVC_RING_DEVICE, base, n * sb)
    for fn in (kvc.kvc_staging_ring_commit_host, kvc.kvc_staging_ring_sync_filled,
               kvc.kvc_staging_ring_release_host):
        with pytest.raises(kvc.KvcError) as e:       # nothing acquired yet
            fn(ring, 0)
        assert e.value.status == kvc.KVC_ERR_STATE
    slot, _, _ = kvc.kvc_staging_ring_acquire(ring)
    kvc.kvc_staging_ring_commit_host(ring, slot)      # host filled it: no event recorded
    assert fake_events.recorded == []
    kvc.kvc_staging_ring_sync_filled(ring, slot)      # returns at once
    kvc.kvc_staging_ring_wait_filled(ring, slot, 5)   # adds no dependency
    kvc.kvc_staging_ring_release_host(ring, slot)     # host consumer done: free immediately
    assert kvc.kvc_staging_ring_stats(ring)[0] == 0
    # GPU producer, host consumer: sync_filled waits on the recorded event
    slot2, _, _ = kvc.kvc_staging_ring_acquire(ring)
    kvc.kvc_staging_ring_commit(ring, slot2, 9)
    ev = fake_events.recorded[-1][0]
    assert fake_events.done[ev] is False
    kvc.kvc_staging_ring_sync_filled(ring, slot2)     # the fake "synchronize" completes it
    assert fake_events.done[ev] is True
    kvc.kvc_staging_ring_release_host(ring, slot2)
    assert [kvc.kvc_staging_ring_acquire(ring)[0] for _ in range(2)] == [0, 1]
    kvc.kvc_staging_ring_destroy(ring)


def test_ring_trace_records_transitions_in_order(fake_events):
    n, sb = 2, 4096
    mem = np.zeros(n * sb + 64, dtype=np.uint8)
    base = (mem.ctypes.data + 15) // 16 * 16
    ring = kvc.kvc_staging_ring_create(sb, n, kvc.KVC_RING_DEVICE, base, n * sb)
    tr = kvc.kvc_staging_ring_set_trace(ring, 6)
    for _ in range(2):
        slot, _, _ = kvc.kvc_staging_ring_acquire(ring)
        kvc.kvc_staging_ring_commit(ring, slot, 1)
        kvc.kvc_staging_ring_release(ring, slot, 2)
    with pytest.raises(kvc.KvcError):
        kvc.kvc_staging_ring_acquire(ring)            # both slots wait for their events: a stall
    assert kvc.kvc_staging_ring_trace_count(ring) == 7        # one more than the buffer holds
    A, C, R = kvc.KVC_TRACE_ACQUIRE, kvc.KVC_TRACE_COMMIT, kvc.KVC_TRACE_RELEASE
    assert list(zip(tr["slot"].tolist(), tr["what"].tolist())) == [(0, A), (0, C), (0, R), (1, A), (1, C), (1, R)]
    assert (np.diff(tr["t_ns"].astype(np.int64)) >= 0).all() and tr["t_ns"][0] > 0
    kvc.kvc_staging_ring_set_trace(ring, 0)
    fake_events.complete_all()
    kvc.kvc_staging_ring_acquire(ring)
    assert kvc.kvc_staging_ring_trace_count(ring) == 0
    kvc.kvc_staging_ring_destroy(ring)


def test_header_is_plain_c99():
    import shutil
    import subprocess
    if shutil.which("gcc") is None:
        pytest.skip("needs gcc")
    r = subprocess.run(["gcc", "-std=c99", "-Wall", "-Wextra", "-pedantic", "-Werror", "-fsyntax-only",
                        "-x", "c", os.path.join(ROOT, "include", "kvc.h")], capture_output=True, text=True)
    assert r.returncode == 0, r.stderr


def test_descriptor_fuzz_never_crashes_and_derived_sizes_hold():
    """Random descriptors, valid or not: creation either fails with a status or yields a handle whose
    derived sizes obey the Sec. 2.1 formula; nothing crashes."""
    rng = np.random.default_rng(99)
    made = 0
    def pick(good, bad):
        return int(rng.choice(good)) if rng.random() < 0.9 else int(rng.choice(bad))

    for _ in range(400):
        L, P = pick([1, 2, 4], [0]), pick([1, 2], [0, 3])
        NB, B = pick([1, 7, 40], [0]), pick([1, 4, 16], [0, 3])
        H, D = pick([1, 2, 4], [0, 5]), pick([8, 16, 64, 128], [0, 1, 3, 100])
        e = pick([1, 2, 4], [0, 3, 8])
        chunk = pick([B, 2 * B, 16 * B], [0, B + 1, 7])
        base = pick([0x10000, 0x10010], [0, 0x10004])
        slab = B * H * D * e
        plane = pick([slab * NB, slab * NB + 16], [0, 8])
        try:
            lay = kvc.kvc_layout_create(L, P, NB, B, H, D, e, chunk, base=base,
                                        layer_stride=plane * max(P, 1), plane_stride=plane,
                                        block_stride=pick([0, slab], [slab + 16, 7]),
                                        chunk_order=pick([0, 1], [2]))
        except kvc.KvcError as err:
            assert 1 <= err.status <= 13
            continue
        made += 1
        assert kvc.kvc_layout_slab_bytes(lay) == slab and slab % 16 == 0
        assert kvc.kvc_layout_bytes_per_token(lay) == L * P * H * D * e
        assert chunk % B == 0 and kvc.kvc_layout_blocks_per_chunk(lay) == chunk // B
        n = int(rng.integers(0, 200))
        assert kvc.kvc_layout_chunk_bytes(lay, n) == L * P * n * slab
        d = kvc.kvc_map_request(lay, n)
        assert sum(x[3] for x in d) == n and sum(x[4] for x in d) == L * P * n * slab
        kvc.kvc_layout_destroy(lay)
    assert made > 3
