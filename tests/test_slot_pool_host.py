"""The slot policy of Sec. 6.5 (host only): reserve for foreground work, shared slots for equal
keys, claims, reclaiming, cancellation, retention; then a synthetic arrival trace in which
speculative preloads never cost a demand request its slot."""
import numpy as np
import pytest

from paper_2609_11744_b200 import kvc

D, S, P = kvc.KVC_CLASS_DEMAND_LOAD, kvc.KVC_CLASS_STORE, kvc.KVC_CLASS_PRELOAD


def test_reserve_and_speculative_limit():
    pool = kvc.kvc_slot_pool_create(6, 2, max_speculative=3)
    got = [kvc.kvc_slot_pool_acquire(pool, P, 100 + i) for i in range(5)]
    # 3 preloads in flight is the limit, although 3 slots are still free (> reserve of 2)
    assert [g is not None for g in got] == [True, True, True, False, False]
    for slot, joined in got[:3]:
        assert not joined
        kvc.kvc_slot_pool_mark_staged(pool, slot)
    # staged preloads no longer count as in flight; now the reserve is what stops them
    assert kvc.kvc_slot_pool_acquire(pool, P, 200) is not None            # 4th slot: 2 left free
    assert kvc.kvc_slot_pool_acquire(pool, P, 201) is None                # free == reserve
    # foreground work may use the reserved slots
    a = kvc.kvc_slot_pool_acquire(pool, D, 300)
    b = kvc.kvc_slot_pool_acquire(pool, S, 301)
    assert a is not None and b is not None
    c = kvc.kvc_slot_pool_get_counters(pool)
    assert (c["n_free"], c["preload_refusals"], c["acquires"]) == (0, 3, 6)


def test_equal_keys_share_a_slot_and_demand_claims_a_preload():
    pool = kvc.kvc_slot_pool_create(4, 1, max_speculative=0)
    s1, j1 = kvc.kvc_slot_pool_acquire(pool, P, 7)
    s2, j2 = kvc.kvc_slot_pool_acquire(pool, P, 7)        # second candidate with the same prefix
    s3, j3 = kvc.kvc_slot_pool_acquire(pool, D, 7)        # the request gets scheduled: joins the read
    assert (s1, j1) == (s1, False) and (s2, j2) == (s1, True) and (s3, j3) == (s1, True)
    c = kvc.kvc_slot_pool_get_counters(pool)
    assert (c["acquires"], c["joins"], c["claims"], c["n_in_flight"]) == (1, 2, 1, 1)
    with pytest.raises(kvc.KvcError) as e:                # claimed: it can no longer be cancelled
        kvc.kvc_slot_pool_cancel(pool, s1)
    assert e.value.status == kvc.KVC_ERR_STATE
    kvc.kvc_slot_pool_mark_staged(pool, s1)
    for _ in range(3):
        kvc.kvc_slot_pool_release(pool, s1)
    assert kvc.kvc_slot_pool_get_counters(pool)["n_free"] == 4
    with pytest.raises(kvc.KvcError) as e:
        kvc.kvc_slot_pool_release(pool, s1)
    assert e.value.status == kvc.KVC_ERR_STATE


def test_foreground_takes_over_unclaimed_preloads_and_cancel():
    pool = kvc.kvc_slot_pool_create(3, 1, max_speculative=0)
    a, _ = kvc.kvc_slot_pool_acquire(pool, P, 1)
    b, _ = kvc.kvc_slot_pool_acquire(pool, P, 2)
    assert kvc.kvc_slot_pool_acquire(pool, P, 3) is None          # reserve
    kvc.kvc_slot_pool_mark_staged(pool, a)
    kvc.kvc_slot_pool_release(pool, a)                            # finished preload, waits unclaimed
    d1, _ = kvc.kvc_slot_pool_acquire(pool, D, 10)                # uses the reserved slot
    # no free slot left: the next demand load takes over the staged, unclaimed preload (key 1)
    d2, joined = kvc.kvc_slot_pool_acquire(pool, D, 11)
    assert d2 == a and not joined
    assert kvc.kvc_slot_pool_get_counters(pool)["reclaims"] == 1
    # key 1 is gone: asking for it now starts a new operation -- but nothing is free
    assert kvc.kvc_slot_pool_acquire(pool, D, 1) is None
    # the preload still in flight (key 2) can be cancelled to make room
    kvc.kvc_slot_pool_cancel(pool, b)
    d3, joined = kvc.kvc_slot_pool_acquire(pool, D, 1)
    assert d3 == b and not joined
    c = kvc.kvc_slot_pool_get_counters(pool)
    assert (c["cancels"], c["foreground_refusals"], c["n_free"]) == (1, 1, 0)


def test_staged_preload_that_is_still_held_is_not_taken_over():
    """A preload whose read has finished but whose holder has not let go yet (its copy into the
    slot may still be running) must not be handed to foreground work; nor may a preload that
    other candidates joined be cancelled under them."""
    pool = kvc.kvc_slot_pool_create(2, 1, max_speculative=0)
    a, _ = kvc.kvc_slot_pool_acquire(pool, P, 1)
    kvc.kvc_slot_pool_mark_staged(pool, a)                        # staged, the preloader still holds it
    d, _ = kvc.kvc_slot_pool_acquire(pool, D, 10)                 # the reserved slot
    assert d != a
    assert kvc.kvc_slot_pool_acquire(pool, D, 11) is None         # nothing to take: WOULD_BLOCK
    assert kvc.kvc_slot_pool_get_counters(pool)["reclaims"] == 0
    kvc.kvc_slot_pool_release(pool, a)                            # now it waits unreferenced
    got = kvc.kvc_slot_pool_acquire(pool, D, 11)
    assert got == (a, False)
    assert kvc.kvc_slot_pool_get_counters(pool)["reclaims"] == 1

    pool = kvc.kvc_slot_pool_create(4, 1, max_speculative=0)
    b, _ = kvc.kvc_slot_pool_acquire(pool, P, 5)
    b2, joined = kvc.kvc_slot_pool_acquire(pool, P, 5)            # a second candidate joins the read
    assert b2 == b and joined
    with pytest.raises(kvc.KvcError) as e:
        kvc.kvc_slot_pool_cancel(pool, b)
    assert e.value.status == kvc.KVC_ERR_STATE
    kvc.kvc_slot_pool_release(pool, b)                            # the joiner leaves
    kvc.kvc_slot_pool_cancel(pool, b)                             # sole holder: allowed
    assert kvc.kvc_slot_pool_get_counters(pool)["n_free"] == 4


def test_retention_is_an_lru_cache():
    pool = kvc.kvc_slot_pool_create(3, 0, retain_completed=True)
    slots = {}
    for key in (1, 2, 3):
        s, _ = kvc.kvc_slot_pool_acquire(pool, D, key)
        kvc.kvc_slot_pool_mark_staged(pool, s)
        kvc.kvc_slot_pool_release(pool, s)
        slots[key] = s
    assert kvc.kvc_slot_pool_get_counters(pool)["n_retained"] == 3
    s, joined = kvc.kvc_slot_pool_acquire(pool, D, 1)             # hit: no read needed
    assert joined and s == slots[1]
    kvc.kvc_slot_pool_release(pool, s)
    s4, joined = kvc.kvc_slot_pool_acquire(pool, D, 4)            # miss: evicts key 2 (least recent)
    assert not joined and s4 == slots[2]
    assert kvc.kvc_slot_pool_acquire(pool, D, 2)[1] is False      # key 2 has to be read again
    assert kvc.kvc_slot_pool_acquire(pool, D, 1)[1] is True       # key 1 survived
    assert kvc.kvc_slot_pool_acquire(pool, P, 9) is None          # preloads never evict


def test_synthetic_trace_preloads_never_starve_demand():
    """Requests arrive in a queue; the scheduler admits `width` at a time; every waiting request in
    a bounded lookahead is offered as a preload candidate.  Reads take a few ticks.  With the
    reserve equal to the demand width no demand request is ever refused a slot, preloads that
    finish early turn into joins, and every slot is returned at the end."""
    rng = np.random.default_rng(3)
    n_slots, width, lookahead = 8, 3, 6
    pool = kvc.kvc_slot_pool_create(n_slots, width, max_speculative=2)
    n_req = 200
    keys = rng.integers(0, 60, n_req)            # repeated prefixes among requests
    queue = list(range(n_req))
    running = {}                                  # request -> (slot, ticks left, joined)
    preloads = {}                                 # slot -> ticks left
    demand_refused = 0
    tick = 0
    while queue or running or preloads:
        tick += 1
        for slot in list(preloads):               # reads in flight make progress
            preloads[slot] -= 1
            if preloads[slot] == 0:
                kvc.kvc_slot_pool_mark_staged(pool, slot)
                kvc.kvc_slot_pool_release(pool, slot)
                del preloads[slot]
        for r in list(running):
            slot, left, joined = running[r]
            if left <= 1:
                if not joined:
                    kvc.kvc_slot_pool_mark_staged(pool, slot)
                kvc.kvc_slot_pool_release(pool, slot)
                del running[r]
            else:
                running[r] = (slot, left - 1, joined)
        while queue and len(running) < width:     # demand first
            r = queue[0]
            got = kvc.kvc_slot_pool_acquire(pool, D, int(keys[r]))
            if got is None:
                demand_refused += 1
                break
            queue.pop(0)
            slot, joined = got
            if joined and slot in preloads:
                # joined a preload still being read: it finishes as this request's read now
                left = preloads.pop(slot)
                running[r] = (slot, left, False)
                kvc.kvc_slot_pool_release(pool, slot)      # the preload's own reference
            else:
                running[r] = (slot, 1 if joined else 3, joined)
        for r in queue[:lookahead]:               # then speculative work
            got = kvc.kvc_slot_pool_acquire(pool, P, int(keys[r]))
            if got is None:
                break
            slot, joined = got
            if joined:
                kvc.kvc_slot_pool_release(pool, slot)      # somebody reads it already
            else:
                preloads[slot] = 3
        assert tick < 5000
    c = kvc.kvc_slot_pool_get_counters(pool)
    assert demand_refused == 0 and c["foreground_refusals"] == 0
    assert c["joins"] > 0 and c["claims"] > 0 and c["preload_refusals"] > 0
    # only finished, never-claimed preloads may still hold slots; foreground work can take them all
    assert c["n_in_flight"] == 0 and c["n_retained"] == 0
    taken = [kvc.kvc_slot_pool_acquire(pool, S, 10_000 + i) for i in range(n_slots)]
    assert all(t is not None and not t[1] for t in taken)
