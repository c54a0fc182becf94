"""The K~/V~ cache of the serving path is host-side bookkeeping over a device arena that it never touches, so it is
tested here without a GPU: an address range stands in for the arena."""
import pytest

from paper_2603_22943_b200 import binding as tb

ARENA = 0x7F0000000000          # any 128-byte aligned number: the cache only does arithmetic on it
ENTRY = 4096


def test_prompt_hash_is_fnv1a_over_little_endian_token_bytes():
    assert tb.taq_hash_prompt([]) == 0xCBF29CE484222325                       # the FNV-1a offset basis
    h = 0xCBF29CE484222325
    for t in (49406, 320, 1125, 49407):
        for b in range(4):
            h = ((h ^ ((t >> (8 * b)) & 0xFF)) * 0x100000001B3) % (1 << 64)
    assert tb.taq_hash_prompt([49406, 320, 1125, 49407]) == h
    assert tb.taq_hash_prompt([1, 2]) != tb.taq_hash_prompt([2, 1])


def test_hits_misses_and_least_recently_used_eviction():
    c = tb.KvCache(ARENA, 3 * ENTRY + 100, ENTRY)                              # three entries (the tail is unused)
    assert c.stats()["capacity"] == 3
    a, hit = c.acquire(1, 10); assert not hit and a == ARENA
    b, hit = c.acquire(1, 11); assert not hit and b == ARENA + ENTRY
    u, hit = c.acquire(1, 0); assert not hit and u == ARENA + 2 * ENTRY        # the unconditional prompt of checkpoint 1
    for k in ((1, 10), (1, 11), (1, 0)):
        c.release(*k)
    u2, hit = c.acquire(1, 0); assert hit and u2 == u                          # shared by the next request
    c.release(1, 0)
    a2, hit = c.acquire(1, 10); assert hit and a2 == a
    c.release(1, 10)
    # a new pair evicts the least recently used entry: (1, 11)
    n, hit = c.acquire(2, 10); assert not hit and n == b
    c.release(2, 10)
    _, hit = c.acquire(1, 11); assert not hit                                  # gone; takes the oldest again: (1, 0)
    st = c.stats()
    assert st == {"capacity": 3, "used": 3, "hits": 2, "misses": 5, "evictions": 2}
    c.close()


def test_pinned_entries_are_never_evicted_and_checkpoints_can_be_dropped():
    c = tb.KvCache(ARENA, 2 * ENTRY, ENTRY)
    c.acquire(7, 1)
    c.acquire(7, 2)
    with pytest.raises(tb.TaqError) as e:                                      # both entries are in use
        c.acquire(8, 1)
    assert e.value.status == tb.TAQ_ERR_BUFFER_TOO_SMALL
    with pytest.raises(tb.TaqError):
        c.drop_checkpoint(7)
    c.release(7, 1)
    p, hit = c.acquire(8, 1); assert not hit and p == ARENA                    # the released one was taken, not the pinned one
    with pytest.raises(tb.TaqError):
        c.release(7, 1)                                                        # no longer there
    c.release(7, 2); c.release(8, 1)
    with pytest.raises(tb.TaqError):
        c.release(8, 1)                                                        # not pinned any more
    c.drop_checkpoint(7)
    assert c.stats()["used"] == 1
    _, hit = c.acquire(7, 2); assert not hit
    c.close()


def test_create_rejects_bad_arguments():
    for args in ((0, 1 << 20, ENTRY), (ARENA + 8, 1 << 20, ENTRY), (ARENA, 1 << 20, 100), (ARENA, ENTRY - 1, ENTRY), (ARENA, 1 << 20, 0)):
        with pytest.raises(ValueError):
            tb.KvCache(*args)
