"""Pins of the oracle's hash index of a run (Sec. 2.2: auxiliary structures of a run that shorten
point lookups). The table layout is worked out by hand on small cases, lookups are checked
against a Python dict, and the lookup rule is shown to work on any table filled by the same
rule in any order -- which is what a parallel builder produces."""
import numpy as np

import oracle

P61 = 2**61


def key(j, w1, w2, w3=0):
    return [j, w1, w2, w3]


def entry(w2, pos):
    return ((w2 & 0xFF) << 24) | (pos + 1)


def test_bucket_count():
    assert [oracle.hindex_buckets(n) for n in (0, 1, 2, 3, 4, 5, 1000, 1001)] == \
        [1, 1, 1, 2, 2, 3, 500, 501]


def test_hand_worked_table_of_five_keys():
    # 5 keys -> 3 buckets (24 slots); home = floor(w1 * 3 / 2^61)
    third = P61 // 3
    keys = np.array([key(0, 5, 0x1AB),                  # bucket 0
                     key(0, third + 7, 0x2CD),          # bucket 1
                     key(1, 9, 0x3EF),                  # bucket 0, second slot
                     key(1, 2 * third + 11, 0x401),     # bucket 2
                     key(2, third + 1, 0x5CD)],         # bucket 1, second slot (same tag as key 1)
                    dtype=np.uint64)
    t = oracle.hindex_build(keys)
    want = np.zeros(24, dtype=np.uint32)
    want[0], want[1] = entry(0xAB, 0), entry(0xEF, 2)
    want[8], want[9] = entry(0xCD, 1), entry(0xCD, 4)
    want[16] = entry(0x01, 3)
    assert np.array_equal(t, want)
    for i, k in enumerate(keys):
        assert oracle.hindex_find(t, keys, k) == i
    assert oracle.hindex_find(t, keys, key(2, third + 1, 0x6CD)) == -1     # tag matches twice, key differs
    assert oracle.hindex_find(t, keys, key(0, 2 * third + 12, 0x401)) == -1


def test_overflow_runs_into_the_next_buckets_and_wraps():
    # 10 keys, 5 buckets, all at home in the last bucket: slots 32..39, then 0 and 1
    keys = np.array([key(i, P61 - 2 - i, 0x100 + i) for i in range(10)], dtype=np.uint64)
    t = oracle.hindex_build(keys)
    want = np.zeros(40, dtype=np.uint32)
    for i in range(8):
        want[32 + i] = entry(i, i)
    want[0], want[1] = entry(8, 8), entry(9, 9)
    assert np.array_equal(t, want)
    for i, k in enumerate(keys):
        assert oracle.hindex_find(t, keys, k) == i
    # an absent key at home in the full bucket is searched past the wrap and ends at slot 2
    assert oracle.hindex_find(t, keys, key(3, P61 - 20, 0x103)) == -1


def random_keys(rng, n, w1_hi=P61 - 1):
    k = np.zeros((n, 4), dtype=np.uint64)
    k[:, 0] = rng.integers(0, 50, n)
    k[:, 1] = rng.integers(0, w1_hi, n, dtype=np.uint64)
    k[:, 2] = rng.integers(0, 2**61 - 1, n, dtype=np.uint64)
    k[:, 3] = rng.integers(0, 2**64, n, dtype=np.uint64)
    return k


def test_lookup_equals_a_dict_also_with_crowded_buckets_and_equal_tags():
    rng = np.random.default_rng(11)
    for w1_hi, few_tags in ((P61 - 1, False), (P61 // 64, True)):   # second case: 1/64 of the buckets
        keys = random_keys(rng, 3000, w1_hi)
        if few_tags:                                                 # and only four different tags
            keys[:, 2] = (keys[:, 2] >> np.uint64(8) << np.uint64(8)) | (keys[:, 2] & np.uint64(3))
        where = {tuple(int(x) for x in k): i for i, k in enumerate(keys)}
        assert len(where) == len(keys)
        t = oracle.hindex_build(keys)
        for i in range(0, len(keys), 7):
            assert oracle.hindex_find(t, keys, keys[i]) == i
        absent = random_keys(rng, 500, w1_hi)
        for k in absent:
            assert oracle.hindex_find(t, keys, k) == where.get(tuple(int(x) for x in k), -1)
        # same digests, another chunk index: only the full comparison tells them apart
        for i in range(0, 300, 3):
            k = keys[i].copy()
            k[0] += np.uint64(1)
            assert oracle.hindex_find(t, keys, k) == where.get(tuple(int(x) for x in k), -1)


def test_every_real_key_has_exactly_its_entry_and_padding_has_none():
    rng = np.random.default_rng(3)
    keys = random_keys(rng, 1000)
    keys[700:] = np.uint64(2**64 - 1)                    # padding of a flushed run
    t = oracle.hindex_build(keys)
    assert t.size == 8 * 500
    want = sorted(entry(int(keys[i, 2]), i) for i in range(700))
    assert sorted(int(x) for x in t[t != 0]) == want


def test_lookup_works_on_a_table_filled_in_any_order():
    rng = np.random.default_rng(5)
    keys = random_keys(rng, 2000, P61 // 16)             # crowded: long chains
    nb = oracle.hindex_buckets(len(keys))
    table = np.zeros(8 * nb, dtype=np.uint32)
    for i in rng.permutation(len(keys)):                 # the insertion rule, in a random order
        s = 8 * ((int(keys[i, 1]) * nb) >> 61)
        while table[s]:
            s = (s + 1) % table.size
        table[s] = entry(int(keys[i, 2]), int(i))
    assert not np.array_equal(table, oracle.hindex_build(keys))
    for i in range(len(keys)):
        assert oracle.hindex_find(table, keys, keys[i]) == i
    for k in random_keys(rng, 300, P61 // 16):
        assert oracle.hindex_find(table, keys, k) == -1


def test_too_many_keys_are_refused():
    import ctypes
    assert oracle.lib().orc_hindex_build(None, ctypes.c_uint64(2**24 - 1), None) == -1
