"""Pins for the oracle's Bloom filter: what the definition of a Bloom filter fixes -- no false
negatives, union = bitwise OR, at most six bits per key in one 32-byte block, a false-positive
rate near the textbook value -- plus bit positions worked out by hand for one key."""
import numpy as np

import oracle


def rand_keys(rng, n):
    k = np.zeros((n, 4), dtype=np.uint64)
    k[:, 0] = rng.integers(0, 2000, n)
    k[:, 1] = rng.integers(0, 2**61 - 1, n, dtype=np.uint64)
    k[:, 2] = rng.integers(0, 2**61 - 1, n, dtype=np.uint64)
    k[:, 3] = rng.integers(0, 2**64, n, dtype=np.uint64)
    return k


def test_size_rule():
    assert oracle.bloom_blocks(0) == 1 and oracle.bloom_blocks(1) == 1
    assert oracle.bloom_blocks(25) == 1 and oracle.bloom_blocks(26) == 2
    assert oracle.bloom_blocks(1_000_000) == (10_000_000 + 255) // 256


def test_single_key_bits_by_hand():
    # one key, one block: the six positions are the six low bytes of w2
    key = np.array([7, 0x1234567890ABCDE, 0x00_0F_FF_80_07_01_00, 99], dtype=np.uint64)
    bloom = oracle.bloom_build(key.reshape(1, 4))
    assert bloom.size == 32
    # w2 bytes (least significant first): 00 01 07 80 FF 0F -> positions 0, 1, 7, 128, 255, 15
    want = np.zeros(32, dtype=np.uint8)
    for p in (0, 1, 7, 128, 255, 15):
        want[p >> 3] |= 1 << (p & 7)
    assert np.array_equal(bloom, want)
    assert oracle.bloom_may_contain(bloom, key)


def test_block_choice_follows_w1():
    rng = np.random.default_rng(1)
    keys = rand_keys(rng, 1000)
    nb = oracle.bloom_blocks(1000)
    full = oracle.bloom_build(keys)
    want = np.zeros(32 * nb, dtype=np.uint8)
    for k in keys:                                           # the definition, with Python integers
        blk = (int(k[1]) * nb) >> 61
        for i in range(6):
            p = (int(k[2]) >> (8 * i)) & 255
            want[32 * blk + (p >> 3)] |= 1 << (p & 7)
    assert np.array_equal(full, want)


def test_no_false_negatives_and_union_is_or():
    rng = np.random.default_rng(2)
    keys = rand_keys(rng, 5000)
    bloom = oracle.bloom_build(keys)
    assert all(oracle.bloom_may_contain(bloom, k) for k in keys)
    # same number of blocks -> the filter of a union is the OR of the filters: build halves
    # inside a filter sized for the whole set by padding with repeats
    a = np.concatenate([keys[:2500], keys[:2500]])
    b = np.concatenate([keys[2500:], keys[2500:]])
    assert np.array_equal(oracle.bloom_build(a) | oracle.bloom_build(b), bloom)
    # at most 6 bits per key
    assert int(np.unpackbits(bloom).sum()) <= 6 * 5000


def test_false_positive_rate_is_near_theory():
    rng = np.random.default_rng(3)
    keys = rand_keys(rng, 20000)
    bloom = oracle.bloom_build(keys)
    others = rand_keys(rng, 20000)
    fp = sum(oracle.bloom_may_contain(bloom, k) for k in others) / len(others)
    # 10 bits/key, 6 probes: ~0.8 % for an ideal filter, a few times that for a blocked one
    assert 0.002 < fp < 0.05, fp
    fill = np.unpackbits(bloom).mean()
    assert 0.35 < fill < 0.55                                # ~1 - exp(-6/10.2)


def test_empty_filter_rejects_everything():
    bloom = oracle.bloom_build(np.zeros((0, 4), np.uint64))
    assert bloom.size == 32 and not bloom.any()
    assert not oracle.bloom_may_contain(bloom, np.array([0, 5, 9, 0], np.uint64))
