"""Pins for the oracle's chunk keys: brute force against token tuples on tiny alphabets.

The index must order keys so that a token prefix sorts before its extensions, and a key must
name exactly one token prefix (Sec. 3.1/3.2 of the paper: key order follows prefix order, keys
are not flattened into unordered hashes)."""
import itertools

import numpy as np
import pytest

import oracle
from oracle import Geom

P = (1 << 61) - 1
BASE = (0x0B4E0EF37BC32127, 0x16A09E667F3BCC90)


def G(C, ns=0):
    return Geom(n_layers=1, n_kv_heads=1, head_dim=8, elem_bytes=2, page_tokens=C,
                chunk_tokens=C, ns=ns)


def poly(tokens, lane):
    n = len(tokens)
    return sum((int(t) + 1) * pow(BASE[lane], n - 1 - i, P) for i, t in enumerate(tokens)) % P


def test_key_fields_from_definition():
    C = 4
    toks = np.array([7, 1, 2, 9, 5, 5, 5, 6, 3, 3], dtype=np.uint32)   # 2 whole chunks + tail
    k = oracle.chunk_keys(G(C, ns=0xABCD), toks)
    assert k.shape == (2, 4)
    for j in range(2):
        assert int(k[j, 0]) == (0xABCD << 32) | j
        assert int(k[j, 1]) == poly(toks[:(j + 1) * C], 0)      # digest of the WHOLE prefix
        assert int(k[j, 2]) == poly(toks[:(j + 1) * C], 1)
        assert int(k[j, 3]) == (int(toks[j * C]) << 32) | int(toks[j * C + C - 1])


def test_partial_chunk_is_never_keyed():
    for n in range(0, 9):
        assert len(oracle.chunk_keys(G(4), np.arange(n, dtype=np.uint32))) == n // 4


def test_start_chunk_keeps_full_prefix_digest():
    rng = np.random.default_rng(3)
    toks = rng.integers(0, 50, 16 * 9 + 5, dtype=np.uint32)
    full = oracle.chunk_keys(G(16), toks)
    for jb in (0, 1, 4, 8, 9, 12):
        assert np.array_equal(oracle.chunk_keys(G(16), toks, jb), full[jb:])


def test_large_token_ids_and_chunk_64():
    toks = np.full(128, 2**32 - 1, dtype=np.uint32)
    k = oracle.chunk_keys(G(64), toks)
    assert int(k[1, 3]) == ((2**32 - 1) << 32) | (2**32 - 1)
    assert int(k[1, 1]) == poly(toks, 0) and int(k[0, 2]) == poly(toks[:64], 1)


@pytest.mark.parametrize("C,vocab,nchunks", [(1, 2, 6), (2, 2, 3), (2, 3, 2)])
def test_brute_force_identity_and_order(C, vocab, nchunks):
    """All strings over a tiny alphabet: key equality <=> prefix equality; a proper prefix has a
    smaller key; along one sequence keys strictly increase."""
    g = G(C)
    seqs = list(itertools.product(range(vocab), repeat=C * nchunks))
    table = {}     # token prefix tuple -> key tuple
    for s in seqs:
        k = oracle.chunk_keys(g, np.array(s, dtype=np.uint32))
        prev = None
        for j in range(nchunks):
            pre, key = s[:(j + 1) * C], tuple(int(x) for x in k[j])
            assert table.setdefault(pre, key) == key          # same prefix -> same key
            if prev is not None:
                assert prev < key                             # strictly increasing in j
            prev = key
    assert len(set(table.values())) == len(table)             # different prefix -> different key
    items = list(table.items())
    for (pa, ka), (pb, kb) in itertools.combinations(items, 2):
        if len(pa) < len(pb) and pb[:len(pa)] == pa:
            assert ka < kb
        if len(pb) < len(pa) and pa[:len(pb)] == pb:
            assert kb < ka
    # sorting by key is a topological order of the prefix relation
    order = sorted(table, key=lambda p: table[p])
    pos = {p: i for i, p in enumerate(order)}
    for p_ in table:
        if len(p_) > C:
            assert pos[p_[:-C]] < pos[p_]


def test_key_cmp_is_unsigned_lexicographic():
    rng = np.random.default_rng(5)
    ks = rng.integers(0, 2**64, (200, 4), dtype=np.uint64)
    ks[:50, 0] = ks[50:100, 0]             # force ties in the leading word
    ks[:20, 1] = ks[50:70, 1]
    ks[0] = ks[50]
    ks[1, :3] = ks[51, :3]
    for a, b in zip(ks[:100], ks[50:150]):
        ta, tb = tuple(int(x) for x in a), tuple(int(x) for x in b)
        assert oracle.key_cmp(a, b) == (ta > tb) - (ta < tb)
    hi = np.array([2**63, 0, 0, 0], dtype=np.uint64)     # top bit set must compare as large
    lo = np.array([1, 2**64 - 1, 2**64 - 1, 2**64 - 1], dtype=np.uint64)
    assert oracle.key_cmp(hi, lo) == 1 and oracle.key_cmp(lo, hi) == -1


def test_namespace_separates_equal_prefixes():
    toks = np.arange(32, dtype=np.uint32)
    a, b = oracle.chunk_keys(G(16, ns=1), toks), oracle.chunk_keys(G(16, ns=2), toks)
    assert np.array_equal(a[:, 1:], b[:, 1:]) and not np.any(a[:, 0] == b[:, 0])
    assert all(tuple(x) < tuple(y) for x in a.tolist() for y in b.tolist())


def test_logical_key_bytes_order_equals_token_order():
    """The logical key (big-endian u32 serialisation of the prefix) sorts, as bytes, exactly
    like the token tuples, a prefix before its extensions -- the order the fixed-width key
    extends linearly."""
    rng = np.random.default_rng(9)
    pres = [tuple(int(x) for x in rng.integers(0, 2**32, rng.integers(1, 5), dtype=np.uint64))
            for _ in range(300)]
    pres += [p[:1] for p in pres[:50]]
    ser = lambda p: b"".join(int(t).to_bytes(4, "big") for t in p)
    assert sorted(pres) == sorted(pres, key=ser)
