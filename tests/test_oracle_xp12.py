"""Pins for the oracle's compressing codec (lossless exponent packing of bf16 slabs)."""
import numpy as np
import pytest

import oracle
from oracle import Geom, VAL_DTYPE
from paper_2511_16138_b200 import synth

MAGIC = 0x32315058


def bf16(s, e, m):
    return (s << 15) | (e << 7) | m


def test_hand_worked_slab_of_eight():
    # exponents 127,126,120,127,113,112,127,100: e_max = 127 -> base = 113; 112 and 100 are exceptions
    v = np.array([bf16(0, 127, 1), bf16(1, 126, 2), bf16(0, 120, 3), bf16(1, 127, 0x7F),
                  bf16(0, 113, 0), bf16(1, 112, 5), bf16(0, 127, 6), bf16(0, 100, 7)], np.uint16)
    got = oracle.xp12_slab_encode(v)
    want = bytearray(32)                                   # 16 + 8 + 4 + 2 = 30 -> padded to 32
    want[0:4] = MAGIC.to_bytes(4, "little")
    want[4:8] = (2).to_bytes(4, "little")                  # n_exc
    want[8] = 113                                          # base
    want[9] = 0                                            # mode: packed
    want[12:16] = (32).to_bytes(4, "little")               # size
    want[16:24] = bytes([0x01, 0x82, 0x03, 0xFF, 0x00, 0x85, 0x06, 0x07])   # sign<<7 | mantissa
    # codes 14,13,7,14,0,15,14,15 -> bytes (low nibble = even element)
    want[24:28] = bytes([0xDE, 0xE7, 0xF0, 0xFE])
    want[28:30] = bytes([112, 100])                        # exceptions in element order
    assert bytes(got) == bytes(want)
    assert np.array_equal(oracle.xp12_slab_decode(got, 8), v)


def kinds(rng, n):
    """Slabs that stress different paths."""
    yield "normal", synth.bf16_normal_bits(rng, n)
    yield "zeros", np.zeros(n, np.uint16)
    yield "neg-zero-inf-nan", rng.choice(np.array([0x8000, 0x7F80, 0xFF80, 0x7FC1, 0x0001, 0x3F80],
                                                  np.uint16), n)
    yield "uniform-bits", rng.integers(0, 65536, n, dtype=np.uint16)      # -> raw mode
    x = synth.bf16_normal_bits(rng, n)
    x[rng.random(n) < 0.4] = 0x0001                                        # many tiny values
    yield "many-exceptions", x
    x = synth.bf16_normal_bits(rng, n)
    x[:n // 2] = 0                                                         # exactly N/2 candidates
    yield "half-zero", x


@pytest.mark.parametrize("n", [8, 16, 1000 * 8, 16384])
def test_roundtrip_and_size_law(n):
    rng = np.random.default_rng(n)
    for name, v in kinds(rng, n):
        b = oracle.xp12_slab_encode(v)
        e = (v >> 7) & 0xFF
        base = max(0, int(e.max()) - 14)
        n_exc = int((e < base).sum())
        if n_exc < n // 2:
            assert len(b) == (16 + n + n // 2 + n_exc + 15) // 16 * 16, name
            assert b[8] == base and b[9] == 0
            assert int.from_bytes(bytes(b[4:8]), "little") == n_exc
        else:
            assert len(b) == 16 + 2 * n and b[9] == 1, name
            assert bytes(b[16:]) == v.tobytes()
        assert int.from_bytes(bytes(b[0:4]), "little") == MAGIC
        assert int.from_bytes(bytes(b[12:16]), "little") == len(b) and len(b) % 16 == 0
        assert len(b) <= 16 + 2 * n
        assert np.array_equal(oracle.xp12_slab_decode(b, n), v), name


def test_planes_equal_a_vectorised_derivation():
    rng = np.random.default_rng(1)
    n = 4096
    v = synth.bf16_normal_bits(rng, n)
    v[rng.integers(0, n, 40)] = 0x0080                     # a few tiny values: exceptions
    b = oracle.xp12_slab_encode(v)
    e = ((v >> 7) & 0xFF).astype(np.int64)
    base = int(e.max()) - 14
    sm = (((v >> 15) << 7) | (v & 0x7F)).astype(np.uint8)
    code = np.where(e >= base, e - base, 15).astype(np.uint8)
    nib = (code[0::2] | (code[1::2] << 4)).astype(np.uint8)
    exc = e[e < base].astype(np.uint8)
    assert np.array_equal(b[16:16 + n], sm)
    assert np.array_equal(b[16 + n:16 + n + n // 2], nib)
    assert np.array_equal(b[16 + n + n // 2:16 + n + n // 2 + len(exc)], exc)
    assert not b[16 + n + n // 2 + len(exc):].any()        # zero padding


def test_normal_data_compresses_to_three_quarters():
    rng = np.random.default_rng(2)
    v = synth.bf16_normal_bits(rng, 16384)
    assert 0.750 <= len(oracle.xp12_slab_encode(v)) / (2 * 16384) < 0.752


def test_malformed_slabs_are_rejected():
    rng = np.random.default_rng(3)
    v = synth.bf16_normal_bits(rng, 64)
    v[5] = 0x0001
    b = oracle.xp12_slab_encode(v)
    assert oracle.xp12_slab_decode(b, 64) is not None
    for mutate in ("magic", "trunc", "nexc", "mode", "size"):
        c = b.copy()
        if mutate == "magic":
            c[0] ^= 1
        elif mutate == "trunc":
            c = c[:-16]
        elif mutate == "nexc":
            c[4] += 1
        elif mutate == "mode":
            c[9] = 7
        elif mutate == "size":
            c[12] += 16
        assert oracle.xp12_slab_decode(c, 64) is None, mutate
    assert oracle.xp12_slab_decode(b, 128) is None          # wrong element count


def test_batch_layout_records_and_identity():
    g = Geom(n_layers=3, n_kv_heads=2, head_dim=16, page_tokens=4, chunk_tokens=4)   # 256-byte pages
    rng = np.random.default_rng(4)
    b = synth.make_batch([rng.integers(0, 99, n, dtype=np.uint32) for n in (12, 9, 4)])
    nch = synth.chunk_counts(b.seq_off, 4)
    coff = synth.offsets(nch)
    n = int(coff[-1])
    pool = synth.random_pool_bytes(rng, 6, 12, g.page_bytes)
    pool[2, 3] = 0                                          # an all-zero slab
    pool[4, 5] = rng.integers(0, 256, g.page_bytes, dtype=np.uint8)   # an incompressible one
    pages = synth.random_pages(rng, 12, n)
    keys, vals, blob = oracle.encode_batch_xp12(g, b.tokens, b.seq_off, None, coff, pages, pool,
                                                7, 4096)
    k0, v0, _ = oracle.encode_batch(g, b.tokens, b.seq_off, None, coff, None, None, 7, 4096,
                                    with_blob=False)
    assert np.array_equal(keys, k0)                          # keys do not depend on the codec
    dirb = oracle.xp12_dir_bytes(g)
    assert dirb == 32                                        # 7 u32 -> 28 -> 32
    at = 0
    for i in range(n):
        assert int(vals["file_id"][i]) == 7 and int(vals["offset"][i]) == 4096 + at
        size = int(vals["reserved"][i])
        d = blob[at:at + dirb].view(np.uint32)[:7]
        assert d[0] == dirb and d[6] == size and np.all(np.diff(d.astype(np.int64)) > 0)
        for s in range(6):                                   # blob order K0 V0 K1 V1 K2 V2
            buf = (s & 1) * 3 + (s >> 1)
            want = oracle.xp12_slab_encode(pool[buf, pages[i]].view(np.uint16))
            assert np.array_equal(blob[at + d[s]:at + d[s + 1]], want)
        at += size
    assert at == blob.size and blob.size < n * g.chunk_bytes
    assert oracle.xp12_chunk_bound(g) == dirb + 6 * (16 + g.page_bytes)
    # decode restores the pages exactly and touches nothing else
    arena = np.concatenate([np.zeros(4096, np.uint8), blob])
    hit = nch.astype(np.uint32)
    hit[0] = 2
    dst = synth.random_pages(rng, 12, n)
    out = np.zeros_like(pool)
    recs = vals.copy()
    recs["file_id"] = 0
    oracle.decode_batch_xp12(g, coff, hit, recs, [arena], dst, out)
    touched = np.zeros(12, bool)
    for q in range(b.n):
        for j in range(int(hit[q])):
            i = int(coff[q]) + j
            assert np.array_equal(out[:, dst[i]], pool[:, pages[i]])
            touched[dst[i]] = True
    assert not out[:, ~touched].any()
    # a record whose length disagrees with the directory is refused
    bad = recs.copy()
    bad["reserved"][0] += 16
    with pytest.raises(oracle.OracleError):
        oracle.decode_batch_xp12(g, coff, hit, bad, [arena], dst, np.zeros_like(pool))
