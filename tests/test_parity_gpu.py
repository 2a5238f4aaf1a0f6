"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle -- byte
equality of keys, records, blobs, hit lengths, hit records and the whole restored pool."""
import numpy as np
import pytest
import torch

import oracle
from oracle import VAL_DTYPE
import hostindex
from paper_2511_16138_b200 import lsmkv, synth

import gpu_harness as H

pytestmark = pytest.mark.gpu

TINY = lsmkv.Geom(n_layers=4, n_kv_heads=8, head_dim=128, page_tokens=16, chunk_tokens=16)


@pytest.mark.parametrize("n_runs", [1, 2])
@pytest.mark.parametrize("tuning", [
    {},                                                     # bulk copies, 32 KiB stages
    {"copy_stage_bytes": 4096, "copy_stages": 12},
    {"copy_stage_bytes": 12288, "copy_l2_hint": 1},         # ragged last piece of a 32 KiB slab
    {"copy_mode": 1},
])
def test_config1_tiny_codec_full_compare(n_runs, tuning):
    """Config 1: 4x8x128 bf16, page 16, 32 requests x 512 tokens sharing 0-256 tokens, probes
    with the last 64 tokens re-drawn."""
    w = synth.tiny_codec()
    out = H.roundtrip(TINY, w.store, w.query, n_runs=n_runs, tuning=tuning, seed=1)
    assert np.array_equal(out["hit"], w.expected_hit_tokens // 16)
    assert out["n"] == 1024


def test_start_chunk_and_base_offset():
    w = synth.tiny_codec(n_req=12, seq_len=300)
    g = lsmkv.Geom(2, 2, 64, page_tokens=16, chunk_tokens=16, ns=7)
    rng = np.random.default_rng(3)
    start = rng.integers(0, 22, 12).astype(np.uint32)      # some beyond the 18 chunks
    start[0] = 0
    H.roundtrip(g, w.store, w.query, start_chunk=start, n_runs=3, seed=2, base_offset=4096)


@pytest.mark.parametrize("g", [
    lsmkv.Geom(3, 4, 128, page_tokens=64, chunk_tokens=64),              # 64 KiB pages
    lsmkv.Geom(2, 1, 24, elem_bytes=2, page_tokens=3, chunk_tokens=3),   # 144-byte pages
    lsmkv.Geom(1, 1, 8, elem_bytes=1, page_tokens=2, chunk_tokens=2),    # 16-byte pages
    lsmkv.Geom(5, 2, 40, elem_bytes=2, page_tokens=1, chunk_tokens=1),   # one token per chunk
    lsmkv.Geom(1, 2, 8, elem_bytes=2, page_tokens=24, chunk_tokens=24),  # a 16-token block + 8 tokens
    lsmkv.Geom(2, 1, 16, elem_bytes=2, page_tokens=40, chunk_tokens=40), # two blocks + 8 tokens
    lsmkv.Geom(1, 1, 8, elem_bytes=2, page_tokens=17, chunk_tokens=17),  # odd: no 16-byte token loads
])
@pytest.mark.parametrize("mode", [0, 1])
def test_geometries_and_ragged_lengths(g, mode):
    rng = np.random.default_rng(5)
    C = g.chunk_tokens
    lens = [0, 1, C - 1, C, C + 1, 33 * C + 2, 70 * C, 5 * C, 32 * C, 31 * C + C // 2]
    base = rng.integers(0, 5, 80 * C, dtype=np.uint32)
    seqs = []
    for n in lens:
        s = base[:n].copy()
        cut = int(rng.integers(0, n + 1))
        s[cut:] = rng.integers(5, 10, n - cut)
        seqs.append(s)
    store = synth.make_batch(seqs)
    qs = [s.copy() for s in seqs] + [base[:64 * C].copy(), rng.integers(5, 10, 9 * C, dtype=np.uint32)]
    qs[5][20 * C + 1] ^= 1
    query = synth.make_batch(qs)
    H.roundtrip(g, store, query, n_runs=2, seed=6,
                tuning={"copy_mode": mode, "copy_stage_bytes": 64})


def test_long_sequences_cross_many_warp_batches():
    g = lsmkv.Geom(1, 1, 8, elem_bytes=2, page_tokens=16, chunk_tokens=16)
    w = synth.long_context(n_req=4, seq_len=16 * 700 + 5, shared=16 * 300, n_mutate=16 * 100)
    out = H.roundtrip(g, w.store, w.query, n_runs=2, seed=7)
    assert list(out["hit"]) == [600] * 4


def test_empty_batches_and_no_runs():
    g = TINY
    with lsmkv.Context(g, 0) as ctx:
        z = torch.zeros(64, dtype=torch.uint8, device=H.DEV)
        ctx.encode_batch(0, z, z, None, z, 0, None, None, 0, 0, z, z, None, 0)
        ctx.probe_batch(0, z, z, z, 0, [], z, z, None)
        pool = H.DevPool(g, 2)
        ctx.decode_batch(0, z, 0, z, z, [(z, 64)], z, pool.table)
        # queries against an empty index: nothing is found
        b = synth.make_batch([np.arange(40, dtype=np.uint32), np.arange(3, dtype=np.uint32)])
        qoff = synth.offsets(synth.chunk_counts(b.seq_off, 16))
        hit, recs, keys, _ = H.gpu_probe(ctx, b, qoff, [])
        assert list(hit) == [0, 0] and not recs.view(np.uint8).any()
        assert np.array_equal(keys, oracle.chunk_keys(H.ogeom(g), b.seq(0)))
        H.assert_status_clean(ctx)


def test_bad_inputs_are_flagged_and_skipped_without_faulting():
    g = lsmkv.Geom(1, 1, 64, page_tokens=4, chunk_tokens=4)
    og = H.ogeom(g)
    b = synth.make_batch([np.arange(16, dtype=np.uint32)])
    coff = synth.offsets([4])
    rng = np.random.default_rng(8)
    pool_np = synth.random_pool_bytes(rng, 2, 6, g.page_bytes)
    with lsmkv.Context(g, 0) as ctx:
        pool = H.DevPool(g, 6, pool_np)
        pages = np.array([0, 9, 2, 3], dtype=np.uint32)                  # 9 is out of range
        keys, vals, blob, d_blob = H.gpu_encode(ctx, g, b, None, coff, pages, pool)
        st = ctx.last_status()
        assert st["flags"] == lsmkv.ST_BAD_PAGE and st["first_bad"] == 1
        good = np.array([0, 1, 2, 3], dtype=np.uint32)
        _, _, want, = oracle.encode_batch(og, b.tokens, b.seq_off, None, coff, good, pool_np, 0, 0)
        cb = g.chunk_bytes
        assert np.array_equal(blob[:cb], want[:cb]) and np.array_equal(blob[2 * cb:], want[2 * cb:])
        assert not blob[cb:2 * cb].any()                                 # skipped, left untouched
        # chunk_off that disagrees with the sequence lengths
        H.gpu_encode(ctx, g, b, None, synth.offsets([3]), good[:3], pool)
        assert ctx.last_status()["flags"] == lsmkv.ST_BAD_COUNT
        # records pointing outside the arena / unknown file / misaligned
        recs = np.zeros(4, dtype=VAL_DTYPE)
        recs["offset"] = [0, cb * 4, 8, cb]
        recs["file_id"] = [0, 0, 0, 3]
        dst = H.DevPool(g, 6)
        arena = torch.from_numpy(want.copy()).to(H.DEV)
        hit = np.array([4], dtype=np.uint32)
        ctx.decode_batch(1, H.dev(coff), 4, H.dev(hit), H.dev(recs), [(arena, want.size)],
                         H.dev(good), dst.table)
        st = ctx.last_status()
        assert st["flags"] == lsmkv.ST_BAD_RECORD and st["first_bad"] == 1
        out = dst.numpy()
        assert np.array_equal(out[:, 0], pool_np[:, 0]) and not out[:, 1:].any()
        # hit length larger than the query's chunk count
        ctx.decode_batch(1, H.dev(coff), 4, H.dev(np.array([5], np.uint32)), H.dev(recs),
                         [(arena, want.size)], H.dev(good), dst.table)
        assert ctx.last_status()["flags"] == lsmkv.ST_BAD_COUNT
        # host-side rejections
        with pytest.raises(lsmkv.LsmkvError) as e:
            ctx.encode_batch(1, H.dev(b.tokens), H.dev(b.seq_off), None, H.dev(coff), 4,
                             H.dev(good), pool.table, 0, 0, H.dev(keys), H.dev(vals), d_blob,
                             4 * cb - 1)
        assert e.value.code == lsmkv.ECAPACITY
        with pytest.raises(lsmkv.LsmkvError):
            ctx.set_tuning("no_such_knob", 1)


def test_extreme_token_ids_and_namespace():
    """Token ids up to 2^32-1 (t + 1 needs 33 bits), the largest namespace, and sequences built
    from the token triples whose digest is exactly zero."""
    import json
    import os
    with open(os.path.join(os.path.dirname(__file__), "golden", "digest_zero_sequences.json")) as f:
        zero = json.load(f)["zero_digest"]
    g = lsmkv.Geom(2, 1, 32, page_tokens=3, chunk_tokens=3, ns=0xFFFFFFFF)   # 192-byte pages
    rng = np.random.default_rng(12)
    seqs = [np.full(3 * 40, 0xFFFFFFFF, dtype=np.uint32),
            rng.integers(2**32 - 5, 2**32, 3 * 33 + 1, dtype=np.uint64).astype(np.uint32),
            np.array(zero[0] * 7, dtype=np.uint32),          # lane A digest returns to 0 every chunk
            np.array(zero[1] * 5 + [1, 2], dtype=np.uint32),
            np.zeros(3 * 35, dtype=np.uint32)]
    store = synth.make_batch(seqs)
    query = synth.make_batch([s.copy() for s in seqs] + [np.array(zero[0] * 9, dtype=np.uint32)])
    out = H.roundtrip(g, store, query, n_runs=2, seed=13)
    assert list(out["hit"]) == [40, 33, 7, 5, 35, 7]


@pytest.mark.parametrize("tuning", [{"probe_warps_per_cta": 1}, {"probe_warps_per_cta": 2},
                                    {"probe_warps_per_cta": 8}, {"copy_ctas_per_sm": 4, "copy_stages": 3},
                                    {"copy_mode": 1, "simt_ctas_per_sm": 1}])
def test_launch_shapes_do_not_change_results(tuning):
    """Every tuning knob is a launch shape only: long sequences (many rounds per query whatever
    the CTA width), several runs, start chunks -- same bytes as the oracle."""
    g = lsmkv.Geom(2, 2, 32, page_tokens=16, chunk_tokens=16)
    w = synth.long_context(n_req=5, seq_len=16 * 530 + 7, shared=16 * 200, n_mutate=16 * 40 + 3)
    start = np.array([0, 3, 200, 529, 600], dtype=np.uint32)
    H.roundtrip(g, w.store, w.query, start_chunk=start, n_runs=3, tuning=tuning, seed=17)


def test_more_queries_than_the_hand_out_order_covers():
    """Batches beyond 65 536 queries are handed out in their given order (no length sort): the
    answers must not depend on which of the two the probe does."""
    g = lsmkv.Geom(1, 1, 8, elem_bytes=2, page_tokens=4, chunk_tokens=4)
    og = H.ogeom(g)
    rng = np.random.default_rng(21)
    stored = [rng.integers(0, 3, int(rng.integers(4, 40)), dtype=np.uint32) for _ in range(300)]
    store = synth.make_batch(stored)
    coff = synth.offsets(synth.chunk_counts(store.seq_off, 4))
    n_q = 70_000
    lens = rng.integers(0, 30, n_q)
    toks = rng.integers(0, 3, int(lens.sum()), dtype=np.uint32)
    q_off = np.concatenate([[0], np.cumsum(lens)]).astype(np.uint64)
    # every third query starts with a stored sequence
    for i in range(0, n_q, 3):
        s = stored[i % len(stored)]
        m = min(len(s), int(lens[i]))
        toks[int(q_off[i]):int(q_off[i]) + m] = s[:m]
    query = synth.Batch(toks, q_off)
    qoff = synth.offsets(synth.chunk_counts(query.seq_off, 4))
    with lsmkv.Context(g, 0) as ctx:
        keys, vals, _, _ = H.gpu_encode(ctx, g, store, None, coff, None, None)
        run = H.gpu_flush_run(ctx, keys, vals)
        o_hit, o_recs, _, _ = oracle.probe_batch(og, query.tokens, query.seq_off, qoff, [run])
        hit, recs, _, _ = H.gpu_probe(ctx, query, qoff, [run], want_keys=False)
        assert np.array_equal(hit, o_hit) and np.array_equal(recs, o_recs)
        assert 10_000 < int((o_hit > 0).sum()) < n_q
        assert ctx.last_status()["flags"] == 0


@pytest.mark.parametrize("extra", [-1, 0, 1, 700])
def test_as_many_queries_as_resident_ctas_and_one_more(extra):
    """Up to six CTAs of four warps per SM a probe through hash indexes gives every query a CTA
    of its own (no hand-out order, no counter); one query more and the queries are ordered and
    drawn from a counter. Both sides of that edge, and well beyond it, equal the oracle."""
    g = lsmkv.Geom(1, 1, 8, elem_bytes=2, page_tokens=4, chunk_tokens=4)
    og = H.ogeom(g)
    rng = np.random.default_rng(31 + extra)
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    n_q = 6 * sms + extra
    stored = [rng.integers(0, 3, int(rng.integers(4, 400)), dtype=np.uint32) for _ in range(200)]
    store = synth.make_batch(stored)
    coff = synth.offsets(synth.chunk_counts(store.seq_off, 4))
    qs = []
    for i in range(n_q):
        q = rng.integers(0, 3, int(rng.integers(0, 500)), dtype=np.uint32)
        if i % 2 == 0:                                         # starts with a stored sequence
            s = stored[i % len(stored)]
            m = min(len(s), len(q))
            q[:m] = s[:m]
        qs.append(q)
    query = synth.make_batch(qs)
    qoff = synth.offsets(synth.chunk_counts(query.seq_off, 4))
    with lsmkv.Context(g, 0) as ctx:
        keys, vals, _, _ = H.gpu_encode(ctx, g, store, None, coff, None, None)
        run = H.gpu_flush_run(ctx, keys, vals)
        o_hit, o_recs, o_keys, _ = oracle.probe_batch(og, query.tokens, query.seq_off, qoff, [run],
                                                      want_keys=True)
        for want_keys in (False, True):
            hit, recs, qk, _ = H.gpu_probe(ctx, query, qoff, [run], want_keys=want_keys)
            assert np.array_equal(hit, o_hit) and np.array_equal(recs, o_recs)
            if want_keys:
                assert np.array_equal(qk, o_keys)
        assert int((o_hit > 0).sum()) > n_q // 4
        assert ctx.last_status()["flags"] == 0


@pytest.mark.parametrize("n_runs", [5, 11, 64])
def test_many_runs_are_searched_in_groups_newest_first(n_runs):
    """More runs than one lock-step group holds (4), up to the most a probe accepts; keys are
    dealt to the runs at random, so a query's chunks are answered by many different runs."""
    g = lsmkv.Geom(1, 2, 32, elem_bytes=2, page_tokens=8, chunk_tokens=8)
    w = synth.tiny_codec(n_req=10, seq_len=8 * 50 + 3, max_shared=200, n_mutate=40, config_id=60)
    out = H.roundtrip(g, w.store, w.query, n_runs=n_runs, seed=n_runs)
    assert np.array_equal(out["hit"], w.expected_hit_tokens // 8)


@pytest.mark.parametrize("shift", [0, 1, 2, 3])
@pytest.mark.parametrize("C", [16, 32, 20])
def test_keys_do_not_depend_on_where_the_token_array_starts(shift, C):
    """The token array starts `shift` tokens past a 16-byte boundary and ends with the last token
    of the last chunk. A block of 16 tokens is fetched with the aligned 16-byte loads that cover
    it where those stay inside the array up to the end of its sequence, and token by token at the
    edges; sequences of odd lengths packed back to back give every misalignment in one batch.
    Keys from the encoder and from both probes equal the oracle's, and every stored chunk hits."""
    g = lsmkv.Geom(2, 1, 32, page_tokens=C, chunk_tokens=C)
    og = H.ogeom(g)
    rng = np.random.default_rng(100 + 4 * C + shift)
    lens = [3 * C, 2 * C + 5, 7, 40 * C + 1, 33 * C + 2, C + 3, 5 * C]
    batch = synth.make_batch([rng.integers(0, 2**32, n, dtype=np.uint64).astype(np.uint32)
                              for n in lens])
    want = np.concatenate([oracle.chunk_keys(og, batch.seq(i)) for i in range(batch.n)])
    nch = synth.chunk_counts(batch.seq_off, C)
    coff = synth.offsets(nch)
    n = int(coff[-1])
    assert int(batch.seq_off[-1]) == sum(lens) and lens[-1] % C == 0   # the array ends with a chunk
    raw = torch.zeros(4 * (shift + len(batch.tokens)), dtype=torch.uint8, device=H.DEV)
    assert raw.data_ptr() % 16 == 0
    d_tok = raw[4 * shift:]
    d_tok.copy_(torch.from_numpy(batch.tokens.view(np.uint8).copy()))
    assert d_tok.data_ptr() % 16 == 4 * shift
    with lsmkv.Context(g, 0) as ctx:
        d_off, d_coff = H.dev(batch.seq_off), H.dev(coff)
        d_keys = torch.zeros(n * 32, dtype=torch.uint8, device=H.DEV)
        d_vals = torch.zeros(n * 16, dtype=torch.uint8, device=H.DEV)
        ctx.encode_batch(batch.n, d_tok, d_off, None, d_coff, n, None, None, 0, 0, d_keys, d_vals,
                         None, 0)
        torch.cuda.synchronize()
        keys = H.host(d_keys, np.uint64, n * 32).reshape(-1, 4)
        assert np.array_equal(keys, want)
        vals = H.host(d_vals, VAL_DTYPE, n * 16)
        run = H.gpu_flush_run(ctx, keys, vals)
        druns, keep = H.dev_runs([run])
        hruns, hkeep = H.with_hindex(ctx, druns)
        for rr in (druns, hruns):
            d_hit = torch.full((batch.n,), -1, dtype=torch.int32, device=H.DEV)
            d_recs = torch.full((n * 16,), 0xAB, dtype=torch.uint8, device=H.DEV)
            d_qk = torch.zeros(n * 32, dtype=torch.uint8, device=H.DEV)
            ctx.probe_batch(batch.n, d_tok, d_off, d_coff, n, rr, d_hit, d_recs, d_qk)
            torch.cuda.synchronize()
            assert np.array_equal(d_hit.cpu().numpy().view(np.uint32), nch.astype(np.uint32))
            assert np.array_equal(H.host(d_qk, np.uint64, n * 32).reshape(-1, 4), want)
            assert np.array_equal(H.host(d_recs, VAL_DTYPE, n * 16), vals)
        H.assert_status_clean(ctx)
