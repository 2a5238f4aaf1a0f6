"""Pins for the oracle's probe: the longest cached prefix (App. B "Probe") checked against a
brute force that never builds a key -- a set of token tuples -- and against planted hit
lengths from the generators."""
import numpy as np

import oracle
from oracle import Geom, VAL_DTYPE
from paper_2511_16138_b200 import synth


def G(C):
    return Geom(n_layers=1, n_kv_heads=1, head_dim=8, page_tokens=C, chunk_tokens=C)


def store_as_runs(g, batch, n_runs, rng, start=None):
    """Encode (index-only), deal keys to runs at random, flush each."""
    nch = synth.chunk_counts(batch.seq_off, g.chunk_tokens)
    st = np.zeros(batch.n, np.uint32) if start is None else start
    coff = synth.offsets(np.maximum(nch - st.astype(np.int64), 0))
    keys, vals, _ = oracle.encode_batch(g, batch.tokens, batch.seq_off, st, coff, None, None,
                                        0, 0, with_blob=False)
    vals["offset"] = np.arange(len(vals)) * 16 + 16        # distinct, non-zero records
    owner = rng.integers(0, n_runs, len(keys))
    return [oracle.flush(keys[owner == r], vals[owner == r]) for r in range(n_runs)], keys, vals


def brute_hits(C, store, query):
    have = set()
    for i in range(store.n):
        s = store.seq(i)
        for j in range(len(s) // C):
            have.add(tuple(int(t) for t in s[:(j + 1) * C]))
    hits = []
    for q in range(query.n):
        s = query.seq(q)
        h = 0
        while h < len(s) // C and tuple(int(t) for t in s[:(h + 1) * C]) in have:
            h += 1
        hits.append(h)
    return np.array(hits)


def test_probe_equals_token_tuple_brute_force_tiny_alphabet():
    C = 2
    rng = np.random.default_rng(1)
    store = synth.make_batch([rng.integers(0, 3, rng.integers(0, 13), dtype=np.uint32)
                              for _ in range(40)])
    query = synth.make_batch([rng.integers(0, 3, rng.integers(0, 15), dtype=np.uint32)
                              for _ in range(64)])
    runs, keys, vals = store_as_runs(G(C), store, 3, rng)
    qoff = synth.offsets(synth.chunk_counts(query.seq_off, C))
    hit, recs, qkeys, lookups = oracle.probe_batch(G(C), query.tokens, query.seq_off, qoff, runs,
                                                   want_keys=True)
    want = brute_hits(C, store, query)
    assert np.array_equal(hit, want) and want.max() >= 3 and want.min() == 0
    for q in range(query.n):
        a, b = int(qoff[q]), int(qoff[q + 1])
        assert np.array_equal(qkeys[a:b], oracle.chunk_keys(G(C), query.seq(q)))
        for j in range(b - a):
            if j < hit[q]:
                assert recs[a + j] == oracle.lookup(runs, qkeys[a + j])[0]
                assert int(recs[a + j]["offset"]) != 0
            else:
                assert recs[a + j] == np.zeros(1, VAL_DTYPE)[0]      # zero-filled past the hit
    nch = synth.chunk_counts(query.seq_off, C)
    assert lookups == int(np.sum(np.minimum(want + 1, nch)))       # stops at the first miss


def test_probe_planted_hits_tiny_codec():
    w = synth.tiny_codec(n_req=8, seq_len=128, max_shared=64, n_mutate=32)
    g = G(16)
    rng = np.random.default_rng(2)
    for n_runs in (1, 2):
        runs, _, _ = store_as_runs(g, w.store, n_runs, rng)
        qoff = synth.offsets(synth.chunk_counts(w.query.seq_off, 16))
        hit, recs, _, _ = oracle.probe_batch(g, w.query.tokens, w.query.seq_off, qoff, runs)
        assert np.array_equal(hit, w.expected_hit_tokens // 16) and hit[0] == 6


def test_probe_planted_hits_probe_heavy_small():
    w = synth.probe_heavy(n_keys=6000, run_sizes=(60, 540, 5400), n_query=80, min_len=64,
                          max_len=1024, n_prefix=8)
    g = G(16)
    nch = synth.chunk_counts(w.store.seq_off, 16)
    coff = synth.offsets(nch - w.store_start_chunk)
    assert int(coff[-1]) == w.n_stored
    keys, vals, _ = oracle.encode_batch(g, w.store.tokens, w.store.seq_off, w.store_start_chunk,
                                        coff, None, None, 0, 0, with_blob=False)
    assert len(np.unique(keys, axis=0)) == w.n_stored          # generator promised unique keys
    vals["offset"] = (np.arange(w.n_stored) % 64) * 512
    runs = []
    for r in range(3):
        sel = w.run_of_key == r
        k, v = keys[sel], vals[sel].copy()
        d = w.dup_idx[w.dup_run == r]
        dv = vals[d].copy()
        dv["offset"] += 7                                       # newer copy, different record
        runs.append(oracle.flush(np.concatenate([k, keys[d]]), np.concatenate([v, dv])))
    assert [len(k) for k, _ in runs] == [60 + (w.dup_run == 0).sum(), 540 + (w.dup_run == 1).sum(),
                                          5400]
    qoff = synth.offsets(synth.chunk_counts(w.query.seq_off, 16))
    hit, recs, qkeys, _ = oracle.probe_batch(g, w.query.tokens, w.query.seq_off, qoff, runs,
                                             want_keys=True)
    assert np.array_equal(hit, w.expected_hit)
    assert 0.4 < (hit > 0).mean() < 0.8
    assert np.array_equal(hit, brute_hits(16, w.store, w.query))
    # the planted newer duplicates decide their lookups
    dupset = {tuple(int(x) for x in keys[i]) for i in w.dup_idx}
    seen_dup = 0
    for q in range(w.query.n):
        for j in range(int(hit[q])):
            i = int(qoff[q]) + j
            if tuple(int(x) for x in qkeys[i]) in dupset:
                assert int(recs[i]["offset"]) % 512 == 7
                seen_dup += 1
            else:
                assert int(recs[i]["offset"]) % 512 == 0
    assert seen_dup > 0


def test_first_miss_rule_on_a_store_that_is_not_prefix_closed():
    """With chunk 1 missing, the longest fully cached prefix is 1 chunk although chunks 2..3
    are present; a binary search over the prefix length would be free to answer otherwise."""
    g = G(2)
    toks = np.arange(8, dtype=np.uint32)
    k = oracle.chunk_keys(g, toks)
    v = np.zeros(4, VAL_DTYPE)
    v["offset"] = [16, 32, 48, 64]
    keep = [0, 2, 3]
    run = oracle.flush(k[keep], v[keep])
    hit, recs, _, lookups = oracle.probe_batch(g, toks, np.array([0, 8], np.uint64),
                                               np.array([0, 4], np.uint64), [run])
    assert hit[0] == 1 and lookups == 2
    assert [int(x) for x in recs["offset"]] == [16, 0, 0, 0]


def test_binary_search_over_prefix_length_agrees_on_prefix_closed_stores():
    """The paper's probe is a binary search over prefix length with point lookups; on a
    prefix-closed store it returns the first-miss answer."""
    C = 4
    rng = np.random.default_rng(5)
    base = rng.integers(0, 50, 200, dtype=np.uint32)
    store = synth.make_batch([base[:n] for n in (200, 64, 120)])
    g = G(C)
    runs, _, _ = store_as_runs(g, store, 2, rng)
    queries = []
    for cut in (0, 3, 4, 37, 120, 199, 200):
        q = rng.integers(50, 100, 220, dtype=np.uint32)
        q[:cut] = base[:cut]
        queries.append(q)
    query = synth.make_batch(queries)
    qoff = synth.offsets(synth.chunk_counts(query.seq_off, C))
    hit, _, qkeys, _ = oracle.probe_batch(g, query.tokens, query.seq_off, qoff, runs,
                                          want_keys=True)
    for q in range(query.n):
        ks = qkeys[int(qoff[q]):int(qoff[q + 1])]
        lo, hi = 0, len(ks)              # invariant: chunks < lo present, chunk hi absent
        while lo < hi:
            mid = (lo + hi) // 2
            if oracle.lookup(runs, ks[mid]) is not None:
                lo = mid + 1
            else:
                hi = mid
        assert lo == hit[q]
    assert list(hit) == [0, 0, 1, 9, 30, 49, 50]


def test_empty_and_short_queries():
    g = G(16)
    rng = np.random.default_rng(6)
    store = synth.make_batch([rng.integers(0, 9, 64, dtype=np.uint32)])
    runs, _, _ = store_as_runs(g, store, 1, rng)
    query = synth.make_batch([store.seq(0)[:15], store.seq(0)[:16], np.zeros(0, np.uint32)])
    qoff = synth.offsets(synth.chunk_counts(query.seq_off, 16))
    hit, recs, _, _ = oracle.probe_batch(g, query.tokens, query.seq_off, qoff, runs)
    assert list(hit) == [0, 1, 0] and len(recs) == 1
    hit, _, _, _ = oracle.probe_batch(g, query.tokens, query.seq_off, qoff, [])
    assert list(hit) == [0, 0, 0]
