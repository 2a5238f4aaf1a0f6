"""Pins for the oracle's exact prefix index: its hit lengths must equal those of the digest-keyed
probe on the same stores (two independent routes to the longest cached prefix), its records the
owner rule worked out with Python tuples, and planted hit lengths of the generators."""
import numpy as np

import oracle
from oracle import Geom, VAL_DTYPE
from paper_2511_16138_b200 import synth


def G(C):
    return Geom(n_layers=1, n_kv_heads=1, head_dim=8, page_tokens=C, chunk_tokens=C)


def make_xrun(g, batch, file_id):
    nch = synth.chunk_counts(batch.seq_off, g.chunk_tokens)
    v = np.zeros(int(nch.sum()), dtype=VAL_DTYPE)
    v["file_id"] = file_id
    v["offset"] = np.arange(len(v)) * 16 + 16
    return (batch.tokens, batch.seq_off, v), nch


def py_expected(C, query, stores):
    """The definition with Python tuples (tuple order: a prefix is smaller). Per run: L = longest
    shared token prefix; the records come from the neighbour of Q among the sequences reaching L:
    the largest (sequence, arrival) not above Q, else the smallest above."""
    hits, recs = [], []
    for q in range(query.n):
        Q = tuple(int(t) for t in query.seq(q))
        nq = len(Q) // C
        rec = [None] * nq
        hit = 0
        for (batch, vals) in stores:                         # newest first
            seqs = [tuple(int(t) for t in batch.seq(s)) for s in range(batch.n)]
            coff = np.concatenate([[0], np.cumsum([len(s) // C for s in seqs])])

            def shared(s):
                n = 0
                while n < min(len(Q), len(s)) and Q[n] == s[n]:
                    n += 1
                return n
            L = max([shared(s) for s in seqs] + [0])
            m = L // C
            if m <= hit:
                continue
            reach = [i for i, s in enumerate(seqs) if shared(s) == L]
            below = [i for i in reach if seqs[i] <= Q]
            above = [i for i in reach if seqs[i] > Q]
            owner = (max(below, key=lambda i: (seqs[i], i)) if below
                     else min(above, key=lambda i: (seqs[i], i)))
            for j in range(hit, m):
                rec[j] = (int(vals["file_id"][coff[owner] + j]), int(vals["offset"][coff[owner] + j]))
            hit = m
        hits.append(hit)
        recs.append(rec)
    return hits, recs


def test_tiny_alphabet_against_python_tuples():
    C = 2
    g = G(C)
    rng = np.random.default_rng(1)
    stores = []
    for r in range(3):
        b = synth.make_batch([rng.integers(0, 2, rng.integers(0, 14), dtype=np.uint32)
                              for _ in range(12)] + [np.array([0, 1, 0, 1], np.uint32)] * 2)
        (t, so, v), _ = make_xrun(g, b, r)
        stores.append((b, v))
    query = synth.make_batch([rng.integers(0, 2, rng.integers(0, 16), dtype=np.uint32)
                              for _ in range(60)] + [np.array([0, 1, 0, 1, 2, 2], np.uint32)])
    qoff = synth.offsets(synth.chunk_counts(query.seq_off, C))
    hit, recs = oracle.xprobe_batch(g, query.tokens, query.seq_off, qoff,
                                    [(b.tokens, b.seq_off, v) for b, v in stores])
    want_hit, want_recs = py_expected(C, query, stores)
    assert list(hit) == want_hit and max(want_hit) >= 3
    for q in range(query.n):
        a = int(qoff[q])
        for j, w in enumerate(want_recs[q]):
            got = (int(recs[a + j]["file_id"]), int(recs[a + j]["offset"]))
            assert got == (w if w is not None else (0, 0))


def test_hits_equal_the_digest_probe_on_the_same_store():
    """Two independent routes: exact token comparison here, digest keys + sorted runs there."""
    g = G(16)
    w = synth.probe_heavy(n_keys=5000, run_sizes=(50, 450, 4500), n_query=60, min_len=64,
                          max_len=900, n_prefix=6)
    # the exact index stores whole sequences, so compare on the whole-sequence store
    store = w.store
    nch = synth.chunk_counts(store.seq_off, 16)
    coff = synth.offsets(nch)
    keys, vals, _ = oracle.encode_batch(g, store.tokens, store.seq_off, None, coff, None, None,
                                        0, 0, with_blob=False)
    run = oracle.flush(keys, vals)
    qoff = synth.offsets(synth.chunk_counts(w.query.seq_off, 16))
    d_hit, _, _, _ = oracle.probe_batch(g, w.query.tokens, w.query.seq_off, qoff, [run])
    x_hit, x_recs = oracle.xprobe_batch(g, w.query.tokens, w.query.seq_off, qoff,
                                        [(store.tokens, store.seq_off, vals)])
    assert np.array_equal(x_hit, d_hit) and np.array_equal(x_hit, w.expected_hit.astype(np.uint32))
    assert (x_hit > 0).sum() > 20
    # every returned record is a record of a chunk with that index (offset = i * chunk_bytes)
    for q in range(w.query.n):
        for j in range(int(x_hit[q])):
            assert int(x_recs[int(qoff[q]) + j]["offset"]) % g.chunk_bytes == 0


def test_planted_hits_and_newest_run_wins():
    g = G(16)
    w = synth.tiny_codec(n_req=6, seq_len=160, max_shared=64, n_mutate=48)
    (x_old, _), (x_new, _) = make_xrun(g, w.store, 7), make_xrun(g, synth.make_batch(
        [w.store.seq(0)[:64], w.store.seq(1)[:32]]), 9)
    qoff = synth.offsets(synth.chunk_counts(w.query.seq_off, 16))
    hit, recs = oracle.xprobe_batch(g, w.query.tokens, w.query.seq_off, qoff, [x_new, x_old])
    assert list(hit) == [7] * 6
    a = int(qoff[0])
    assert [int(r["file_id"]) for r in recs[a:a + 7]] == [9, 9, 9, 9, 7, 7, 7]
    a = int(qoff[1])
    assert [int(r["file_id"]) for r in recs[a:a + 3]] == [9, 9, 7]
    hit2, _ = oracle.xprobe_batch(g, w.query.tokens, w.query.seq_off, qoff, [])
    assert not hit2.any()


def test_order_is_pythons_tuple_order():
    rng = np.random.default_rng(5)
    seqs = [rng.integers(0, 3, rng.integers(0, 9), dtype=np.uint32) for _ in range(300)]
    seqs += [np.array([2**32 - 1, 0], np.uint32), np.array([2**31, 5], np.uint32),
             np.array([], np.uint32), np.array([], np.uint32)]
    b = synth.make_batch(seqs)
    want = sorted(range(b.n), key=lambda i: (tuple(int(t) for t in b.seq(i)), i))
    assert list(oracle.xrun_order(b.tokens, b.seq_off)) == want
