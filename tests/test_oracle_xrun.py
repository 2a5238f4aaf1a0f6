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


def _shared_len(a, b):
    n = 0
    while n < min(len(a), len(b)) and a[n] == b[n]:
        n += 1
    return n


def _store_with_copied_records(C, seqs, file_id):
    """Records as a put after a probe writes them: chunk j of sequence s takes a copy of the record
    of the earliest stored sequence whose first (j + 1) * C tokens are the same, else a fresh one."""
    vals, fresh = [], 0
    rows = []
    for s, seq in enumerate(seqs):
        row = []
        for j in range(len(seq) // C):
            src = next((t for t in range(s) if _shared_len(seqs[t], seq) >= (j + 1) * C), None)
            if src is None:
                fresh += 1
                row.append((file_id, 16 * fresh))
            else:
                row.append(rows[src][j])
        rows.append(row)
        vals += row
    v = np.zeros(len(vals), dtype=VAL_DTYPE)
    v["file_id"] = [a for a, _ in vals]
    v["offset"] = [b for _, b in vals]
    return v, rows


def _brute_force_any_owner(C, Q, stores, pick):
    """Longest shared prefix per run, records from the holder chosen by ``pick`` (min = the first
    sequence put that reaches it, max = the last); no ordering of the stored sequences is used."""
    nq = len(Q) // C
    rec, hit = [(0, 0)] * nq, 0
    for seqs, rows in stores:                                # newest first
        lens = [_shared_len(s, Q) for s in seqs]
        m = max(lens + [0]) // C
        if m <= hit:
            continue
        owner = pick(i for i, n in enumerate(lens) if n == max(lens))
        rec[hit:m] = rows[owner][hit:m]
        hit = m
    return hit, rec


def test_records_do_not_depend_on_which_holder_is_taken():
    """With records of shared chunks copied from their first owner (the state every put after a
    probe leaves), whichever stored sequence reaches the longest shared prefix supplies the same
    records: the oracle's answer must equal a brute force that takes the first holder and one that
    takes the last, neither of which knows the neighbour rule."""
    C = 2
    g = G(C)
    rng = np.random.default_rng(11)
    stores, xruns = [], []
    for r in range(3):
        seqs = [tuple(int(t) for t in rng.integers(0, 2, rng.integers(0, 15))) for _ in range(40)]
        seqs += [(0, 1, 0, 1, 1, 1)] * 2 + [(0, 1, 0, 1)]
        v, rows = _store_with_copied_records(C, seqs, file_id=r + 1)
        b = synth.make_batch([np.array(s, np.uint32) for s in seqs])
        stores.append((seqs, rows))
        xruns.append((b.tokens, b.seq_off, v))
    queries = [tuple(int(t) for t in rng.integers(0, 2, rng.integers(0, 18))) for _ in range(200)]
    queries += [(0, 1, 0, 1, 1, 1, 0, 0), (0, 1, 0, 1, 2), ()]
    qb = synth.make_batch([np.array(q, np.uint32) for q in queries])
    qoff = synth.offsets(synth.chunk_counts(qb.seq_off, C))
    hit, recs = oracle.xprobe_batch(g, qb.tokens, qb.seq_off, qoff, xruns)
    n_multi = 0
    for q, Q in enumerate(queries):
        h_first, r_first = _brute_force_any_owner(C, Q, stores, min)
        h_last, r_last = _brute_force_any_owner(C, Q, stores, max)
        assert h_first == h_last == int(hit[q])
        assert r_first == r_last
        a = int(qoff[q])
        got = [(int(recs[a + j]["file_id"]), int(recs[a + j]["offset"])) for j in range(len(Q) // C)]
        assert got == r_first
        lens = [_shared_len(s, Q) for s in stores[0][0]]
        n_multi += sum(1 for n in lens if n == max(lens)) > 1 and max(lens) >= C
    assert n_multi > 50                       # the choice of holder was a real one in many queries
