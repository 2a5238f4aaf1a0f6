"""Hash indexes of runs on the GPU: the table holds exactly the entries of the run's keys and
every key is found in it by the oracle's lookup rule (slot order inside the table depends on
insertion order, so the bytes need not equal the oracle's), and probing through hash indexes
gives exactly the answers of the searching probe and of the oracle."""
import numpy as np
import pytest
import torch

import oracle
from oracle import VAL_DTYPE
from paper_2511_16138_b200 import lsmkv, synth

import gpu_harness as H

pytestmark = pytest.mark.gpu

G = lsmkv.Geom(1, 1, 8, elem_bytes=2, page_tokens=16, chunk_tokens=16)


def digest_keys(rng, n, w1_hi=2**61 - 1):
    k = np.zeros((n, 4), dtype=np.uint64)
    k[:, 0] = rng.integers(0, 3000, n)
    k[:, 1] = rng.integers(0, w1_hi, n, dtype=np.uint64)
    k[:, 2] = rng.integers(0, 2**61 - 1, n, dtype=np.uint64)
    k[:, 3] = rng.integers(0, 2**64, n, dtype=np.uint64)
    return k


def gpu_hindex(ctx, keys_dev, n):
    nb = lsmkv.lsmkv_hindex_buckets(n)
    out = torch.full((nb * 32,), 0xFF, dtype=torch.uint8, device=H.DEV)
    ctx.hindex_build(keys_dev, n, out)
    torch.cuda.synchronize()
    return out, nb


@pytest.mark.parametrize("n,w1_hi", [(0, 2**61 - 1), (1, 2**61 - 1), (2, 2**61 - 1),
                                      (9, 2**61 - 1), (1000, 2**61 - 1), (123457, 2**61 - 1),
                                      (5000, 2**61 // 40)])
def test_table_is_valid_for_the_oracles_lookup(n, w1_hi):
    rng = np.random.default_rng(n + 1)
    keys = digest_keys(rng, n, w1_hi)                    # last case: crowded buckets, long chains
    with lsmkv.Context(G, 0) as ctx:
        out, nb = gpu_hindex(ctx, H.dev(keys), n)
        assert nb == oracle.hindex_buckets(n)
        table = out.cpu().numpy().view(np.uint32)
        want = oracle.hindex_build(keys)
        assert table.size == want.size
        assert np.array_equal(np.sort(table[table != 0]), np.sort(want[want != 0]))
        step = max(1, n // 3000)
        for i in range(0, n, step):
            assert oracle.hindex_find(table, keys, keys[i]) == i
        for k in digest_keys(rng, 200, w1_hi):
            assert oracle.hindex_find(table, keys, k) == -1


def test_build_refuses_runs_beyond_24_bit_positions():
    with lsmkv.Context(G, 0) as ctx:
        buf = torch.zeros(64, dtype=torch.uint8, device=H.DEV)
        rc = lsmkv.lib().lsmkv_hindex_build(ctx.handle, None, buf.data_ptr(), 2**24 - 1,
                                            buf.data_ptr())
        assert rc == lsmkv.EINVAL


def off16(t):
    """A copy of a device byte tensor that starts 16 bytes past a 32-byte boundary."""
    buf = torch.empty(t.numel() + 48, dtype=torch.uint8, device=t.device)
    at = 16 + (-buf.data_ptr()) % 32
    out = buf[at:at + t.numel()]
    out.copy_(t.view(torch.uint8).reshape(-1))
    return out


def build_runs(ctx, w, g):
    nch = synth.chunk_counts(w.store.seq_off, 16)
    coff = synth.offsets(nch - w.store_start_chunk)
    keys, _, _, _ = H.gpu_encode(ctx, g, w.store, w.store_start_chunk, coff, None, None)
    vals = np.zeros(w.n_stored, dtype=VAL_DTYPE)
    vals["offset"] = np.arange(w.n_stored) * 16 + 16
    runs = []
    for r in range(4):
        sel = w.run_of_key == r
        d = w.dup_idx[w.dup_run == r]
        dv = vals[d].copy()
        dv["file_id"] = 1
        runs.append(H.gpu_flush_run(ctx, np.concatenate([keys[sel], keys[d]]),
                                    np.concatenate([vals[sel], dv])))
    return runs


def probe(ctx, w, qoff, total, rr, batch):
    d_tok, d_off, d_qoff = H.dev(batch.tokens), H.dev(batch.seq_off), H.dev(qoff)
    d_hit = torch.full((batch.n,), -1, dtype=torch.int32, device=H.DEV)
    d_recs = torch.full((max(1, total) * 16,), 0xAB, dtype=torch.uint8, device=H.DEV)
    ctx.probe_batch(batch.n, d_tok, d_off, d_qoff, total, rr, d_hit, d_recs, None)
    torch.cuda.synchronize()
    st = ctx.last_status()
    assert st["flags"] == 0
    return d_hit.cpu().numpy().view(np.uint32), H.host(d_recs, VAL_DTYPE, total * 16), st


@pytest.mark.parametrize("which", ["queries", "stored"])
def test_probe_through_hash_indexes_equals_the_searching_probe_and_the_oracle(which):
    w = synth.probe_heavy(n_keys=60000, run_sizes=(60, 540, 5400, 54000), n_query=300,
                          min_len=64, max_len=4096, n_prefix=16)
    g, og = G, H.ogeom(G)
    # "stored": every stored sequence is probed, so every key of the store is looked up --
    # also the few that were pushed out of their home bucket
    batch = w.query if which == "queries" else w.store
    with lsmkv.Context(g, 0) as ctx:
        runs = build_runs(ctx, w, g)
        qoff = synth.offsets(synth.chunk_counts(batch.seq_off, 16))
        total = int(qoff[-1])
        o_hit, o_recs, _, _ = oracle.probe_batch(og, batch.tokens, batch.seq_off, qoff, runs)
        druns, keep = H.dev_runs(runs)
        hashed, tables = [], []
        for (dk, dv, n), (k, _) in zip(druns, runs):
            t, nb = gpu_hindex(ctx, dk, n)
            tables.append(t)
            hashed.append((dk, dv, n, None, 0, t, nb))
        mixed = hashed[:2] + [druns[2]] + hashed[3:]       # one run without a table: all searched
        # keys and tables 16 bytes off a 32-byte boundary: the probe may not use 32-byte loads
        odd = [(off16(dk), dv, n, None, 0, off16(t), nb) for (dk, dv, n, _, _, t, nb) in hashed]
        assert all(r[0].data_ptr() % 32 == 16 and r[5].data_ptr() % 32 == 16 for r in odd)
        ctx.last_status()
        for rr in (druns, hashed, mixed, odd):
            hit, recs, st = probe(ctx, w, qoff, total, rr, batch)
            assert np.array_equal(hit, o_hit) and np.array_equal(recs, o_recs)
            assert st["chunks_hit"] == int(o_hit.sum())
        if which == "queries":
            assert np.array_equal(o_hit, w.expected_hit.astype(np.uint32))
        else:
            assert int(o_hit.sum()) >= w.n_stored            # shared prefixes count once per sequence


def test_hash_index_over_a_padded_flush_output_and_an_empty_run():
    rng = np.random.default_rng(5)
    g, og = G, H.ogeom(G)
    w = synth.tiny_codec(n_req=6, seq_len=256, max_shared=128, n_mutate=32)
    nch = synth.chunk_counts(w.store.seq_off, 16)
    coff = synth.offsets(nch)
    with lsmkv.Context(g, 0) as ctx:
        keys, _, _, _ = H.gpu_encode(ctx, g, w.store, None, coff, None, None)
        n = len(keys)
        vals = np.zeros(2 * n, dtype=VAL_DTYPE)
        vals["offset"] = np.arange(2 * n) * 16
        both = np.concatenate([keys, keys])                    # every key twice: half is padding
        ok = torch.empty(2 * n * 32, dtype=torch.uint8, device=H.DEV)
        ov = torch.empty(2 * n * 16, dtype=torch.uint8, device=H.DEV)
        cnt = torch.zeros(1, dtype=torch.int64, device=H.DEV)
        ctx.flush_batch(H.dev(both), H.dev(vals), 2 * n, ok, ov, cnt)
        t, nb = gpu_hindex(ctx, ok, 2 * n)                     # built over the padded length
        n_real = int(cnt.item())
        table = t.cpu().numpy().view(np.uint32)
        assert int((table != 0).sum()) == n_real
        run_keys = H.host(ok, np.uint64, 2 * n * 32).reshape(-1, 4)
        run_vals = H.host(ov, VAL_DTYPE, 2 * n * 16)
        empty = torch.zeros(32, dtype=torch.uint8, device=H.DEV)
        rr = [(empty, empty, 0, None, 0, None, 0), (ok, ov, 2 * n, None, 0, t, nb)]
        qoff = synth.offsets(synth.chunk_counts(w.query.seq_off, 16))
        total = int(qoff[-1])
        o_hit, o_recs, _, _ = oracle.probe_batch(og, w.query.tokens, w.query.seq_off, qoff,
                                                 [(run_keys[:n_real], run_vals[:n_real])])
        hit, recs, _ = probe(ctx, w, qoff, total, rr, w.query)
        assert np.array_equal(hit, o_hit) and np.array_equal(recs, o_recs)
        assert np.array_equal(hit, (w.expected_hit_tokens // 16).astype(np.uint32))
