"""An index under the (T, K) compaction policy, end to end on the GPU: batches of real chunk keys
(with keys repeated across batches) are flushed and compacted as the planner says; the device
runs must equal the oracle's runs put through the same plan byte for byte, lookups must give
what a dict that keeps the newest record gives, and probes through the index must equal the
oracle's."""
import numpy as np
import pytest
import torch

import oracle
from oracle import VAL_DTYPE
from paper_2511_16138_b200 import lsmkv, synth
from paper_2511_16138_b200.lsmindex import LsmIndex

import gpu_harness as H

pytestmark = pytest.mark.gpu

G = lsmkv.Geom(1, 1, 8, elem_bytes=2, page_tokens=16, chunk_tokens=16)


def alloc(nbytes):
    return torch.empty(max(16, nbytes), dtype=torch.uint8, device=H.DEV)


def oracle_compact(runs, levels, M, T, K):
    """The oracle's runs (newest first) through the same planner."""
    while True:
        plan = lsmkv.lsmkv_plan_compaction(levels, [len(k) for k, _ in runs], M, T, K)
        if plan is None:
            return
        a, cnt, to = plan
        if cnt > 1:
            runs[a:a + cnt] = [oracle.merge_runs(runs[a:a + cnt])]
        levels[a:a + cnt] = [to]


@pytest.mark.parametrize("T,K", [(2, 1), (4, 1), (4, 3), (3, 2)])
def test_index_under_the_policy_equals_the_oracle_and_a_dict(T, K):
    g, og = G, H.ogeom(G)
    rng = np.random.default_rng(10 * T + K)
    M = 200
    # a pool of sequences with shared prefixes; every batch re-inserts some earlier sequences
    w = synth.probe_heavy(n_keys=6000, run_sizes=(60, 540, 2400, 3000), n_query=120, min_len=64,
                          max_len=1024, n_prefix=8)
    seqs = [w.store.seq(i) for i in range(w.store.n)]
    newest = {}
    with lsmkv.Context(g, 0) as ctx:
        idx = LsmIndex(ctx, alloc, M, T, K)
        o_runs, o_levels = [], []
        for b in range(14):
            pick = rng.choice(len(seqs), size=int(rng.integers(2, 6)), replace=False)
            batch = synth.make_batch([seqs[i] for i in pick])
            coff = synth.offsets(synth.chunk_counts(batch.seq_off, 16))
            n = int(coff[-1])
            keys, vals, _, _ = H.gpu_encode(ctx, g, batch, None, coff, None, None, file_id=b,
                                            base_offset=1000 * b)
            d_keys, d_vals = H.dev(keys), H.dev(vals)
            idx.add_batch(d_keys, d_vals, n)
            o_runs.insert(0, oracle.flush(keys, vals))
            o_levels.insert(0, 1)
            oracle_compact(o_runs, o_levels, M, T, K)
            for k, v in zip(keys, vals):
                newest[tuple(int(x) for x in k)] = (int(v["file_id"]), int(v["offset"]))
            # shape and contents: the device index is the oracle's, run by run
            assert idx.levels == o_levels and idx.entries == [len(k) for k, _ in o_runs]
            for r, (ok, ov) in zip(idx._runs, o_runs):
                torch.cuda.synchronize()
                assert np.array_equal(H.host(r["keys"], np.uint64, 32 * r["n"]).reshape(-1, 4), ok)
                assert np.array_equal(H.host(r["vals"], VAL_DTYPE, 16 * r["n"]), ov)
            for i in set(idx.levels):                        # the policy's limits hold
                assert idx.levels.count(i) <= K
                assert sum(e for lv, e in zip(idx.levels, idx.entries) if lv == i) < M * T ** i
        assert idx.merges > 0 and sum(idx.entries) >= len(newest)      # runs may still share keys
        # newest record wins, as in a dict
        for k, want in list(newest.items())[::17]:
            got = oracle.lookup(o_runs, np.array(k, dtype=np.uint64))
            assert got is not None
            assert (int(got[0]["file_id"]), int(got[0]["offset"])) == want
        # probes through the index (hash indexes attached) equal the oracle's
        qoff = synth.offsets(synth.chunk_counts(w.query.seq_off, 16))
        total = int(qoff[-1])
        o_hit, o_recs, _, _ = oracle.probe_batch(og, w.query.tokens, w.query.seq_off, qoff, o_runs)
        d_hit = torch.zeros(w.query.n, dtype=torch.int32, device=H.DEV)
        d_recs = torch.full((max(1, total) * 16,), 0xAB, dtype=torch.uint8, device=H.DEV)
        ctx.probe_batch(w.query.n, H.dev(w.query.tokens), H.dev(w.query.seq_off), H.dev(qoff),
                        total, idx.runs(), d_hit, d_recs, None)
        torch.cuda.synchronize()
        assert np.array_equal(d_hit.cpu().numpy().view(np.uint32), o_hit)
        assert np.array_equal(H.host(d_recs, VAL_DTYPE, total * 16), o_recs)
        assert ctx.last_status()["flags"] == 0


def test_policy_change_is_lazy():
    g = G
    rng = np.random.default_rng(3)
    with lsmkv.Context(g, 0) as ctx:
        idx = LsmIndex(ctx, alloc, 50, 4, 3, hash_index=False)
        for b in range(7):
            keys = np.zeros((50, 4), np.uint64)
            keys[:, 0] = rng.integers(0, 100, 50)
            keys[:, 1] = rng.integers(0, 2**61 - 1, 50, dtype=np.uint64)
            vals = np.zeros(50, VAL_DTYPE)
            idx.add_batch(H.dev(keys), H.dev(vals), 50)
        assert idx.levels == [1, 1, 1, 2]
        idx.set_policy(4, 1)
        assert idx.levels == [1, 1, 1, 2]                    # nothing moves by itself
        assert idx.compact() >= 1 and idx.levels == [1, 2]
