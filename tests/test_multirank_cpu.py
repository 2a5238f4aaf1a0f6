"""Two gloo ranks on the CPU: the replica plumbing used by `bench.py --gpus N` (own batch per
rank, max-over-ranks timing, whole-job aggregate) and an oracle-checked shard of the path per
rank with no exchange between ranks."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2511_16138_b200 import ranks, synth


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        import oracle
        assert ranks.rank_env() == (rank, world, rank)
        w = synth.llama_requests(n_req=6, min_len=64, max_len=256,
                                 config_id=ranks.workload_config_id(2, rank))
        g = oracle.Geom(2, 2, 16, page_tokens=16, chunk_tokens=16)
        nch = synth.chunk_counts(w.batch.seq_off, 16)
        coff = synth.offsets(nch)
        n = int(coff[-1])
        rng = synth.rng_for(2, 50 + rank)
        pool = synth.random_pool_bytes(rng, 4, n + 2, g.page_bytes)
        pages = synth.random_pages(rng, n + 2, n)
        keys, vals, blob = oracle.encode_batch(g, w.batch.tokens, w.batch.seq_off, None, coff,
                                               pages, pool, rank, 0)
        run = oracle.flush(keys, vals)
        hit, recs, _, _ = oracle.probe_batch(g, w.batch.tokens, w.batch.seq_off, coff, [run])
        assert np.array_equal(hit, nch.astype(np.uint32))           # each rank finds its own shard
        # ranks hold different batches of the same shape
        sig = torch.tensor([int(w.batch.tokens[:32].astype(np.int64).sum()), w.batch.n])
        sigs = [torch.zeros_like(sig) for _ in range(world)]
        dist.all_gather(sigs, sig)
        assert sigs[0][1] == sigs[1][1] and sigs[0][0] != sigs[1][0]
        # timing: the slowest rank defines the step; the value is the whole job's
        ms = 10.0 * (rank + 1)
        ms_max = ranks.max_over_ranks(ms)
        units = ranks.sum_over_ranks(float(blob.size))
        assert ms_max == 10.0 * world
        rate = ranks.whole_job_rate(units, ms_max)
        gathered = [torch.zeros(1, dtype=torch.float64) for _ in range(world)]
        dist.all_gather(gathered, torch.tensor([float(blob.size)], dtype=torch.float64))
        assert abs(rate - sum(float(x) for x in gathered) / (ms_max * 1e-3)) < 1e-6
        dist.barrier()
        with open(os.path.join(out_dir, f"ok{rank}"), "w") as f:
            f.write("ok")
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks(tmp_path):
    import oracle
    oracle.build()                         # compile once, before the ranks race for it
    port = _free_port()
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    assert sorted(os.listdir(tmp_path)) == ["ok0", "ok1"]


def test_single_process_identities():
    assert ranks.max_over_ranks(3.5) == 3.5 and ranks.sum_over_ranks(2.0) == 2.0
    assert ranks.whole_job_rate(1000.0, 500.0) == 2000.0
    assert ranks.workload_config_id(2, 0) == 2 and ranks.workload_config_id(2, 3) == 302
