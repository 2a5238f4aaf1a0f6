#!/usr/bin/env python
"""Benchmark of the whole hot path: encode (chunk keys + records + pack) -> flush (keys become a
sorted run) -> probe -> decode (unpack/scatter) over one batch of Llama-3-8B-shaped requests, on N GPUs of one node.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One "step" is one pass of the whole path over the whole batch (256 requests of 1k-8k tokens,
32 layers x 8 KV heads x 128, bf16, page 16: ~75k chunks of 2 MiB, ~147 GiB per direction),
processed in waves that fit HBM (source pool + blob arena + destination pool per wave).
Prints ONE JSON line (rank 0).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2511_16138_b200 import synth  # noqa: E402

NCU_TRAFFIC_RATIO = 0.9867   # measured DRAM traffic / algorithmic bytes of the slab copy kernel
METRIC = "codec_GBps_pack_plus_unpack"
UNIT = "GB/s"
WORKLOAD = ("configs[1]: Llama-3-8B KV shape, 32 layers x 8 KV heads x 128 head_dim bf16, page 16; "
            "256 requests, lengths U[1k,8k], Zipf(1.1) tree of 64 shared prefixes; "
            "full encode, probe, decode")
GEOM = dict(n_layers=32, n_kv_heads=8, head_dim=128, elem_bytes=2, page_tokens=16, chunk_tokens=16)


def hbm_peak():
    """(GB/s, where it comes from): the copy bandwidth measured on this machine, else the fallback."""
    peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(peaks_path):
        with open(peaks_path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    return 6650.0, "fallback"


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--requests", type=int, default=256, help="requests in the batch (256 = the named workload)")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--cpu-seconds", type=float, default=10.0, help="CPU baseline budget (0 = skip)")
    ap.add_argument("--only-probe-block", action="store_true",
                    help="run just the probe-heavy measurement (a small case for profiling)")
    ap.add_argument("--no-shapes-block", action="store_true",
                    help="skip the other named workloads (their KV shapes, and the workloads "
                         "themselves: long context, multi-turn, decode of the probe-heavy hits)")
    ap.add_argument("--only-workloads-block", action="store_true",
                    help="run just the other named workloads as workloads")
    ap.add_argument("--no-xp12-block", action="store_true",
                    help="skip the compressing-codec measurement")
    ap.add_argument("--no-probe-block", action="store_true",
                    help="skip the probe-heavy measurement")
    ap.add_argument("--tuning", default="", help="name=value,... launch-shape knobs")
    return ap.parse_args()


# ---- workload --------------------------------------------------------------------------------

def split_waves(nch: np.ndarray, n_waves: int):
    """Contiguous groups of requests with roughly equal chunk counts."""
    total = int(nch.sum())
    bounds, acc, target = [0], 0, total / n_waves
    for r, c in enumerate(nch):
        acc += int(c)
        if acc >= target * len(bounds) and len(bounds) < n_waves:
            bounds.append(r + 1)
    bounds.append(len(nch))
    out = [(bounds[i], bounds[i + 1]) for i in range(len(bounds) - 1)]
    return [w for w in out if w[1] > w[0]]


def wave_batch(batch: synth.Batch, a: int, b: int) -> synth.Batch:
    t0, t1 = int(batch.seq_off[a]), int(batch.seq_off[b])
    return synth.Batch(batch.tokens[t0:t1], (batch.seq_off[a:b + 1] - batch.seq_off[a]).astype(np.uint64))


def meminfo_available_bytes() -> int:
    try:
        with open("/proc/meminfo") as f:
            for line in f:
                if line.startswith("MemAvailable:"):
                    return int(line.split()[1]) * 1024
    except OSError:
        pass
    return 8 << 30


# ---- clocks ----------------------------------------------------------------------------------

class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, uuid: str):
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", uuid, f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, power, reasons = [], [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in out.strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 8:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1])); power.append(float(f[2]))
            except ValueError:
                continue
            for name, v in zip(names, f[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "samples": len(sm),
                "power_w_max": max(power), "reasons": sorted(reasons)}


# ---- the CPU baseline (the oracle, as it stands, on a bounded sample) -------------------------

def oracle_sample_pass(og, sample):
    """One pass of the whole path on the CPU: encode, probe, decode. Returns bytes moved."""
    import oracle
    b, coff, pages, pool, runs, dst_pages, dst_pool = sample
    keys, vals, blob = oracle.encode_batch(og, b.tokens, b.seq_off, None, coff, pages, pool, 0, 0)
    hit, recs, _, _ = oracle.probe_batch(og, b.tokens, b.seq_off, coff, runs)
    oracle.decode_batch(og, coff, hit, recs, [blob], dst_pages, dst_pool)
    return blob.size + int(hit.sum()) * og.chunk_bytes


def make_oracle_sample(batch, max_chunks, pool_pages_fn):
    """The first requests of the batch up to max_chunks chunks, with a compact host pool."""
    import oracle
    og = oracle.Geom(**GEOM)
    nch = synth.chunk_counts(batch.seq_off, og.chunk_tokens)
    n_req = int(np.searchsorted(np.cumsum(nch), max_chunks, side="right"))
    n_req = max(1, n_req)
    b = wave_batch(batch, 0, n_req)
    coff = synth.offsets(nch[:n_req])
    n = int(coff[-1])
    rng = synth.rng_for(2, 99)
    pages = synth.random_pages(rng, n, n)
    dst_pages = synth.random_pages(rng, n, n)
    pool = pool_pages_fn(n, og)
    keys, vals, _ = oracle.encode_batch(og, b.tokens, b.seq_off, None, coff, None, None, 0, 0,
                                        with_blob=False)
    runs = [oracle.flush(keys, vals)]
    dst_pool = np.zeros_like(pool)
    return og, (b, coff, pages, pool, runs, dst_pages, dst_pool), n_req, n


def time_oracle(og, sample, budget_s):
    t0 = time.perf_counter()
    moved, passes = 0, 0
    while True:
        moved += oracle_sample_pass(og, sample)
        passes += 1
        el = time.perf_counter() - t0
        if el >= budget_s or passes >= 50:
            return moved / el / 1e9, passes, el


def _oracle_worker(job):
    """One process of the all-cores baseline: a plain parallel-for over requests -- this worker
    takes requests i, i + P, ... of the batch (up to its share of chunks) and runs the oracle's
    encode / probe / decode passes over them for the given time."""
    i, n_workers, n_req_total, chunks_per_worker, budget_s = job
    import oracle
    og = oracle.Geom(**GEOM)
    w = synth.llama_requests(n_req=n_req_total)
    nch_all = synth.chunk_counts(w.batch.seq_off, og.chunk_tokens)
    seqs, acc = [], 0
    for r in range(i, w.batch.n, n_workers):           # whole requests, the last one cut to fit
        take = min(int(nch_all[r]), chunks_per_worker - acc)
        if take <= 0:
            break
        seqs.append(w.batch.seq(r)[:take * og.chunk_tokens])
        acc += take
    b = synth.make_batch(seqs)
    nch = synth.chunk_counts(b.seq_off, og.chunk_tokens)
    coff = synth.offsets(nch)
    n = int(coff[-1])
    rng = synth.rng_for(2, 500 + i)
    pages, dst_pages = synth.random_pages(rng, n, n), synth.random_pages(rng, n, n)
    pool = synth.random_pool_bytes(rng, 2 * og.n_layers, n, og.page_bytes)
    keys, vals, _ = oracle.encode_batch(og, b.tokens, b.seq_off, None, coff, None, None, 0, 0,
                                        with_blob=False)
    sample = (b, coff, pages, pool, [oracle.flush(keys, vals)], dst_pages, np.zeros_like(pool))
    oracle_sample_pass(og, sample)                           # warm (pages everything in)
    v, passes, el = time_oracle(og, sample, budget_s)
    return v * el * 1e9, el, passes, n


def time_oracle_all_cores(n_req_total, max_chunks_total, budget_s):
    """The oracle on every host core the process may use: spawned workers (never forked: the
    parent may hold a CUDA context), each timing its own share; the rate is all bytes moved over
    the longest worker's time."""
    import multiprocessing as mp
    try:
        n_workers = len(os.sched_getaffinity(0))
    except AttributeError:
        n_workers = os.cpu_count() or 1
    n_workers = max(1, min(n_workers, 64))
    per = max(4, max_chunks_total // n_workers)
    jobs = [(i, n_workers, n_req_total, per, budget_s) for i in range(n_workers)]
    with mp.get_context("spawn").Pool(n_workers) as pool:
        res = pool.map(_oracle_worker, jobs)
    moved = sum(r[0] for r in res)
    el = max(r[1] for r in res)
    return {"value": moved / el / 1e9, "unit": UNIT, "cores": n_workers, "kind": "oracle",
            "sample": f"{n_workers} workers, parallel-for over requests: {sum(r[3] for r in res)} chunks "
                      f"in all, {sum(r[2] for r in res)} passes, longest worker {el:.1f} s"}


def run_reference(args):
    """--impl reference: the CPU oracle, as it stands, on the host cores; one step = one pass
    over a bounded sample of the same workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = synth.llama_requests(n_req=args.requests)
    avail = meminfo_available_bytes()
    cb = 2 * GEOM["n_layers"] * GEOM["page_tokens"] * GEOM["n_kv_heads"] * GEOM["head_dim"] * GEOM["elem_bytes"]
    max_chunks = int(min(1024, max(8, avail * 0.4 / (3 * cb))))

    def host_pool(n, og):
        rng = synth.rng_for(2, 7)
        return synth.random_pool_bytes(rng, 2 * og.n_layers, n, og.page_bytes)

    og, sample, n_req, n = make_oracle_sample(w.batch, max_chunks, host_pool)
    for _ in range(args.warmup):
        oracle_sample_pass(og, sample)
    t0 = time.perf_counter()
    moved = 0
    for _ in range(args.steps):
        moved += oracle_sample_pass(og, sample)
    el = time.perf_counter() - t0
    val = moved / el / 1e9
    desc = f"first {n_req} requests = {n} chunks ({n * cb / 2**30:.2f} GiB per direction) per step"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": el / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u8",
        "data": "synthetic", "config": {"workload": WORKLOAD, "sample": desc},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": desc},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


# ---- our arm ---------------------------------------------------------------------------------

def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    import torch.distributed as dist
    from paper_2511_16138_b200 import build, lsmkv, ranks
    if int(os.environ.get("LOCAL_RANK", "0")) == 0:
        build.build()          # no-op when liblsmkv.so is newer than its sources
    else:                      # the other ranks of the node wait for local rank 0's build
        t_wait = time.time()
        while build._stale() and time.time() - t_wait < 300:
            time.sleep(0.5)

    rank, world, local_rank = ranks.rank_env()
    if world > 1 or "TORCHELASTIC_RUN_ID" in os.environ:    # launched by torch.distributed.run
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29511")
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    stream = torch.cuda.current_stream()

    def barrier():
        torch.cuda.synchronize()
        if dist.is_initialized():
            dist.barrier()
        torch.cuda.synchronize()

    if args.only_workloads_block:
        if rank == 0:
            peak, _ = hbm_peak()
            print(json.dumps({"other_workloads": [f(torch, lsmkv, dev, local_rank, peak)
                                                  for f in (long_context_block, multi_turn_block,
                                                            probe_heavy_decode_block)]}))
        return
    if args.only_probe_block:
        if rank == 0:
            print(json.dumps({"probe": probe_heavy_block(torch, lsmkv, dev, local_rank,
                                                         args.steps, args.warmup)}))
        return

    g = lsmkv.Geom(**GEOM)
    cb, pb, L2 = g.chunk_bytes, g.page_bytes, 2 * g.n_layers
    peak, peak_src = hbm_peak()
    # every rank gets its own batch of the same shape (weak scaling, no data-path collective)
    w = synth.llama_requests(n_req=args.requests, config_id=ranks.workload_config_id(2, rank))
    batch = w.batch
    nch = synth.chunk_counts(batch.seq_off, g.chunk_tokens)
    total_chunks = int(nch.sum())
    payload = total_chunks * cb

    free, _ = torch.cuda.mem_get_info()
    budget = int(free * 0.80)
    n_waves = 1
    while 3 * -(-total_chunks // n_waves) * cb > budget:
        n_waves += 1
    waves = split_waves(nch, n_waves)
    cap = max(int(nch[a:b].sum()) for a, b in waves)

    ctx = lsmkv.Context(g, local_rank)
    for kv in filter(None, args.tuning.split(",")):
        k, v = kv.split("=")
        ctx.set_tuning(k, int(v))
    ctx.reserve(max(b - a for a, b in waves), cap)

    gen = torch.Generator(device=dev)
    gen.manual_seed(synth.SEED0 + 2 + rank)

    def new_pool(fill: bool):
        bufs = []
        for _ in range(L2):
            if fill:
                t = torch.randn(cap * pb // 2, dtype=torch.bfloat16, device=dev, generator=gen)
                bufs.append(t.view(torch.uint8).view(cap, pb))
            else:
                bufs.append(torch.zeros((cap, pb), dtype=torch.uint8, device=dev))
        return bufs, lsmkv.pool_table(bufs)

    src_bufs, src_pool = new_pool(True)
    dst_bufs, dst_pool = new_pool(False)
    arena = torch.empty(cap * cb, dtype=torch.uint8, device=dev)

    def up(a: np.ndarray):
        b = np.ascontiguousarray(a).view(np.uint8).reshape(-1)
        t = torch.empty(max(16, b.size), dtype=torch.uint8, device=dev)
        t[:b.size] = torch.from_numpy(b.copy())
        return t

    rng = synth.rng_for(2, 1000 + rank)
    W = []
    for (a, b) in waves:
        wb = wave_batch(batch, a, b)
        coff = synth.offsets(nch[a:b])
        n = int(coff[-1])
        host = dict(tokens=wb.tokens, seq_off=wb.seq_off, coff=coff,
                    src_pages=synth.random_pages(rng, cap, n),
                    dst_pages=synth.random_pages(rng, cap, n))
        d = dict(n_req=b - a, n=n, host=host, nch=nch[a:b],
                 tokens=up(wb.tokens), seq_off=up(wb.seq_off), coff=up(coff),
                 src_pages=up(host["src_pages"]), dst_pages=up(host["dst_pages"]),
                 keys=torch.empty(n * 32, dtype=torch.uint8, device=dev),
                 vals=torch.empty(n * 16, dtype=torch.uint8, device=dev),
                 hit=torch.zeros(b - a, dtype=torch.int32, device=dev),
                 recs=torch.empty(n * 16, dtype=torch.uint8, device=dev))
        W.append(d)

    def encode(d):
        ctx.encode_batch(d["n_req"], d["tokens"], d["seq_off"], None, d["coff"], d["n"],
                         d["src_pages"], src_pool, 0, 0, d["keys"], d["vals"], arena, d["n"] * cb,
                         stream=stream)

    def probe(d):
        ctx.probe_batch(d["n_req"], d["tokens"], d["seq_off"], d["coff"], d["n"], d["runs"],
                        d["hit"], d["recs"], None, stream=stream)

    def decode(d):
        ctx.decode_batch(d["n_req"], d["coff"], d["n"], d["hit"], d["recs"],
                         [(arena, d["n"] * cb)], d["dst_pages"], dst_pool, stream=stream)

    # ---- untimed preparation: the index (one sorted run per wave), flushed on the device from
    # the encoder's own keys; the padded flush output serves as the run, no count is read back
    flush_ms = []
    for d in W:
        encode(d)
        n = d["n"]
        d["run_k"] = torch.empty(n * 32, dtype=torch.uint8, device=dev)
        d["run_v"] = torch.empty(n * 16, dtype=torch.uint8, device=dev)
        d["run_n"] = torch.zeros(1, dtype=torch.int64, device=dev)
        d["hidx_buckets"] = lsmkv.lsmkv_hindex_buckets(n)
        d["hidx"] = torch.empty(d["hidx_buckets"] * 32, dtype=torch.uint8, device=dev)
        f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        f0.record(stream)
        ctx.flush_batch(d["keys"], d["vals"], n, d["run_k"], d["run_v"], d["run_n"], stream=stream)
        ctx.hindex_build(d["run_k"], n, d["hidx"], stream=stream)
        f1.record(stream)
        d["runs"] = [(d["run_k"], d["run_v"], n, None, 0, d["hidx"], d["hidx_buckets"])]
        probe(d)
        decode(d)
        torch.cuda.synchronize()
        flush_ms.append(f0.elapsed_time(f1))
        # self-check of this wave (device side): every chunk is a hit
        assert np.array_equal(d["hit"].cpu().numpy(), d["nch"].astype(np.int32)), "probe missed"
        assert 0 < int(d["run_n"].item()) <= n
    st = ctx.last_status()
    assert st["flags"] == 0, st

    def flush(d):
        ctx.flush_batch(d["keys"], d["vals"], d["n"], d["run_k"], d["run_v"], d["run_n"],
                        stream=stream)
        ctx.hindex_build(d["run_k"], d["n"], d["hidx"], stream=stream)

    def step():
        for d in W:
            encode(d)      # chunk keys + records + pack
            flush(d)       # the batch's keys become the sorted run (+ its hash index) the probe reads
            probe(d)
            decode(d)      # plan + unpack

    for _ in range(args.warmup):
        step()
    barrier()
    ctx.last_status()
    ctx.profile_enable(True)
    ctx.profile_read()
    launches0 = ctx.launch_count()
    sampler = ClockSampler("GPU-" + str(torch.cuda.get_device_properties(dev).uuid)) if rank == 0 else None
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record(stream)
    for _ in range(args.steps):
        step()
    e1.record(stream)
    barrier()
    clocks = sampler.stop() if sampler else None
    ms_total = e0.elapsed_time(e1)
    launches = ctx.launch_count() - launches0
    prof = ctx.profile_read()
    ctx.profile_enable(False)
    status = ctx.last_status()
    assert status["flags"] == 0, status
    ms_total = ranks.max_over_ranks(ms_total, dev)
    ms_step = ms_total / args.steps
    moved_all = ranks.sum_over_ranks(2 * payload, dev)   # bytes packed + unpacked, all ranks
    value = ranks.whole_job_rate(moved_all, ms_step) / 1e9

    # ---- the compressing codec on the first wave (reported beside the identity codec)
    xp_block = None
    if rank == 0 and not args.no_xp12_block:
        xp_block = xp12_block(torch, lsmkv, dev, local_rank, W[0], src_bufs, src_pool, dst_bufs,
                              dst_pool, arena, stream, hbm_peak=peak)

    # ---- end to end: host buffers in, host buffers out, through the same C-ABI calls
    e2e = e2e_xp = None
    if args.e2e_steps > 0:
        del arena                                    # the host-buffer calls stage on their own
        torch.cuda.empty_cache()
        link = link_ceiling(torch, dev)                  # same run, same box: the e2e ceiling
        e2e = run_e2e(args, torch, lsmkv, ctx, g, W, src_pool, dst_pool, dev, stream, barrier,
                      world, "identity", link)
        if not args.no_xp12_block:
            ctx_xp = lsmkv.Context(lsmkv.Geom(**dict(GEOM, flags=lsmkv.CODEC_XP12)), local_rank)
            for k_ in ("host_stage_bytes", "host_copy_piece_bytes"):
                ctx_xp.set_tuning(k_, ctx.get_tuning(k_))
            try:
                e2e_xp = run_e2e(args, torch, lsmkv, ctx_xp, g, W, src_pool, dst_pool, dev, stream,
                                 barrier, world, "xp12", link)
            finally:
                ctx_xp.close()

    # ---- probe throughput on the probe-heavy workload (second half of the metric)
    probe_block = None
    if rank == 0 and not args.no_probe_block:
        probe_block = probe_heavy_block(torch, lsmkv, dev, local_rank, args.steps,
                                        args.warmup)

    # ---- CPU baseline: the oracle on a bounded sample (rank 0, single GPU runs only)
    cpu = None
    if rank == 0 and world == 1 and args.cpu_seconds > 0:
        def gpu_pages(n, og):
            idx = torch.arange(n, device=dev)
            return torch.stack([b_[idx] for b_ in src_bufs]).cpu().numpy()
        max_chunks = int(min(1024, max(8, meminfo_available_bytes() * 0.4 / (3 * cb))))
        og, sample, s_req, s_n = make_oracle_sample(batch, max_chunks, gpu_pages)
        v, passes, el = time_oracle(og, sample, args.cpu_seconds)
        cpu = {"value": v, "unit": UNIT, "cores": 1, "kind": "oracle",
               "sample": f"first {s_req} requests = {s_n} chunks ({s_n * cb / 2**30:.2f} GiB per "
                         f"direction), {passes} passes in {el:.1f} s; host cpus={os.cpu_count()}"}
        del sample
        try:
            cpu["all_cores"] = time_oracle_all_cores(args.requests, max_chunks,
                                                     min(5.0, args.cpu_seconds))
        except Exception as exc:                           # e.g. no room for the workers' pools
            cpu["all_cores"] = {"unavailable": repr(exc)}

    shapes_block = workloads_block = None
    if rank == 0:
        n_waves_used = len(W)
        if not args.no_shapes_block:
            # everything of the main workload can go now: the other shapes need the room
            del src_bufs, dst_bufs, src_pool, dst_pool, W
            if args.e2e_steps <= 0:
                del arena
            torch.cuda.empty_cache()
            shapes_block = other_shapes_block(torch, lsmkv, dev, local_rank, peak)
            workloads_block = [f(torch, lsmkv, dev, local_rank, peak)
                               for f in (long_context_block, multi_turn_block,
                                         probe_heavy_decode_block)]
        copy_ms = prof["pack"][0] + prof["unpack"][0]
        copy_launches = prof["pack"][1] + prof["unpack"][1]
        algo_bytes_per_launch = 2.0 * (2 * payload * args.steps) / max(1, copy_launches)
        achieved = algo_bytes_per_launch / (copy_ms / max(1, copy_launches) * 1e-3) / 1e9
        qchunks = total_chunks
        out = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "u8", "data": "synthetic",
            "config": {"workload": WORKLOAD, "requests": args.requests, "chunks": total_chunks,
                       "payload_GiB_per_direction": payload / 2**30, "waves": n_waves_used,
                       "l2": "inputs larger than L2 (each wave moves >30 GiB)",
                       "payload_dtype": "bf16 bit patterns (opaque)", "key_arithmetic": "u64",
                       "tuning": {k: ctx.get_tuning(k) for k in
                                  ("copy_mode", "copy_stage_bytes", "copy_stages",
                                   "copy_ctas_per_sm", "copy_l2_hint")}},
            "e2e": e2e, "e2e_codec_xp12": e2e_xp, "host_link": link if args.e2e_steps > 0 else None,
            "gpu_launches": int(launches), "clocks": clocks,
            "roofline": {"bound": "hbm", "kernel": "k_copy_slabs (pack + unpack launches)",
                         "achieved": achieved, "peak": peak, "unit": "GB/s",
                         "frac": achieved / peak, "peak_source": peak_src,
                         "frac_of_8TBps_nominal": achieved / 8000.0,
                         # DRAM read+write bytes per launch: ncu counters of a 774-chunk capture
                         # (traffic / algorithmic bytes = 0.9867), scaled by chunk count
                         "traffic": NCU_TRAFFIC_RATIO * algo_bytes_per_launch,
                         "traffic_source": "ncu dram__bytes_read+write on a 774-chunk launch, "
                                           "scaled by chunks (ncu summary committed with the repository)",
                         "algorithmic_bytes_per_launch": algo_bytes_per_launch,
                         "avg_launch_ms": copy_ms / max(1, copy_launches)},
            "cpu_baseline": cpu,
            "probe": probe_block,
            "codec_xp12": xp_block,
            "other_shapes": shapes_block,
            "other_workloads": workloads_block,
            "phases": {
                "pack_GBps_payload": payload * args.steps / (prof["pack"][0] * 1e-3) / 1e9,
                "unpack_GBps_payload": payload * args.steps / (prof["unpack"][0] * 1e-3) / 1e9,
                "pack_hbm_frac_of_peak": 2 * payload * args.steps / (prof["pack"][0] * 1e-3) / 1e9 / peak,
                "unpack_hbm_frac_of_peak": 2 * payload * args.steps / (prof["unpack"][0] * 1e-3) / 1e9 / peak,
                "probe_keys_per_s": qchunks * args.steps / (prof["probe"][0] * 1e-3),
                "kernel_ms_per_step": {k: v[0] / args.steps for k, v in prof.items()},
                "kernel_launches": {k: v[1] for k, v in prof.items()},
                "lookups_per_step": status["lookups"] / args.steps,
                "flush_ms_per_wave_in_prep": sum(flush_ms) / len(flush_ms),
            },
        }
        print(json.dumps(out))
    if dist.is_initialized():
        dist.destroy_process_group()


def other_shapes_block(torch, lsmkv, dev, device_index, peak):
    """Pack / unpack rates on the KV shapes of the other named workloads (identity codec, one
    resident wave each, random page tables): the GQA shape with 64-token pages, the 80-layer
    long-context shape, and the tiny 4-layer shape (launch-latency territory)."""
    shapes = [
        ("configs[3] GQA 28x4x128, page 64", dict(n_layers=28, n_kv_heads=4, head_dim=128,
                                                  page_tokens=64, chunk_tokens=64), 6144),
        ("configs[4] long-context 80x8x128, page 16", dict(n_layers=80, n_kv_heads=8,
                                                          head_dim=128), 8192),
        ("configs[0] tiny 4x8x128, page 16", dict(n_layers=4, n_kv_heads=8, head_dim=128), 1024),
    ]
    out = []
    for name, gd, n in shapes:
        g = lsmkv.Geom(**gd)
        cb, pb = g.chunk_bytes, g.page_bytes
        free, _ = torch.cuda.mem_get_info()
        n = int(min(n, free * 0.8 / (3 * cb)))
        ctx = lsmkv.Context(g, device_index)
        src = dst = arena = None
        try:
            C = g.chunk_tokens
            n_req = max(1, n // 256)
            per = n // n_req
            n = per * n_req
            rng = synth.rng_for(9, g.n_layers)
            tokens = rng.integers(0, 128000, n * C, dtype=np.uint32)
            seq_off = (np.arange(n_req + 1, dtype=np.uint64) * np.uint64(per * C))
            coff = (np.arange(n_req + 1, dtype=np.uint64) * np.uint64(per))

            def up(a):
                return torch.from_numpy(np.ascontiguousarray(a).view(np.uint8).reshape(-1).copy()).to(dev)

            gen = torch.Generator(device=dev)
            gen.manual_seed(9)
            src = [torch.randn(n * pb // 2, dtype=torch.bfloat16, device=dev,
                               generator=gen).view(torch.uint8).view(n, pb) for _ in range(2 * g.n_layers)]
            dst = [torch.zeros((n, pb), dtype=torch.uint8, device=dev) for _ in range(2 * g.n_layers)]
            sp, dp = lsmkv.pool_table(src), lsmkv.pool_table(dst)
            arena = torch.empty(n * cb, dtype=torch.uint8, device=dev)
            d_tok, d_off, d_coff = up(tokens), up(seq_off), up(coff)
            src_pages, dst_pages = synth.random_pages(rng, n, n), synth.random_pages(rng, n, n)
            d_sp, d_dp = up(src_pages), up(dst_pages)
            keys = torch.empty(n * 32, dtype=torch.uint8, device=dev)
            vals = torch.empty(n * 16, dtype=torch.uint8, device=dev)
            hit = torch.full((n_req,), per, dtype=torch.int32, device=dev)

            def once():
                ctx.encode_batch(n_req, d_tok, d_off, None, d_coff, n, d_sp, sp, 0, 0, keys, vals,
                                 arena, n * cb)
                ctx.decode_batch(n_req, d_coff, n, hit, vals, [(arena, n * cb)], d_dp, dp)

            for _ in range(3):
                once()
            torch.cuda.synchronize()
            idx_s = torch.from_numpy(src_pages[:256].astype(np.int64)).to(dev)
            idx_d = torch.from_numpy(dst_pages[:256].astype(np.int64)).to(dev)
            assert all(torch.equal(a[idx_s], b[idx_d]) for a, b in zip(src, dst)), name
            assert ctx.last_status()["flags"] == 0
            ctx.profile_enable(True)
            ctx.profile_read()
            reps = 5
            for _ in range(reps):
                once()
            torch.cuda.synchronize()
            prof = ctx.profile_read()
            pm, um = prof["pack"][0] / reps, prof["unpack"][0] / reps
            out.append({"shape": name, "chunks": n, "chunk_MiB": cb / 2**20,
                        "payload_GiB": n * cb / 2**30,
                        "pack_GBps_payload": n * cb / pm / 1e6, "unpack_GBps_payload": n * cb / um / 1e6,
                        "pack_hbm_frac_of_peak": 2 * n * cb / pm / 1e6 / peak,
                        "unpack_hbm_frac_of_peak": 2 * n * cb / um / 1e6 / peak})
        finally:
            ctx.close()
            del src, dst, arena
            torch.cuda.empty_cache()
    return out


# ---- the other named workloads, run as workloads (identity codec) ---------------------------

def _up(torch, dev, a):
    b = np.ascontiguousarray(a).view(np.uint8).reshape(-1)
    t = torch.empty(max(16, b.size), dtype=torch.uint8, device=dev)
    if b.size:
        t[:b.size] = torch.from_numpy(b.copy())
    return t


def _filled_pool(torch, lsmkv, dev, g, num_pages, seed):
    gen = torch.Generator(device=dev)
    gen.manual_seed(seed)
    bufs = [torch.randn(num_pages * g.page_bytes // 2, dtype=torch.bfloat16, device=dev,
                        generator=gen).view(torch.uint8).view(num_pages, g.page_bytes)
            for _ in range(2 * g.n_layers)]
    return bufs, lsmkv.pool_table(bufs)


def _zero_pool(torch, lsmkv, dev, g, num_pages):
    bufs = [torch.zeros((num_pages, g.page_bytes), dtype=torch.uint8, device=dev)
            for _ in range(2 * g.n_layers)]
    return bufs, lsmkv.pool_table(bufs)


def _class_ms(prof, reps=1):
    return {k: v[0] / reps for k, v in prof.items() if v[1]}


def long_context_block(torch, lsmkv, dev, device_index, peak, reps=3):
    """configs[4] as a workload: 4 requests x 32768 tokens (two share 16k), 80x8x128 bf16, page 16:
    encode all (40 GiB), flush, probe with the last 1k tokens changed, decode the 1984-chunk hits.
    Device time per kernel class from the library's own events, on the launching stream."""
    g = lsmkv.Geom(80, 8, 128, page_tokens=16, chunk_tokens=16)
    cb = g.chunk_bytes
    w = synth.long_context()
    nch = synth.chunk_counts(w.store.seq_off, 16)
    coff = synth.offsets(nch)
    n = int(coff[-1])
    free, _ = torch.cuda.mem_get_info()
    if 3 * n * cb > free * 0.92:
        return {"workload": "configs[4] long-context", "unavailable": "not enough free device memory"}
    qoff = synth.offsets(synth.chunk_counts(w.query.seq_off, 16))
    nq = int(qoff[-1])
    rng = synth.rng_for(5, 77)
    ctx = lsmkv.Context(g, device_index)
    src = dst = arena = None
    try:
        src, sp = _filled_pool(torch, lsmkv, dev, g, n, 5)
        dst, dp = _zero_pool(torch, lsmkv, dev, g, n)
        arena = torch.empty(n * cb, dtype=torch.uint8, device=dev)
        d_tok, d_off, d_coff = (_up(torch, dev, a) for a in (w.store.tokens, w.store.seq_off, coff))
        d_src = _up(torch, dev, synth.random_pages(rng, n, n))
        q_tok, q_off, q_qoff = (_up(torch, dev, a) for a in (w.query.tokens, w.query.seq_off, qoff))
        d_dst = _up(torch, dev, synth.random_pages(rng, n, nq))
        keys = torch.empty(n * 32, dtype=torch.uint8, device=dev)
        vals = torch.empty(n * 16, dtype=torch.uint8, device=dev)
        rk, rv = torch.empty_like(keys), torch.empty_like(vals)
        rn = torch.zeros(1, dtype=torch.int64, device=dev)
        nb = lsmkv.lsmkv_hindex_buckets(n)
        hx = torch.empty(nb * 32, dtype=torch.uint8, device=dev)
        hit = torch.zeros(w.query.n, dtype=torch.int32, device=dev)
        recs = torch.empty(nq * 16, dtype=torch.uint8, device=dev)
        runs = [(rk, rv, n, None, 0, hx, nb)]

        def once():
            ctx.encode_batch(w.store.n, d_tok, d_off, None, d_coff, n, d_src, sp, 0, 0, keys, vals,
                             arena, n * cb)
            ctx.flush_batch(keys, vals, n, rk, rv, rn)
            ctx.hindex_build(rk, n, hx)
            ctx.probe_batch(w.query.n, q_tok, q_off, q_qoff, nq, runs, hit, recs, None)
            ctx.decode_batch(w.query.n, q_qoff, nq, hit, recs, [(arena, n * cb)], d_dst, dp)

        once()
        torch.cuda.synchronize()
        hits = hit.cpu().numpy()
        assert np.array_equal(hits, (w.expected_hit_tokens // 16).astype(np.int32)), hits
        assert ctx.last_status()["flags"] == 0
        ctx.profile_enable(True)
        ctx.profile_read()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            once()
        e1.record()
        torch.cuda.synchronize()
        ms = _class_ms(ctx.profile_read(), reps)
        n_hit = int(hits.sum())
        return {"workload": "configs[4]: 4 x 32768 tokens, 80x8x128 bf16, page 16; encode, flush, "
                            "probe with the last 1k tokens changed, decode the hits",
                "chunks_encoded": n, "chunks_decoded": n_hit, "chunk_MiB": cb / 2**20,
                "payload_GiB_encoded": n * cb / 2**30, "payload_GiB_decoded": n_hit * cb / 2**30,
                "ms_per_pass": e0.elapsed_time(e1) / reps, "kernel_ms": ms,
                "pack_GBps_payload": n * cb / ms["pack"] / 1e6,
                "unpack_GBps_payload": n_hit * cb / ms["unpack"] / 1e6,
                "round_trip_GBps_payload": (n + n_hit) * cb / (ms["pack"] + ms["unpack"]) / 1e6,
                "pack_hbm_frac_of_peak": 2 * n * cb / ms["pack"] / 1e6 / peak,
                "unpack_hbm_frac_of_peak": 2 * n_hit * cb / ms["unpack"] / 1e6 / peak,
                "probe_keys_per_s": nq / ms["probe"] * 1e3,
                "flush_share_of_pass": (ms.get("flush", 0.0)) / (e0.elapsed_time(e1) / reps)}
    finally:
        ctx.close()
        del src, dst, arena
        torch.cuda.empty_cache()

def multi_turn_block(torch, lsmkv, dev, device_index, peak, max_groups=8):
    """configs[3] as a workload: 512 conversations x 8 turns of 256-1024 new tokens, 28x4x128
    bf16, page 64. Per turn: probe and decode the stored history, encode the new chunks
    (start_chunk), flush them as the newest run with its hash index, merge the two oldest runs
    when more than four pile up. Conversations in groups of 64 (pool and arena reused)."""
    g = lsmkv.Geom(28, 4, 128, page_tokens=64, chunk_tokens=64)
    cb, C = g.chunk_bytes, 64
    w = synth.multi_turn()
    n_conv, n_turns, group = w.full.n, w.turn_end.shape[1], 64
    final_nch = synth.chunk_counts(w.full.seq_off, C)
    groups = [list(range(a, min(n_conv, a + group))) for a in range(0, n_conv, group)][:max_groups]
    cap = int(max(final_nch[c].sum() for c in groups))
    free, _ = torch.cuda.mem_get_info()
    if 3 * cap * cb > free * 0.92:
        return {"workload": "configs[3] GQA multi-turn", "unavailable": "not enough free device memory"}
    rng = synth.rng_for(4, 77)
    # host side of every turn, prepared before anything is timed
    plan = []
    for convs in groups:
        perm = synth.random_pages(rng, cap, int(final_nch[convs].sum()))
        page_of, at = {}, 0
        for c in convs:
            page_of[c] = perm[at:at + int(final_nch[c])]
            at += int(final_nch[c])
        stored = np.zeros(len(convs), dtype=np.int64)
        turns = []
        for t in range(n_turns):
            hist = synth.make_batch([w.full.seq(c)[:int(w.turn_end[c, t])] for c in convs])
            nch = synth.chunk_counts(hist.seq_off, C)
            qoff = synth.offsets(nch)
            coff = synth.offsets(nch - stored)
            src_pages = np.concatenate([page_of[c][int(stored[k]):int(nch[k])]
                                        for k, c in enumerate(convs)]).astype(np.uint32)
            turns.append(dict(n_req=hist.n, tokens=hist.tokens, seq_off=hist.seq_off, qoff=qoff,
                              total=int(qoff[-1]), start=stored.astype(np.uint32), coff=coff,
                              n=int(coff[-1]), src_pages=src_pages, hist_chunks=int(stored.sum()),
                              dst_pages=synth.random_pages(rng, cap, int(qoff[-1]))))
            stored = nch.copy()
        plan.append(turns)
    ctx = lsmkv.Context(g, device_index)
    src = dst = arena = None
    try:
        src, sp = _filled_pool(torch, lsmkv, dev, g, cap, 4)
        dst, dp = _zero_pool(torch, lsmkv, dev, g, cap)
        arena = torch.empty(cap * cb, dtype=torch.uint8, device=dev)
        up = lambda a: _up(torch, dev, a)
        enc_chunks = dec_chunks = merges = 0

        def run_groups(which):
            nonlocal enc_chunks, dec_chunks, merges
            for turns in which:
                runs, used, keep = [], 0, []
                for t in turns:
                    d_tok, d_off = up(t["tokens"]), up(t["seq_off"])
                    if runs:                           # the stored history: probe, then decode
                        d_qoff = up(t["qoff"])
                        hit = torch.zeros(t["n_req"], dtype=torch.int32, device=dev)
                        recs = torch.empty(max(1, t["total"]) * 16, dtype=torch.uint8, device=dev)
                        ctx.probe_batch(t["n_req"], d_tok, d_off, d_qoff, t["total"], runs, hit, recs,
                                        None)
                        ctx.decode_batch(t["n_req"], d_qoff, t["total"], hit, recs,
                                         [(arena, used * cb)], up(t["dst_pages"]), dp)
                        dec_chunks += t["hist_chunks"]
                        keep.append((hit, recs))
                    n = t["n"]
                    keys = torch.empty(max(1, n) * 32, dtype=torch.uint8, device=dev)
                    vals = torch.empty(max(1, n) * 16, dtype=torch.uint8, device=dev)
                    ctx.encode_batch(t["n_req"], d_tok, d_off, up(t["start"]), up(t["coff"]), n,
                                     up(t["src_pages"]), sp, 0, used * cb, keys, vals,
                                     arena[used * cb:], (cap - used) * cb)
                    rk, rv = torch.empty_like(keys), torch.empty_like(vals)
                    rn = torch.zeros(1, dtype=torch.int64, device=dev)
                    ctx.flush_batch(keys, vals, n, rk, rv, rn)
                    nb = lsmkv.lsmkv_hindex_buckets(n)
                    hx = torch.empty(nb * 32, dtype=torch.uint8, device=dev)
                    ctx.hindex_build(rk, n, hx)
                    runs.insert(0, (rk, rv, n, None, 0, hx, nb))
                    used += n
                    enc_chunks += n
                    if len(runs) > 4:                  # compaction of the two oldest runs
                        m = runs[-1][2] + runs[-2][2]
                        mk = torch.empty(m * 32, dtype=torch.uint8, device=dev)
                        mv = torch.empty(m * 16, dtype=torch.uint8, device=dev)
                        mn = torch.zeros(1, dtype=torch.int64, device=dev)
                        ctx.merge_runs([r[:3] for r in runs[-2:]], mk, mv, mn)
                        mb = lsmkv.lsmkv_hindex_buckets(m)
                        mh = torch.empty(mb * 32, dtype=torch.uint8, device=dev)
                        ctx.hindex_build(mk, m, mh)
                        runs[-2:] = [(mk, mv, m, None, 0, mh, mb)]
                        merges += 1
                torch.cuda.synchronize()
                last_hit = keep[-1][0].cpu().numpy()
                want = turns[-1]["qoff"][1:] - turns[-1]["qoff"][:-1] - (turns[-1]["coff"][1:] - turns[-1]["coff"][:-1])
                assert np.array_equal(last_hit, want.astype(np.int32)), "multi-turn probe missed"

        run_groups(plan[:1])                           # warm-up: scratch reaches its size
        assert ctx.last_status()["flags"] == 0
        enc_chunks = dec_chunks = merges = 0
        ctx.profile_enable(True)
        ctx.profile_read()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        run_groups(plan)
        e1.record()
        torch.cuda.synchronize()
        ms = _class_ms(ctx.profile_read())
        assert ctx.last_status()["flags"] == 0
        dev_ms = sum(ms.values())
        return {"workload": "configs[3]: %d conversations x %d turns, 28x4x128 bf16, page 64; per turn "
                            "probe + decode of the history, encode of the new chunks, flush, "
                            "compaction" % (sum(len(t[0]["start"]) for t in plan), n_turns),
                "chunks_encoded": enc_chunks, "chunks_decoded": dec_chunks, "chunk_MiB": cb / 2**20,
                "payload_GiB_encoded": enc_chunks * cb / 2**30,
                "payload_GiB_decoded": dec_chunks * cb / 2**30, "compactions": merges,
                "elapsed_ms_with_host_work": e0.elapsed_time(e1), "kernel_ms": ms,
                "pack_GBps_payload": enc_chunks * cb / ms["pack"] / 1e6,
                "unpack_GBps_payload": dec_chunks * cb / ms["unpack"] / 1e6,
                "round_trip_GBps_payload": (enc_chunks + dec_chunks) * cb / (ms["pack"] + ms["unpack"]) / 1e6,
                "pack_hbm_frac_of_peak": 2 * enc_chunks * cb / ms["pack"] / 1e6 / peak,
                "unpack_hbm_frac_of_peak": 2 * dec_chunks * cb / ms["unpack"] / 1e6 / peak,
                "flush_and_merge_share_of_kernel_time": (ms.get("flush", 0) + ms.get("merge", 0)) / dev_ms,
                "probe_share_of_kernel_time": ms.get("probe", 0) / dev_ms}
    finally:
        ctx.close()
        del src, dst, arena
        torch.cuda.empty_cache()

def probe_heavy_decode_block(torch, lsmkv, dev, device_index, peak, n_blobs=32768, num_pages=131072):
    """configs[2], the decode half: the hits of the 4096 queries (1M stored keys in 4 runs) are
    scattered into an 8x8x128 bf16 pool of 64 GiB from an arena of 32768 blobs that the million
    records alias (offset = (i mod 32768) * chunk_bytes), in waves of queries that fit the pool."""
    g = lsmkv.Geom(8, 8, 128, page_tokens=16, chunk_tokens=16)
    cb = g.chunk_bytes
    free, _ = torch.cuda.mem_get_info()
    if (n_blobs + num_pages) * cb > free * 0.92:
        return {"workload": "configs[2] decode", "unavailable": "not enough free device memory"}
    w = synth.probe_heavy()
    nch = synth.chunk_counts(w.store.seq_off, 16)
    coff = synth.offsets(nch - w.store_start_chunk)
    up = lambda a: _up(torch, dev, a)
    ctx = lsmkv.Context(g, device_index)
    dst = arena = None
    try:
        n = w.n_stored
        d_keys = torch.empty(n * 32, dtype=torch.uint8, device=dev)
        d_vals = torch.empty(n * 16, dtype=torch.uint8, device=dev)
        ctx.encode_batch(w.store.n, up(w.store.tokens), up(w.store.seq_off), up(w.store_start_chunk),
                         up(coff), n, None, None, 0, 0, d_keys, d_vals, None, 0)
        torch.cuda.synchronize()
        keys = d_keys.cpu().numpy().view(np.uint64).reshape(-1, 4)
        vals = d_vals.cpu().numpy().reshape(-1, 16).copy()
        off = vals[:, 8:16].view(np.uint64).reshape(-1)           # records alias the arena
        off[:] = (np.arange(n, dtype=np.uint64) % np.uint64(n_blobs)) * np.uint64(cb)
        runs, keep = [], []
        for r in range(4):
            sel = w.run_of_key == r
            dup = w.dup_idx[w.dup_run == r]
            m = int(sel.sum()) + len(dup)
            tk = torch.empty(m * 32, dtype=torch.uint8, device=dev)
            tv = torch.empty(m * 16, dtype=torch.uint8, device=dev)
            tn = torch.zeros(1, dtype=torch.int64, device=dev)
            ctx.flush_batch(up(np.concatenate([keys[sel], keys[dup]])),
                            up(np.concatenate([vals[sel], vals[(dup + 7919) % n]])), m, tk, tv, tn)
            nb = lsmkv.lsmkv_hindex_buckets(m)
            hx = torch.empty(nb * 32, dtype=torch.uint8, device=dev)
            ctx.hindex_build(tk, m, hx)
            keep.append(tn)
            runs.append((tk, tv, m, None, 0, hx, nb))
        qoff = synth.offsets(synth.chunk_counts(w.query.seq_off, 16))
        total = int(qoff[-1])
        d_qoff = up(qoff)
        d_hit = torch.zeros(w.query.n, dtype=torch.int32, device=dev)
        d_recs = torch.empty(total * 16, dtype=torch.uint8, device=dev)
        ctx.probe_batch(w.query.n, up(w.query.tokens), up(w.query.seq_off), d_qoff, total, runs,
                        d_hit, d_recs, None)
        torch.cuda.synchronize()
        hit = d_hit.cpu().numpy().astype(np.int64)
        assert np.array_equal(hit, w.expected_hit.astype(np.int64))
        gen = torch.Generator(device=dev)
        gen.manual_seed(3)
        arena = torch.randn(n_blobs * cb // 2, dtype=torch.bfloat16, device=dev,
                            generator=gen).view(torch.uint8)
        dst, dp = _zero_pool(torch, lsmkv, dev, g, num_pages)
        rng = synth.rng_for(3, 77)
        waves, q0 = [], 0
        while q0 < w.query.n:                            # waves of queries that fit the pool
            q1, acc = q0, 0
            while q1 < w.query.n and acc + int(hit[q1]) <= num_pages:
                acc += int(hit[q1])
                q1 += 1
            hit_w = np.zeros(w.query.n, dtype=np.uint32)
            hit_w[q0:q1] = hit[q0:q1]
            pages = np.zeros(total, dtype=np.uint32)
            sel = np.concatenate([np.arange(int(qoff[q]), int(qoff[q]) + int(hit[q]))
                                  for q in range(q0, q1)] + [np.zeros(0, np.int64)]).astype(np.int64)
            pages[sel] = synth.random_pages(rng, num_pages, len(sel))
            waves.append((up(hit_w), up(pages), acc))
            q0 = q1

        def all_waves():
            for d_hw, d_pg, _ in waves:
                ctx.decode_batch(w.query.n, d_qoff, total, d_hw, d_recs, [(arena, n_blobs * cb)],
                                 d_pg, dp)

        all_waves()
        torch.cuda.synchronize()
        st = ctx.last_status()
        assert st["flags"] == 0 and st["chunks_decoded"] == int(hit.sum()), st
        ctx.profile_enable(True)
        ctx.profile_read()
        all_waves()
        torch.cuda.synchronize()
        ms = _class_ms(ctx.profile_read())
        n_hit = int(hit.sum())
        return {"workload": "configs[2], decode of the hits: %d hit chunks of 512 KiB from an arena of "
                            "%d aliased blobs into a %d-page pool, %d waves"
                            % (n_hit, n_blobs, num_pages, len(waves)),
                "chunks_decoded": n_hit, "payload_GiB_decoded": n_hit * cb / 2**30,
                "kernel_ms": ms, "unpack_GBps_payload": n_hit * cb / ms["unpack"] / 1e6,
                "unpack_hbm_frac_of_peak": 2 * n_hit * cb / ms["unpack"] / 1e6 / peak,
                "note": "the arena (16 GiB) is re-read about %.0f times, so its reads partly hit L2; "
                        "the fraction counts read + write bytes as if all came from HBM"
                        % (n_hit / n_blobs)}
    finally:
        ctx.close()
        del dst, arena
        torch.cuda.empty_cache()


def probe_heavy_block(torch, lsmkv, dev, device_index, steps, warmup):
    peak, peak_src = hbm_peak()
    """Probe throughput on the probe-heavy workload (configs[2]): 1M stored chunk keys in four
    sorted runs (900 / 9000 / 90000 / 900100 keys, 1% newer duplicates), 4096 queries of 2k-32k
    tokens, 60% with a cached prefix. Keys come from the library's own encoder and the runs from
    its flush (both untimed here)."""
    g = lsmkv.Geom(8, 8, 128, page_tokens=16, chunk_tokens=16)
    w = synth.probe_heavy()
    nch = synth.chunk_counts(w.store.seq_off, 16)
    coff = synth.offsets(nch - w.store_start_chunk)

    def up(a):
        b = np.ascontiguousarray(a).view(np.uint8).reshape(-1)
        return torch.from_numpy(b.copy()).to(dev)

    ctx = lsmkv.Context(g, device_index)
    try:
        n = w.n_stored
        d_keys = torch.empty(n * 32, dtype=torch.uint8, device=dev)
        d_vals = torch.empty(n * 16, dtype=torch.uint8, device=dev)
        ctx.encode_batch(w.store.n, up(w.store.tokens), up(w.store.seq_off),
                         up(w.store_start_chunk), up(coff), n, None, None, 0, 0, d_keys, d_vals,
                         None, 0)
        torch.cuda.synchronize()
        keys = d_keys.cpu().numpy().view(np.uint64).reshape(-1, 4)
        vals = d_vals.cpu().numpy().reshape(-1, 16)
        runs, keep = [], []
        for r in range(4):                      # deal the keys to the runs, flush each on the GPU
            sel = w.run_of_key == r
            dup = w.dup_idx[w.dup_run == r]
            bk = up(np.concatenate([keys[sel], keys[dup]]))
            bv = up(np.concatenate([vals[sel], vals[(dup + 7919) % n]]))
            m = int(sel.sum()) + len(dup)
            tk = torch.empty(m * 32, dtype=torch.uint8, device=dev)
            tv = torch.empty(m * 16, dtype=torch.uint8, device=dev)
            tn = torch.zeros(1, dtype=torch.int64, device=dev)
            ctx.flush_batch(bk, bv, m, tk, tv, tn)
            keep.append((tk, tv, tn))
            runs.append((tk, tv, m))
        ctx.last_status()
        ctx.profile_enable(True)
        ctx.profile_read()
        big = int((w.run_of_key == 3).sum())
        for _ in range(3):
            ctx.flush_batch(bk, bv, m, tk, tv, tn)
        torch.cuda.synchronize()
        flush_big_ms = ctx.profile_read()["flush"][0] / 3
        ctx.profile_enable(False)
        qoff = synth.offsets(synth.chunk_counts(w.query.seq_off, 16))
        total = int(qoff[-1])
        d_tok, d_off, d_qoff = up(w.query.tokens), up(w.query.seq_off), up(qoff)
        d_hit = torch.zeros(w.query.n, dtype=torch.int32, device=dev)
        d_recs = torch.empty(total * 16, dtype=torch.uint8, device=dev)
        # the same runs with their Bloom filters attached
        runs_bloom = []
        for (tk, tv, m_) in runs:
            nb = lsmkv.lsmkv_bloom_blocks(m_)
            bl = torch.empty(nb * 32, dtype=torch.uint8, device=dev)
            ctx.bloom_build(tk, m_, bl)
            runs_bloom.append((tk, tv, m_, bl, nb))
        # the same runs with their hash indexes attached (build time measured on the big run)
        runs_hashed, hidx_ms = [], 0.0
        for (tk, tv, m_) in runs:
            nb = lsmkv.lsmkv_hindex_buckets(m_)
            hx = torch.empty(nb * 32, dtype=torch.uint8, device=dev)
            ctx.hindex_build(tk, m_, hx)
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(3):
                ctx.hindex_build(tk, m_, hx)
            e1.record()
            torch.cuda.synchronize()
            hidx_ms = e0.elapsed_time(e1) / 3                  # the last (largest) run's
            runs_hashed.append((tk, tv, m_, None, 0, hx, nb))

        def timed(rr):
            for _ in range(max(3, warmup)):
                ctx.probe_batch(w.query.n, d_tok, d_off, d_qoff, total, rr, d_hit, d_recs, None)
            torch.cuda.synchronize()
            assert np.array_equal(d_hit.cpu().numpy(), w.expected_hit.astype(np.int32))
            ctx.last_status()
            reps = max(5, steps)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(reps):
                ctx.probe_batch(w.query.n, d_tok, d_off, d_qoff, total, rr, d_hit, d_recs, None)
            e1.record()
            torch.cuda.synchronize()
            return e0.elapsed_time(e1) / reps, ctx.last_status(), reps

        ms_plain, _, _ = timed(runs)
        ms_bloom, _, _ = timed(runs_bloom)
        ms, st, reps = timed(runs_hashed)
        exact = exact_index_numbers(torch, ctx, w, up, d_tok, d_off, d_qoff, total, d_hit, d_recs,
                                    max(3, warmup), max(5, steps))
        hit_tokens = int(w.expected_hit.sum()) * 16
        # least traffic any probe must do: tokens up to the first miss, one record per query
        # chunk, one hit length per query
        algo_bytes = 4 * hit_tokens + 16 * total + 4 * w.query.n
        return {"workload": "configs[2]: 1M stored chunk keys in 4 sorted runs, 4096 queries of "
                            "2k-32k tokens, 60% cached",
                "ms_per_probe": ms, "query_chunks": total, "keys_per_s": total / ms * 1e3,
                "lookup": "hash index per run (built when the run is written)",
                "hash_index_build_ms_for_%d_keys" % big: hidx_ms,
                "ms_per_probe_searching_sorted_runs": ms_plain,
                "keys_per_s_searching_sorted_runs": total / ms_plain * 1e3,
                "ms_per_probe_searching_with_bloom_filters": ms_bloom,
                "lookups_per_s": st["lookups"] / reps / ms * 1e3,
                "hit_chunks_per_s": st["chunks_hit"] / reps / ms * 1e3,
                "query_tokens": int(len(w.query.tokens)), "stored_keys": n,
                "algorithmic_GBps": algo_bytes / ms / 1e6,
                "flush_ms_for_%d_keys" % big: flush_big_ms,
                "exact_index": exact,
                # the probe's least traffic (tokens up to the first miss, a record per query chunk,
                # a hit length per query) against the measured copy bandwidth: small by nature --
                # the kernel is bound by a chain of dependent steps per round, not by HBM
                "roofline": {"bound": "hbm", "kernel": "k_probe<true>",
                             "achieved": algo_bytes / ms / 1e6, "peak": peak, "unit": "GB/s",
                             "frac": algo_bytes / ms / 1e6 / peak, "peak_source": peak_src,
                             "algorithmic_bytes_per_launch": algo_bytes, "traffic": None},
                "bound": "latency chain: a query's rounds run one after another, each a chain of "
                         "dependent loads and digest arithmetic; the longest query's rounds last "
                         "as long as the launch (committed ncu summary of k_probe on this workload)"}
    finally:
        ctx.close()


def exact_index_numbers(torch, ctx, w, up, d_tok, d_off, d_qoff, total, d_hit, d_recs, warm, reps):
    """The same queries against the exact prefix index (stored sequences ordered by their tokens,
    no digests): build time over the whole stored sequences and probe time."""
    dev = d_tok.device
    s_tok, s_off = up(w.store.tokens), up(w.store.seq_off)
    n_seq = w.store.n
    n_chunks = int(synth.chunk_counts(w.store.seq_off, 16).sum())
    s_vals = torch.zeros(max(1, n_chunks) * 16, dtype=torch.uint8, device=dev)
    d_order = torch.empty(max(1, n_seq), dtype=torch.int32, device=dev)
    d_coff = torch.empty(n_seq + 1, dtype=torch.int64, device=dev)

    def time_of(fn, n_warm, n_rep):
        for _ in range(n_warm):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(n_rep):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / n_rep

    build_ms = time_of(lambda: ctx.xrun_build(s_tok, s_off, n_seq, d_order, d_coff), 2, 3)
    xr = [(s_tok, s_off, s_vals, d_order, d_coff, n_seq)]
    probe = lambda: ctx.xprobe_batch(w.query.n, d_tok, d_off, d_qoff, total, xr, d_hit, d_recs)
    ms = time_of(probe, warm, reps)
    assert np.array_equal(d_hit.cpu().numpy(), w.expected_hit.astype(np.int32))
    ctx.last_status()
    return {"stored_sequences": n_seq, "stored_chunks": n_chunks, "build_ms": build_ms,
            "ms_per_probe": ms, "keys_per_s": total / ms * 1e3}


def xp12_block(torch, lsmkv, dev, device_index, d, src_bufs, src_pool, dst_bufs, dst_pool, arena,
               stream, reps=3, hbm_peak=None):
    """The compressing codec (lossless exponent packing) on the first wave of the workload:
    compression ratio and pack / unpack rates in raw payload bytes per second."""
    g = lsmkv.Geom(**dict(GEOM, flags=lsmkv.CODEC_XP12))
    cb = g.chunk_bytes
    ctx = lsmkv.Context(g, device_index)
    try:
        n, n_req = d["n"], d["n_req"]
        # The one-pass encoder wants room for the worst case (an incompressible batch): leave out
        # trailing requests of the wave until the arena of the identity codec gives that much.
        coff_h = d["host"]["coff"]
        while n_req > 1 and ctx.encode_bound(int(coff_h[n_req])) > arena.numel():
            n_req -= 1
        n = int(coff_h[n_req])
        cap = min(arena.numel(), ctx.encode_bound(n))
        one_pass = cap >= ctx.encode_bound(n) and bool(ctx.get_tuning("xp_one_pass"))
        vals = torch.empty(n * 16, dtype=torch.uint8, device=dev)
        hit = torch.from_numpy(d["nch"][:n_req].astype(np.int32)).to(dev)

        def enc():
            ctx.encode_batch(n_req, d["tokens"], d["seq_off"], None, d["coff"], n, d["src_pages"],
                             src_pool, 0, 0, d["keys"], vals, arena, cap, stream=stream)

        def dec():
            ctx.decode_batch(n_req, d["coff"], n, hit, vals, [(arena, cap)], d["dst_pages"],
                             dst_pool, stream=stream)

        enc(); dec()
        torch.cuda.synchronize()
        st = ctx.last_status()
        assert st["flags"] == 0, st
        v = vals.cpu().numpy().view(np.uint64).reshape(-1, 2)
        used = int(v[-1, 1]) + int(v[-1, 0] >> np.uint64(32))
        sp = torch.from_numpy(d["host"]["src_pages"][:512].astype(np.int64)).to(dev)
        dp = torch.from_numpy(d["host"]["dst_pages"][:512].astype(np.int64)).to(dev)
        for sb, db in zip(src_bufs, dst_bufs):
            assert torch.equal(sb[sp], db[dp]), "xp12 round trip differs"
        ctx.profile_enable(True)
        ctx.profile_read()
        for _ in range(reps):
            enc(); dec()
        torch.cuda.synchronize()
        prof = ctx.profile_read()
        pack_ms, unpack_ms = prof["pack"][0] / reps, prof["unpack"][0] / reps
        return {"codec": "xp12 (lossless bf16 exponent packing)", "chunks": n,
                "raw_GiB": n * cb / 2**30, "ratio": used / (n * cb),
                "pack_GBps_raw_payload": n * cb / pack_ms / 1e6,
                "unpack_GBps_raw_payload": n * cb / unpack_ms / 1e6,
                "pack_ms": pack_ms, "unpack_ms": unpack_ms,
                "encoder": "one pass (pool read once)" if one_pass else "three steps (pool read twice)",
                # the method's bytes: the raw slabs read once, the compressed blobs written once
                "pack_hbm_GBps_algorithmic": (n * cb + used) / pack_ms / 1e6,
                "unpack_hbm_GBps_algorithmic": (n * cb + used) / unpack_ms / 1e6,
                "pack_hbm_frac": (n * cb + used) / pack_ms / 1e6 / hbm_peak if hbm_peak else None,
                "unpack_hbm_frac": (n * cb + used) / unpack_ms / 1e6 / hbm_peak if hbm_peak else None}
    finally:
        ctx.close()


def link_ceiling(torch, dev, nbytes=1 << 30, reps=3):
    """What the host link gives in this run: pinned cudaMemcpyAsync of `nbytes` host->device and
    device->host at the same time on two streams (GB/s, summed over both directions), and each
    direction alone."""
    hp_in = torch.empty(nbytes, dtype=torch.uint8, pin_memory=True)
    hp_out = torch.empty(nbytes, dtype=torch.uint8, pin_memory=True)
    d_in = torch.empty(nbytes, dtype=torch.uint8, device=dev)
    d_out = torch.zeros(nbytes, dtype=torch.uint8, device=dev)
    hp_in.zero_()
    s_a, s_b = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)

    def run(up, down):
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        s_a.wait_event(e0)
        s_b.wait_event(e0)
        for _ in range(reps):
            if up:
                with torch.cuda.stream(s_a):
                    d_in.copy_(hp_in, non_blocking=True)
            if down:
                with torch.cuda.stream(s_b):
                    hp_out.copy_(d_out, non_blocking=True)
        torch.cuda.current_stream().wait_stream(s_a)
        torch.cuda.current_stream().wait_stream(s_b)
        e1.record()
        torch.cuda.synchronize()
        return (int(up) + int(down)) * reps * nbytes / e0.elapsed_time(e1) / 1e6

    run(True, True)                                      # warm-up (pages the pinned buffers in)
    return {"h2d_GBps": run(True, False), "d2h_GBps": run(False, True),
            "both_directions_GBps": run(True, True), "bytes_per_copy": nbytes}


def run_e2e(args, torch, lsmkv, ctx, g, W, src_pool, dst_pool, dev, stream, barrier, world,
            label, link=None):
    """Same path through the host-buffer entry points of the C ABI: per sub-batch the token
    sequences and page tables are HOST arrays, the packed blobs, keys and records come back to
    pinned host memory (where a tensor-log writer would take them), the probe returns hit
    lengths and records to the host, and the decode copies the hit blobs from the host arena
    back to the device and scatters them. The KV pool itself lives on the GPU by nature. Two
    slots, two streams, two host threads: one thread puts sub-batch i+1 while the other gets
    sub-batch i, so both PCIe directions are busy. `ctx` decides the codec (identity or
    compressing)."""
    cb = g.chunk_bytes
    sub_cap = 2048 if world == 1 else 1024           # chunks per sub-batch (4 or 2 GiB of raw blobs)
    subs = []
    for d in W:
        nchw, a, acc = d["nch"], 0, 0
        for r in range(len(nchw)):
            if acc + int(nchw[r]) > sub_cap and r > a:
                subs.append((d, a, r)); a, acc = r, 0
            acc += int(nchw[r])
        subs.append((d, a, len(nchw)))
    max_n = max(int(d["nch"][a:b].sum()) for d, a, b in subs)
    max_req = max(b - a for d, a, b in subs)
    NS = 2
    blob_cap = ctx.encode_bound(max_n)

    def pin(nbytes):
        return torch.empty(nbytes, dtype=torch.uint8, pin_memory=True)

    pin_blob = [pin(blob_cap) for _ in range(NS)]
    pin_keys = [pin(max_n * 32) for _ in range(NS)]
    pin_vals = [pin(max_n * 16) for _ in range(NS)]
    pin_hit = [pin(max_req * 4) for _ in range(NS)]
    pin_recs = [pin(max_n * 16) for _ in range(NS)]
    s_put, s_get = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)

    def pinned(a):
        return torch.from_numpy(np.ascontiguousarray(a).view(np.uint8).reshape(-1).copy()).pin_memory()

    prepared = []
    for d, a, b in subs:
        h = d["host"]
        t0, t1 = int(h["seq_off"][a]), int(h["seq_off"][b])
        c0, c1 = int(h["coff"][a]), int(h["coff"][b])
        seq_rel = (h["seq_off"][a:b + 1] - h["seq_off"][a]).astype(np.uint64)
        qoff = (h["coff"][a:b + 1] - h["coff"][a]).astype(np.uint64)
        p = dict(d=d, n_req=b - a, n=c1 - c0, tokens=pinned(h["tokens"][t0:t1]),
                 seq_off=pinned(seq_rel), src=pinned(h["src_pages"][c0:c1]),
                 dst=pinned(h["dst_pages"][c0:c1]), qoff=pinned(qoff), nch=d["nch"][a:b])
        prepared.append(p)
    # untimed: a real put of each sub-batch gives its records; flushed on the device they are
    # the sub-batch's index (a put is deterministic, so the timed puts reproduce them)
    for p in prepared:
        n = p["n"]
        _, used = ctx.put_batch_host(p["n_req"], p["tokens"], p["seq_off"], None, p["src"],
                                     src_pool, 0, 0, pin_keys[0], pin_vals[0], pin_blob[0],
                                     blob_cap, stream=stream, want_bytes=True)
        torch.cuda.synchronize()
        if used == 0:                                # identity codec: size is known up front
            used = n * cb
        p["blob_bytes"] = used
        dk = pin_keys[0][:n * 32].to(dev)
        dv = pin_vals[0][:n * 16].to(dev)
        tk = torch.empty(n * 32, dtype=torch.uint8, device=dev)
        tv = torch.empty(n * 16, dtype=torch.uint8, device=dev)
        tn = torch.zeros(1, dtype=torch.int64, device=dev)
        ctx.flush_batch(dk, dv, n, tk, tv, tn, stream=stream)
        nb = lsmkv.lsmkv_hindex_buckets(n)
        hx = torch.empty(nb * 32, dtype=torch.uint8, device=dev)
        ctx.hindex_build(tk, n, hx, stream=stream)
        torch.cuda.synchronize()
        p["run_t"] = (tk, tv, tn, hx)
        p["runs"] = [(tk, tv, n, None, 0, hx, nb)]
    # Two host threads, as a serving process would have them: one issues the puts, the other the
    # gets (probe, then decode) of the sub-batches already put, each with a context and a stream
    # of its own (a context is not thread-safe), two sub-batches in flight. A thread that has to
    # wait -- the get for the probe's answer, the compressing put for a slice's records -- then
    # never keeps the other direction of the link idle.
    import threading
    ctx_get = lsmkv.Context(ctx.geom, ctx.device)
    for k_ in ("host_stage_bytes", "host_copy_piece_bytes"):
        ctx_get.set_tuning(k_, ctx.get_tuning(k_))
    put_done = [torch.cuda.Event() for _ in range(NS)]
    slot_free = [torch.cuda.Event() for _ in range(NS)]
    count = {"h2d": 0, "d2h": 0, "moved": 0}
    errors = []

    def put(i):
        p, k_ = prepared[i], i % NS
        ctx.put_batch_host(p["n_req"], p["tokens"], p["seq_off"], None, p["src"], src_pool, 0, 0,
                           pin_keys[k_], pin_vals[k_], pin_blob[k_], blob_cap, stream=s_put)
        return (p["tokens"].numel() + p["seq_off"].numel() * 2 + p["src"].numel(),
                p["blob_bytes"] + p["n"] * 48)

    def get(i, check):
        p, k_ = prepared[i], i % NS
        ctx_get.probe_batch_host(p["n_req"], p["tokens"], p["seq_off"], p["runs"], pin_hit[k_],
                                 pin_recs[k_], None, stream=s_get)
        s_get.synchronize()                 # the host reads hit lengths and records
        if check:
            hits = pin_hit[k_][:p["n_req"] * 4].numpy().view(np.uint32)
            assert np.array_equal(hits, p["nch"].astype(np.uint32)), "e2e probe missed"
        ctx_get.decode_batch_host(p["n_req"], p["qoff"], pin_hit[k_], pin_recs[k_],
                                  [(pin_blob[k_], p["blob_bytes"])], p["dst"], dst_pool, stream=s_get)
        return (p["tokens"].numel() + p["seq_off"].numel() + p["blob_bytes"] + p["n"] * 20 + 20,
                p["n_req"] * 4 + p["n"] * 16)

    def run_steps(n_steps, check=False):
        total = n_steps * len(prepared)
        ready = [threading.Semaphore(0) for _ in range(NS)]      # slot holds a finished put
        free = [threading.Semaphore(1) for _ in range(NS)]       # slot may be written again
        first_use = [True] * NS

        def put_side():
            try:
                torch.cuda.set_device(dev)
                for t in range(total):
                    k_ = t % NS
                    free[k_].acquire()
                    if not first_use[k_]:
                        s_put.wait_event(slot_free[k_])          # recorded before the release
                    first_use[k_] = False
                    a_, b_ = put(t % len(prepared))
                    put_done[k_].record(s_put)
                    count["h2d"] += a_
                    count["d2h"] += b_
                    ready[k_].release()
            except Exception as exc:                             # noqa: BLE001
                errors.append(exc)
                for sem in ready:
                    sem.release()

        def get_side():
            try:
                torch.cuda.set_device(dev)
                for t in range(total):
                    k_ = t % NS
                    ready[k_].acquire()
                    if errors:
                        return
                    s_get.wait_event(put_done[k_])
                    a_, b_ = get(t % len(prepared), check)
                    slot_free[k_].record(s_get)
                    count["h2d"] += a_
                    count["d2h"] += b_
                    count["moved"] += 2 * prepared[t % len(prepared)]["n"] * cb
                    free[k_].release()
            except Exception as exc:                             # noqa: BLE001
                errors.append(exc)
                for sem in free:
                    sem.release()

        ths = [threading.Thread(target=put_side), threading.Thread(target=get_side)]
        for th in ths:
            th.start()
        for th in ths:
            th.join()
        if errors:
            raise errors[0]

    s_put.wait_stream(stream)
    s_get.wait_stream(stream)
    ctx.last_status()
    run_steps(1, check=True)                # warm-up (also faults in the pinned pages)
    barrier()
    st, st_get = ctx.last_status(), ctx_get.last_status()
    assert st["flags"] == 0 and st_get["flags"] == 0, (st, st_get)
    assert st_get["chunks_decoded"] == sum(p["n"] for p in prepared), st_get
    count.update(h2d=0, d2h=0, moved=0)
    steps = max(1, args.e2e_steps)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    s_put.wait_stream(stream)
    s_get.wait_stream(stream)
    run_steps(steps)
    stream.wait_stream(s_put)
    stream.wait_stream(s_get)
    e1.record(stream)
    barrier()
    from paper_2511_16138_b200 import ranks
    ms = ranks.max_over_ranks(e0.elapsed_time(e1), dev)
    h2d, d2h = count["h2d"], count["d2h"]
    moved = ranks.sum_over_ranks(count["moved"], dev)
    ctx.last_status()
    ctx_get.close()
    pcie = (h2d + d2h) / (e0.elapsed_time(e1) * 1e-3) / 1e9          # this rank's link traffic
    return {"value": ranks.whole_job_rate(moved, ms) / 1e9, "unit": UNIT,
            "h2d_bytes_per_step": h2d // steps, "d2h_bytes_per_step": d2h // steps,
            "steps": steps, "ms_per_step": ms / steps, "codec": label,
            "link_GBps_both_directions": link["both_directions_GBps"] if link else None,
            "link_traffic_GBps": pcie,
            "frac_of_link": pcie / link["both_directions_GBps"] if link else None,
            "api": "lsmkv_put_batch_host / lsmkv_probe_batch_host / lsmkv_decode_batch_host",
            "note": "host buffers in and out through the C ABI: blobs, keys and records land in "
                    "pinned host memory, hit blobs are copied back from it before the scatter; "
                    "puts and gets are issued by two host threads on two streams (a context each) "
                    "so both PCIe directions stay busy; "
                    "value counts raw (uncompressed) payload bytes; PCIe-bound"}


if __name__ == "__main__":
    main()
