"""Host-side bookkeeping of one LSM index whose runs live in device memory.

The paper's index is an LSM-tree (Sec. 2.2): a flushed write batch becomes a sorted run at
level 1, levels grow by a size ratio T, a level keeps at most K runs, and compaction merges
runs as levels fill. This class keeps the list of runs, asks the library's planner
(lsmkv_plan_compaction) which merge is due, and carries it out with the library's kernels
(lsmkv_flush_batch, lsmkv_merge_runs, lsmkv_hindex_build). It decides nothing itself and moves
no data on the host; it is scheduling around the device calls, outside any timed path.
"""
from __future__ import annotations

from . import lsmkv


class LsmIndex:
    def __init__(self, ctx: "lsmkv.Context", alloc, buffer_entries: int, size_ratio: int = 4,
                 runs_per_level: int = 1, hash_index: bool = True):
        """alloc(nbytes) -> a device buffer object with data_ptr() (e.g. a torch uint8 tensor);
        buffer_entries = M, the nominal size of a flushed batch."""
        self.ctx, self.alloc = ctx, alloc
        self.M, self.T, self.K = int(buffer_entries), int(size_ratio), int(runs_per_level)
        self.hash_index = hash_index
        self._runs = []          # newest first: dict(keys, vals, n, level, hindex, buckets)
        self.merges = 0
        self.entries_merged = 0

    # -- policy ---------------------------------------------------------------------------
    def set_policy(self, size_ratio: int, runs_per_level: int) -> None:
        """New (T, K). Nothing is reorganised now: the values steer the merges planned from
        here on (the paper's lazy transition, Sec. 3.3)."""
        self.T, self.K = int(size_ratio), int(runs_per_level)

    @property
    def levels(self):
        return [r["level"] for r in self._runs]

    @property
    def entries(self):
        return [r["n"] for r in self._runs]

    # -- runs -----------------------------------------------------------------------------
    def _count(self, n_out) -> int:
        import torch
        torch.cuda.synchronize()
        return int(n_out.view(torch.int64)[0].item())

    def _finish(self, keys, vals, n, level):
        run = dict(keys=keys, vals=vals, n=n, level=level, hindex=None, buckets=0)
        if self.hash_index and n:
            run["buckets"] = lsmkv.lsmkv_hindex_buckets(n)
            run["hindex"] = self.alloc(32 * run["buckets"])
            self.ctx.hindex_build(keys, n, run["hindex"])
        return run

    def add_batch(self, keys, vals, n: int) -> None:
        """keys / vals: device buffers of a write batch in arrival order (duplicates allowed,
        the last arrival wins). It becomes the newest run; merges that are due follow."""
        if n == 0:
            return
        rk, rv, cnt = self.alloc(32 * n), self.alloc(16 * n), self.alloc(8)
        self.ctx.flush_batch(keys, vals, n, rk, rv, cnt)
        self._runs.insert(0, self._finish(rk, rv, self._count(cnt), 1))
        self.compact()

    def compact(self) -> int:
        """Carry out every merge the policy asks for; returns how many steps were taken."""
        steps = 0
        while True:
            plan = lsmkv.lsmkv_plan_compaction(self.levels, self.entries, self.M, self.T, self.K)
            if plan is None:
                return steps
            a, cnt, to = plan
            steps += 1
            part = self._runs[a:a + cnt]
            if cnt == 1:                                   # a move: no data is touched
                part[0]["level"] = to
                continue
            total = sum(r["n"] for r in part)
            ok, ov, n_out = self.alloc(32 * total), self.alloc(16 * total), self.alloc(8)
            self.ctx.merge_runs([(r["keys"], r["vals"], r["n"]) for r in part], ok, ov, n_out)
            self._runs[a:a + cnt] = [self._finish(ok, ov, self._count(n_out), to)]
            self.merges += 1
            self.entries_merged += total

    def runs(self):
        """Run descriptors for lsmkv_probe_batch, newest first."""
        return [(r["keys"], r["vals"], r["n"], None, 0, r["hindex"], r["buckets"])
                for r in self._runs]
