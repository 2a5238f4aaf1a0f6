"""The compaction planner (host logic, no GPU): the (T, K) policy of Sec. 2.2 -- level capacities
growing by the size ratio T, at most K runs per level -- checked against what the policy fixes:
tiering (K = T - 1) is a base-T counter, leveling (K = 1) keeps one run per level, no level ends
up over its capacity or its run count, and parameter changes act lazily."""
import ctypes

import pytest

from paper_2511_16138_b200 import lsmkv


def settle(levels, entries, M, T, K, max_steps=1000):
    """Apply planned merges (distinct keys: a merge adds the sizes) until nothing is due.
    Returns the merged-entry total (what compaction wrote)."""
    written = 0
    for _ in range(max_steps):
        plan = lsmkv.lsmkv_plan_compaction(levels, entries, M, T, K)
        if plan is None:
            return written
        a, n, to = plan
        assert n >= 1 and to >= levels[a] and to <= levels[a + n - 1] + 1
        total = sum(entries[a:a + n])
        if n > 1:
            written += total
        levels[a:a + n] = [to]
        entries[a:a + n] = [total]
        assert levels == sorted(levels)
    raise AssertionError("planner does not settle")


def digits(n, base):
    out = []
    while n:
        out.append(n % base)
        n //= base
    return out


@pytest.mark.parametrize("T", [2, 3, 4, 10])
def test_tiering_counts_flushes_in_base_T(T):
    M, K = 100, T - 1
    levels, entries = [], []
    for n in range(1, 3 * T * T + 5):
        levels.insert(0, 1)                      # a flushed batch enters level 1, newest first
        entries.insert(0, M)
        settle(levels, entries, M, T, K)
        want = digits(n, T)
        for i, d in enumerate(want, start=1):
            assert levels.count(i) == d, (n, levels)
        assert max(levels) == len(want)
        for lv, e in zip(levels, entries):       # a run of level i is T^(i-1) batches
            assert e == M * T ** (lv - 1)


@pytest.mark.parametrize("T", [2, 4, 8])
def test_leveling_keeps_one_run_per_level_below_capacity(T):
    M = 64
    levels, entries = [], []
    written = 0
    for n in range(1, 200):
        levels.insert(0, 1)
        entries.insert(0, M)
        written += settle(levels, entries, M, T, 1)
        assert len(set(levels)) == len(levels)               # one run per level
        for lv, e in zip(levels, entries):
            assert e < M * T ** lv                            # below its capacity
        assert sum(entries) == n * M
    # leveling rewrites data about T/2 times per level it passes: more than tiering would
    t_levels, t_entries, t_written = [], [], 0
    for n in range(1, 200):
        t_levels.insert(0, 1)
        t_entries.insert(0, M)
        t_written += settle(t_levels, t_entries, M, T, T - 1)
    assert written >= t_written


def test_random_batches_never_leave_a_level_over_its_limits():
    import random
    rnd = random.Random(5)
    for T, K in ((3, 1), (3, 2), (5, 2), (6, 5), (4, 7)):
        M = 50
        levels, entries = [], []
        for _ in range(300):
            levels.insert(0, 1)
            entries.insert(0, rnd.randint(1, 2 * M))
            settle(levels, entries, M, T, K)
            for i in set(levels):
                assert levels.count(i) <= K
                assert sum(e for lv, e in zip(levels, entries) if lv == i) < M * T ** i


def test_a_move_without_a_merge_and_the_join_with_a_full_next_level():
    # one over-full run at level 1, nothing below: it just moves
    assert lsmkv.lsmkv_plan_compaction([1], [500], 100, 4, 3) == (0, 1, 2)
    # level 1 full (4 runs of 100 = 100 * 4), level 2 already holds K = 1 run: all five merge
    assert lsmkv.lsmkv_plan_compaction([1, 1, 1, 1, 2], [100] * 4 + [700], 100, 4, 1) == (0, 5, 2)
    # with room for another run at level 2 only level 1's runs merge
    assert lsmkv.lsmkv_plan_compaction([1, 1, 1, 1, 2], [100] * 4 + [700], 100, 4, 3) == (0, 4, 2)
    # too many runs, not full: merged in place; the shallowest level that needs work goes first
    assert lsmkv.lsmkv_plan_compaction([1, 1, 2, 2, 2], [10, 10, 300, 300, 300], 100, 4, 1) == (0, 2, 1)
    assert lsmkv.lsmkv_plan_compaction([1, 2, 2, 2], [20, 300, 300, 300], 100, 4, 2) == (1, 3, 2)
    assert lsmkv.lsmkv_plan_compaction([], [], 100, 4, 2) is None
    assert lsmkv.lsmkv_plan_compaction([1, 3], [99, 6399], 100, 4, 1) is None


def test_new_parameters_act_at_the_next_merge_only():
    M = 10
    levels, entries = [], []
    for _ in range(7):                                   # tiering, T = 4: 7 = "13" in base 4
        levels.insert(0, 1)
        entries.insert(0, M)
        settle(levels, entries, M, 4, 3)
    assert levels == [1, 1, 1, 2]
    # K drops to 1: nothing moves until asked, then only what the policy names, level by level
    shape = (list(levels), list(entries))
    assert lsmkv.lsmkv_plan_compaction(levels, entries, M, 4, 1) == (0, 3, 1)
    assert (levels, entries) == (shape[0], shape[1])     # planning changes nothing by itself
    settle(levels, entries, M, 4, 1)
    assert levels == [1, 2] and entries == [30, 40]
    # K rises again: the merged runs stay merged
    assert lsmkv.lsmkv_plan_compaction(levels, entries, M, 4, 3) is None


def test_bad_arguments():
    out = lsmkv.CompactionStruct()
    L = lsmkv.lib()
    lv = (ctypes.c_uint32 * 2)(2, 1)                     # a deeper run listed as the newer one
    en = (ctypes.c_uint64 * 2)(5, 5)
    assert L.lsmkv_plan_compaction(lv, en, 2, 10, 4, 1, ctypes.byref(out)) == lsmkv.EINVAL
    lv = (ctypes.c_uint32 * 2)(0, 1)
    assert L.lsmkv_plan_compaction(lv, en, 2, 10, 4, 1, ctypes.byref(out)) == lsmkv.EINVAL
    lv = (ctypes.c_uint32 * 2)(1, 1)
    assert L.lsmkv_plan_compaction(lv, en, 2, 0, 4, 1, ctypes.byref(out)) == lsmkv.EINVAL
    assert L.lsmkv_plan_compaction(lv, en, 2, 10, 1, 1, ctypes.byref(out)) == lsmkv.EINVAL
    assert L.lsmkv_plan_compaction(lv, en, 2, 10, 4, 0, ctypes.byref(out)) == lsmkv.EINVAL
    assert L.lsmkv_plan_compaction(lv, en, 2, 10, 4, 1, None) == lsmkv.EINVAL
