"""Pins for the oracle's index: point lookup over runs (newest first, first match wins, the
LSM point-lookup rule of Sec. 2.2), flush and run merging."""
import bisect

import numpy as np

import oracle
from oracle import VAL_DTYPE


def rand_keys(rng, n, few_words=True):
    k = rng.integers(0, 2**64, (n, 4), dtype=np.uint64)
    if few_words:                       # many ties in leading words: later words must decide
        k[:, 0] = rng.integers(0, 3, n)
        k[:, 1] = rng.integers(0, 4, n)
        k[:, 2] = rng.integers(0, 2**64, n, dtype=np.uint64) & np.uint64(0xF000000000000000)
    return k


def mkvals(file_id, offs):
    v = np.zeros(len(offs), dtype=VAL_DTYPE)
    v["file_id"] = file_id
    v["offset"] = offs
    return v


def tup(k):
    return tuple(int(x) for x in k)


def py_sorted_run(keys, vals):
    d = {}
    for k, v in zip(keys, vals):
        d[tup(k)] = v                   # last arrival wins
    ks = sorted(d)
    return ks, [d[k] for k in ks]


def test_flush_equals_sorted_dict_last_wins():
    rng = np.random.default_rng(1)
    keys = rand_keys(rng, 500)
    keys[100:200] = keys[0:100]         # duplicates, later arrival must survive
    keys[300] = keys[0]
    vals = mkvals(1, np.arange(500) * 16)
    ko, vo = oracle.flush(keys, vals)
    ks, vs = py_sorted_run(keys, vals)
    assert [tup(k) for k in ko] == ks
    assert [int(v["offset"]) for v in vo] == [int(v["offset"]) for v in vs]
    assert len(ko) == len(set(map(tup, keys)))
    assert oracle.flush(keys[:0], vals[:0])[0].shape == (0, 4)


def test_lookup_equals_linear_scan_and_bisect():
    rng = np.random.default_rng(2)
    pool = rand_keys(rng, 400)
    runs, py = [], []
    for r, n in enumerate((5, 40, 300)):
        idx = rng.choice(400, n, replace=False)
        k, v = oracle.flush(pool[idx], mkvals(r, rng.integers(0, 1 << 40, n)))
        runs.append((k, v))
        py.append(([tup(x) for x in k], v))
    for probe in list(pool[:150]) + list(rand_keys(rng, 50)):
        t = tup(probe)
        # linear scan over the runs in age order
        want = None
        for r, (ks, vs) in enumerate(py):
            for i, kk in enumerate(ks):
                if kk == t:
                    want = (r, int(vs[i]["offset"]))
                    break
            if want:
                break
        # library binary search per run
        want2 = None
        for r, (ks, vs) in enumerate(py):
            i = bisect.bisect_left(ks, t)
            if i < len(ks) and ks[i] == t:
                want2 = (r, int(vs[i]["offset"]))
                break
        assert want == want2
        got = oracle.lookup(runs, probe)
        if want is None:
            assert got is None
        else:
            assert (got[1], int(got[0]["offset"]), int(got[0]["file_id"])) == (want[0], want[1],
                                                                              want[0])


def test_newest_run_wins_on_planted_duplicates():
    rng = np.random.default_rng(3)
    old_k = rand_keys(rng, 64, few_words=False)
    old = oracle.flush(old_k, mkvals(7, np.arange(64) * 100))
    new = oracle.flush(old_k[10:20], mkvals(9, np.arange(10) * 100 + 5))
    for i in range(64):
        rec, r = oracle.lookup([new, old], old_k[i])
        if 10 <= i < 20:
            assert (r, int(rec["file_id"]), int(rec["offset"])) == (0, 9, (i - 10) * 100 + 5)
        else:
            assert (r, int(rec["file_id"]), int(rec["offset"])) == (1, 7, i * 100)
    rec, r = oracle.lookup([old, new], old_k[12])          # order of runs is what counts
    assert (r, int(rec["file_id"])) == (0, 7)
    assert oracle.lookup([], old_k[0]) is None
    assert oracle.lookup([(old_k[:0], mkvals(0, []))], old_k[0]) is None


def test_lookup_boundaries():
    k = np.array([[1, 0, 0, 5], [1, 0, 0, 7], [1, 0, 1, 0], [2, 0, 0, 0]], dtype=np.uint64)
    run = (k, mkvals(0, [10, 20, 30, 40]))
    for i in range(4):
        assert int(oracle.lookup([run], k[i])[0]["offset"]) == 10 * (i + 1)
    for miss in ([0, 9, 9, 9], [1, 0, 0, 6], [1, 0, 0, 8], [3, 0, 0, 0], [1, 0, 0, 4]):
        assert oracle.lookup([run], np.array(miss, dtype=np.uint64)) is None


def test_merge_runs_equals_dict_union_newest_wins():
    rng = np.random.default_rng(4)
    pool = rand_keys(rng, 300)
    runs = []
    for r, n in enumerate((20, 100, 250)):
        idx = rng.choice(300, n, replace=False)
        runs.append(oracle.flush(pool[idx], mkvals(r, rng.integers(0, 1 << 30, n))))
    d = {}
    for k, v in reversed(runs):                     # oldest first; newer overwrite
        for kk, vv in zip(k, v):
            d[tup(kk)] = (int(vv["file_id"]), int(vv["offset"]))
    mk, mv = oracle.merge_runs(runs)
    assert [tup(x) for x in mk] == sorted(d)
    assert [(int(v["file_id"]), int(v["offset"])) for v in mv] == [d[k] for k in sorted(d)]
    # lookups through the merged run equal lookups through the run list
    for probe in pool[:100]:
        a, b = oracle.lookup(runs, probe), oracle.lookup([(mk, mv)], probe)
        assert (a is None) == (b is None)
        if a is not None:
            assert a[0] == b[0]


def test_relocate_records_equals_a_numpy_rewrite():
    """Merging tensor files moves records: file ids are renamed and offsets shifted; records of
    other files are untouched."""
    rng = np.random.default_rng(8)
    v = np.zeros(500, dtype=VAL_DTYPE)
    v["file_id"] = rng.integers(0, 6, 500)
    v["reserved"] = rng.integers(0, 99, 500)
    v["offset"] = rng.integers(0, 1 << 40, 500)
    table = np.array([(1, 0, 1 << 33), (2, 0, 5 << 33), (4, 3, 4096)], dtype=oracle.RELOC_DTYPE)
    got, changed = oracle.relocate_records(v, table)
    want = v.copy()
    for old, new, delta in table.tolist():
        m = v["file_id"] == old
        want["file_id"][m] = new
        want["offset"][m] = v["offset"][m] + np.uint64(delta)
    assert np.array_equal(got, want) and changed == int(np.isin(v["file_id"], [1, 2, 4]).sum())
    assert np.array_equal(got["reserved"], v["reserved"])
    # chained names are not followed: 0 -> 7 does not re-move what 1 -> 0 just moved
    got2, _ = oracle.relocate_records(v, np.array([(1, 0, 8), (0, 7, 16)], dtype=oracle.RELOC_DTYPE))
    assert set(got2["file_id"][v["file_id"] == 1]) == {0}
    assert np.array_equal(got2["offset"][v["file_id"] == 0], v["offset"][v["file_id"] == 0] + np.uint64(16))
    assert oracle.relocate_records(v, np.zeros(0, oracle.RELOC_DTYPE))[1] == 0
