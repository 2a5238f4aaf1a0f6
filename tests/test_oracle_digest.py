"""Pins for the oracle's digest (polynomial hash over the Mersenne prime 2^61-1).

Everything here is computed with Python's arbitrary-precision integers from closed forms or
from the polynomial written as an explicit sum, never by calling the oracle on itself.
"""
import json
import os

import numpy as np
import pytest

import oracle

P = (1 << 61) - 1
BASE = (0x0B4E0EF37BC32127, 0x16A09E667F3BCC90)
GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "digest_zero_sequences.json")


def poly_sum(tokens, lane):
    """sum_i (t_i + 1) * B^(n-1-i) mod p, as an explicit sum of powers."""
    n = len(tokens)
    return sum((int(t) + 1) * pow(BASE[lane], n - 1 - i, P) for i, t in enumerate(tokens)) % P


def test_bases_are_canonical():
    assert all(0 < b < P for b in BASE) and BASE[0] != BASE[1]


@pytest.mark.parametrize("lane", [0, 1])
def test_empty_and_single_token(lane):
    assert oracle.digest([], lane) == 0
    for t in (0, 1, 31999, 127999, 2**31, 2**32 - 1):
        assert oracle.digest([t], lane) == t + 1   # t+1 < p: no reduction happens


@pytest.mark.parametrize("lane", [0, 1])
@pytest.mark.parametrize("n", [1, 2, 15, 16, 17, 1000, 32768])
def test_all_zero_tokens_geometric_closed_form(lane, n):
    b = BASE[lane]
    closed = (pow(b, n, P) - 1) * pow(b - 1, P - 2, P) % P   # (B^n - 1) / (B - 1)
    assert oracle.digest(np.zeros(n, dtype=np.uint32), lane) == closed


@pytest.mark.parametrize("lane", [0, 1])
def test_constant_token_geometric_closed_form(lane):
    b, t, n = BASE[lane], 2**32 - 1, 777
    closed = (t + 1) * (pow(b, n, P) - 1) * pow(b - 1, P - 2, P) % P
    assert oracle.digest(np.full(n, t, dtype=np.uint32), lane) == closed


@pytest.mark.parametrize("lane", [0, 1])
def test_random_tokens_equal_explicit_polynomial(lane):
    rng = np.random.default_rng(7)
    for n in (2, 3, 16, 64, 257):
        toks = rng.integers(0, 2**32, n, dtype=np.uint64).astype(np.uint32)
        d = oracle.digest(toks, lane)
        assert d == poly_sum(toks, lane)
        assert 0 <= d < P


@pytest.mark.parametrize("lane", [0, 1])
def test_concatenation_law(lane):
    rng = np.random.default_rng(11)
    toks = rng.integers(0, 128000, 500, dtype=np.uint32)
    for cut in (0, 1, 16, 250, 499, 500):
        x, y = toks[:cut], toks[cut:]
        lhs = oracle.digest(toks, lane)
        rhs = (oracle.digest(x, lane) * pow(BASE[lane], len(y), P) + oracle.digest(y, lane)) % P
        assert lhs == rhs


def test_lanes_differ_and_order_matters():
    a = oracle.digest([5, 9], 0)
    assert a != oracle.digest([5, 9], 1)
    assert a != oracle.digest([9, 5], 0)
    assert a == ((5 + 1) * BASE[0] + (9 + 1)) % P


def test_step_is_horner():
    h = 0x1234567890ABCDEF % P
    for lane in (0, 1):
        assert oracle.digest_step(h, 41, lane) == (h * BASE[lane] + 42) % P
        assert oracle.digest_step(P - 1, 2**32 - 1, lane) == ((P - 1) * BASE[lane] + 2**32) % P


def test_digest_value_p_is_normalised_to_zero():
    """Sequences whose un-reduced Horner value is an exact multiple of p must give 0, never p.
    The stored token triples are checked here against the polynomial with big integers."""
    with open(GOLDEN) as f:
        gold = json.load(f)
    for lane in (0, 1):
        t = gold["zero_digest"][lane]
        assert all(0 <= x < 2**32 for x in t)
        b = BASE[lane]
        raw = (t[0] + 1) * b * b + (t[1] + 1) * b + (t[2] + 1)
        assert raw > 0 and raw % P == 0
        assert oracle.digest(t, lane) == 0
        # after a zero digest, appended tokens hash like a fresh string
        assert oracle.digest(t + [77, 3], lane) == oracle.digest([77, 3], lane)
        assert oracle.digest(t, 1 - lane) != 0


def test_golden_closed_forms():
    """Stored closed-form values (written by tests/golden/make_golden.py from big-int
    arithmetic only)."""
    with open(GOLDEN) as f:
        gold = json.load(f)
    for case in gold["all_zero"]:
        got = oracle.digest(np.zeros(case["n"], dtype=np.uint32), case["lane"])
        assert got == int(case["digest"], 16)
