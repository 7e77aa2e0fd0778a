"""Pins for the oracle's exhaustive c_max^(q) search: the paper's printed tables, Claim 2, the
expansion bound gamma, and an independent itertools brute force on small clusters.  CPU only."""
import itertools
import math

import numpy as np
import pytest

import oracle
from conftest import read_golden_rows

# q up to which each printed table is re-derived on the CPU (kept to a few seconds each; the
# remaining rows of the (35,49,7,5) table are checked on the GPU against the same fixture).
_CPU_Q_LIMIT = {(15, 25, 5, 3): 7, (25, 25, 5, 5): 12, (21, 49, 7, 3): 10, (35, 49, 7, 5): 8}


def _gamma(K, l, r, q):
    # Eq. (5) and Claim 1 with mu_1 = 1/r (Lemma 2).
    mu1 = 1.0 / r
    beta = (q * l / r) / (mu1 + (1.0 - mu1) * q / K)
    return (q * l - beta) / ((r - 1) / 2.0)


def _table_rows():
    out = []
    for K, f, l, r, q, cmax, gamma in read_golden_rows("cmax_tables.txt"):
        out.append((int(K), int(f), int(l), int(r), int(q), int(cmax), float(gamma)))
    return out


@pytest.mark.parametrize("K,f,l,r,q,cmax,gamma", _table_rows())
def test_printed_tables(K, f, l, r, q, cmax, gamma):
    # the printed gamma column (two decimals; one entry is truncated rather than rounded)
    assert abs(_gamma(K, l, r, q) - gamma) <= 0.011
    assert cmax <= _gamma(K, l, r, q) + 1e-9
    if q > _CPU_Q_LIMIT[(K, f, l, r)]:
        pytest.skip("row checked on the GPU only (C(%d,%d) subsets)" % (K, q))
    wf, fw, _ = oracle.assign(l, r)
    got, arg, n = oracle.worst_case(wf, f, r, q)
    assert got == cmax
    assert n == math.comb(K, q)
    assert list(arg) == sorted(set(arg.tolist())) and len(arg) == q
    assert oracle.count_distorted(fw, arg) == cmax


@pytest.mark.parametrize("l,r", [(5, 3), (7, 3), (11, 3), (7, 5), (5, 5), (7, 7), (11, 5)])
def test_claim2_small_q(l, r):
    # Claim 2: r = 3 -> 0, 1, 3 files for q < 2, q = 2, q = 3;
    #          r > 3 -> 0 for q < r', 1 for r' <= q < r, 2 for q = r.
    wf, _, _ = oracle.assign(l, r)
    rp = (r + 1) // 2
    for q in range(0, r + 1):
        if r == 3:
            want = {0: 0, 1: 0, 2: 1, 3: 3}[q]
        else:
            want = 0 if q < rp else (1 if q < r else 2)
        got, _, _ = oracle.worst_case(wf, l * l, r, q)
        assert got == want, (l, r, q)


def _brute(wf, f, r, q):
    """Independent restatement with Python sets: first maximiser in itertools' lexicographic order."""
    K = len(wf)
    rp = (r + 1) // 2
    best, arg = -1, None
    for S in itertools.combinations(range(K), q):
        holders = [0] * f
        for u in S:
            for x in wf[u]:
                holders[x] += 1
        cnt = sum(1 for h in holders if h >= rp)
        if cnt > best:
            best, arg = cnt, S
    return best, list(arg)


@pytest.mark.parametrize("l,r,qs", [(3, 3, [1, 2, 3, 4]), (5, 3, [2, 3, 4]), (5, 5, [3, 4]), (3, 2, [1, 2, 3])])
def test_against_itertools(l, r, qs):
    wf, _, _ = oracle.assign(l, r)
    for q in qs:
        want, warg = _brute(wf.tolist(), l * l, r, q)
        got, arg, _ = oracle.worst_case(wf, l * l, r, q)
        assert got == want and list(arg) == warg


def test_first_maximisers_of_the_benchmark_clusters():
    # Not printed in the paper; pinned here through the independent brute force above.
    for (l, r, q) in [(5, 3, 2), (5, 3, 3)]:
        wf, _, _ = oracle.assign(l, r)
        assert list(oracle.worst_case(wf, l * l, r, q)[1]) == _brute(wf.tolist(), l * l, r, q)[1]
    wf, _, _ = oracle.assign(5, 3)
    assert list(oracle.worst_case(wf, 25, 3, 2)[1]) == [0, 5]


def test_monotone_in_q():
    wf, _, _ = oracle.assign(5, 3)
    vals = [oracle.worst_case(wf, 25, 3, q)[0] for q in range(0, 9)]
    assert vals == sorted(vals)
    assert oracle.worst_case(wf, 25, 3, 15)[0] == 25  # all workers Byzantine
