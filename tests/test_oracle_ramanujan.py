"""Pins for the oracle's Ramanujan-bigraph assignment (Sec. 4.2.1, Eq. 7) and the library's host
implementation of it.  CPU only."""
import numpy as np
import pytest

import oracle
from conftest import read_golden_rows
from paper_2010_04902_b200 import binding as bz
from paper_2010_04902_b200 import build as bz_build


def _H(wf, f):
    H = np.zeros((len(wf), f), np.int64)
    for u in range(len(wf)):
        H[u, wf[u]] = 1
    return H


@pytest.mark.parametrize("m,s", [(2, 3), (3, 5), (4, 5), (3, 7), (5, 7), (5, 5), (7, 7), (10, 5), (6, 3), (7, 5)])
def test_shape_degrees_and_lists(m, s):
    K, f, l, r = oracle.ramanujan_dims(m, s)
    assert (K, f, l, r) == ((m * s, s * s, s, m) if m < s else (s * s, m * s, m, s))   # Eq. (7)
    wf, fw, _ = oracle.assign_ramanujan(m, s)
    H = _H(wf, f)
    assert (H.sum(1) == l).all() and (H.sum(0) == r).all()
    for u in range(K):
        assert list(wf[u]) == sorted(set(wf[u].tolist()))
    for x in range(f):
        assert list(fw[x]) == sorted(set(fw[x].tolist())) and all(x in wf[u] for u in fw[x])


@pytest.mark.parametrize("m,s", [(3, 5), (4, 5), (3, 7), (5, 7), (2, 3)])
def test_case1_spectrum_and_intersections(m, s):
    # Lemma 2, Ramanujan Case 1: spectrum of A A^T = {(1,1), (1/r, r(l-1)), (0, r-1)} with (l, r) = (s, m);
    # proof of Claim 2: workers of one class share no file, workers of two classes share exactly one
    K, f, l, r = oracle.ramanujan_dims(m, s)
    wf, _, _ = oracle.assign_ramanujan(m, s)
    H = _H(wf, f).astype(np.float64)
    ev = np.sort(np.linalg.eigvalsh(H @ H.T / (l * r)))[::-1]
    want = np.array([1.0] + [1.0 / r] * (r * (l - 1)) + [0.0] * (r - 1))
    assert np.allclose(ev, want, atol=1e-9)
    G = (H @ H.T).astype(np.int64)
    for u in range(K):
        for v in range(K):
            assert G[u, v] == (l if u == v else (0 if u // s == v // s else 1))


@pytest.mark.parametrize("m,s", [(5, 5), (10, 5), (6, 3), (7, 7)])
def test_case2_spectrum_when_s_divides_m(m, s):
    # Lemma 2, Ramanujan Case 2 (requires s | m): {(1,1), (1/r, r(r-1)), (0, r-1)} with r = s
    K, f, l, r = oracle.ramanujan_dims(m, s)
    wf, _, _ = oracle.assign_ramanujan(m, s)
    H = _H(wf, f).astype(np.float64)
    ev = np.sort(np.linalg.eigvalsh(H @ H.T / (l * r)))[::-1]
    want = np.array([1.0] + [1.0 / r] * (r * (r - 1)) + [0.0] * (r - 1))
    assert np.allclose(ev, want, atol=1e-9)


def test_case1_reproduces_the_printed_table():
    # Sec. 5.3.2: for (K, f, l, r) = (15, 25, 5, 3) the simulated c_max of the Ramanujan Case 1 scheme
    # was identical to the MOLS one, so the paper prints one table for both
    wf, fw, _ = oracle.assign_ramanujan(3, 5)
    for K, f, l, r, q, cmax, _ in read_golden_rows("cmax_tables.txt"):
        if (K, f, l, r) == ("15", "25", "5", "3"):
            got, arg, _ = oracle.worst_case(wf, 25, 3, int(q))
            assert got == int(cmax)
            assert oracle.count_distorted(fw, arg) == int(cmax)


def test_case2_square_equals_the_r_equals_l_assignment():
    for s in (3, 5, 7):
        a, b = oracle.assign_ramanujan(s, s), oracle.assign(s, s)
        assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])


@pytest.mark.parametrize("m,s", [(3, 5), (5, 7), (4, 7)])
def test_claim2_case1(m, s):
    # Claim 2 also covers the Ramanujan schemes
    wf, _, _ = oracle.assign_ramanujan(m, s)
    r, rp = m, (m + 1) // 2
    if r % 2 == 0:
        pytest.skip("the majority rule needs odd r")
    for q in range(0, r + 1):
        want = {0: 0, 1: 0, 2: 1, 3: 3}[q] if r == 3 else (0 if q < rp else (1 if q < r else 2))
        assert oracle.worst_case(wf, s * s, r, q)[0] == want


@pytest.mark.parametrize("m,s", [(1, 5), (3, 4), (3, 9), (0, 3), (3, 1)])
def test_rejected(m, s):
    with pytest.raises(ValueError):
        oracle.assign_ramanujan(m, s)
    bz_build.build()
    with pytest.raises(bz.BzError) as e:
        bz.assign_ramanujan(m, s)
    assert e.value.status == bz.ERR_INVALID_ARG


@pytest.mark.parametrize("m,s", [(2, 3), (3, 5), (4, 5), (3, 7), (5, 7), (5, 5), (7, 7), (10, 5), (12, 5), (6, 3), (13, 11)])
def test_library_matches_the_oracle(m, s):
    bz_build.build()
    wf, fw, mask = bz.assign_ramanujan(m, s)
    owf, ofw, omask = oracle.assign_ramanujan(m, s)
    assert np.array_equal(wf, owf) and np.array_equal(fw, ofw)
    K, f, l, r = bz.ramanujan_dims(m, s)
    if f <= 64:
        assert np.array_equal(mask, omask)
    else:
        assert mask is None
