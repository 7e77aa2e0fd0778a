"""Pins for the oracle's assignment (Algorithm 2 and Ramanujan Case 2) against what the paper prints
and what its lemmas fix.  CPU only."""
import itertools

import numpy as np
import pytest

import oracle
from conftest import read_golden_rows


def _golden_squares():
    rows = read_golden_rows("mols_degree5.txt")
    squares, cur = [], None
    for row in rows:
        if row[0].startswith("L"):
            cur = []
            squares.append(cur)
        else:
            cur.append([int(x) for x in row])
    return [np.array(s) for s in squares]


def test_printed_mols_of_degree_5():
    # Table "three MOLS of degree 5": the symbol in cell (i, j) of square k is the worker's
    # index inside parallel class k.
    _, fw, _ = oracle.assign(5, 3)
    for k, sq in enumerate(_golden_squares()):
        got = (fw[:, k] - 5 * k).reshape(5, 5)
        assert np.array_equal(got, sq), "square L%d" % (k + 1)


def test_printed_assignment_l5_r3():
    wf, fw, mask = oracle.assign(5, 3)
    rows = read_golden_rows("assignment_l5_r3.txt")
    assert len(rows) == 15
    for row in rows:
        u = int(row[0])
        assert list(wf[u]) == [int(x) for x in row[1:]], "worker U_%d" % u
    # Example 1: symbol 0 of L_1 sits in cells (0,0),(1,4),(2,3),(3,2),(4,1).
    assert list(wf[0]) == [0, 9, 13, 17, 21]
    for u in range(15):
        assert int(mask[u]) == sum(1 << int(x) for x in wf[u])
        for x in wf[u]:
            assert u in fw[x]


@pytest.mark.parametrize("l,r", [(3, 2), (5, 3), (5, 4), (5, 5), (7, 3), (7, 5), (7, 7), (11, 4), (13, 13)])
def test_structure(l, r):
    wf, fw, _ = oracle.assign(l, r)
    K, f = r * l, l * l
    assert wf.shape == (K, l) and fw.shape == (f, r)
    # every file: one holder in each parallel class
    for x in range(f):
        assert sorted(int(u) // l for u in fw[x]) == list(range(r))
    # every worker: l distinct files, ascending
    for u in range(K):
        assert len(set(wf[u].tolist())) == l and list(wf[u]) == sorted(wf[u])
    H = np.zeros((K, f), np.int64)
    for u in range(K):
        H[u, wf[u]] = 1
    assert (H.sum(0) == r).all() and (H.sum(1) == l).all()
    # H H^T: l on the diagonal, 0 inside a class, exactly 1 across classes (Sec. 4.1.2 and the
    # block form in the proof of Lemma 2).
    G = H @ H.T
    for u, v in itertools.product(range(K), repeat=2):
        want = l if u == v else (0 if u // l == v // l else 1)
        assert G[u, v] == want


@pytest.mark.parametrize("l,r", [(5, 3), (7, 3), (7, 5), (5, 5), (7, 7)])
def test_spectrum_of_AAt(l, r):
    # Lemma 2: spectrum {(1, 1), (1/r, r(l-1)), (0, r-1)}; Case 2 with l = r has the same form.
    wf, _, _ = oracle.assign(l, r)
    K, f = r * l, l * l
    H = np.zeros((K, f))
    for u in range(K):
        H[u, wf[u]] = 1.0
    A = H / np.sqrt(l * r)
    ev = np.sort(np.linalg.eigvalsh(A @ A.T))[::-1]
    want = np.array([1.0] + [1.0 / r] * (r * (l - 1)) + [0.0] * (r - 1))
    assert np.allclose(ev, want, atol=1e-9)


@pytest.mark.parametrize("s", [3, 5, 7])
def test_ramanujan_case2_array_code(s):
    # Sec. 4.2.1 with m = s: B is an s x s block matrix whose block (a, b) is P^(a*b), with P the
    # cyclic shift P_ij = 1 iff j = i - 1 (mod s); H = B, rows are workers, columns are files.
    P = np.zeros((s, s), np.int64)
    for i in range(s):
        P[i, (i - 1) % s] = 1
    B = np.block([[np.linalg.matrix_power(P, a * b) for b in range(s)] for a in range(s)])
    wf, _, _ = oracle.assign(s, s)
    H = np.zeros((s * s, s * s), np.int64)
    for u in range(s * s):
        H[u, wf[u]] = 1
    assert np.array_equal(H, B)


@pytest.mark.parametrize("l,r", [(4, 2), (6, 3), (9, 2), (5, 6), (5, 7), (5, 0), (1, 1)])
def test_rejected(l, r):
    with pytest.raises(ValueError):
        oracle.assign(l, r)
