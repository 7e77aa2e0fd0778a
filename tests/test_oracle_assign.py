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


@pytest.mark.parametrize("l,r", [(4, 4), (6, 3), (10, 2), (5, 6), (5, 7), (5, 0), (1, 1)])
def test_rejected(l, r):
    with pytest.raises(ValueError):
        oracle.assign(l, r)


# ---- prime-power l (Sec. 4.1.1: rows, columns and symbols are the elements of F_l) ----------------

@pytest.mark.parametrize("l", [2, 3, 4, 5, 7, 8, 9, 16, 25, 27])
def test_field_axioms_by_brute_force(l):
    add, mul = oracle.field_tables(l)
    e = np.arange(l)
    # abelian group under +, identity 0; nonzero elements a group under *, identity 1
    assert np.array_equal(add, add.T) and np.array_equal(mul, mul.T)
    assert np.array_equal(add[0], e) and np.array_equal(mul[1], e) and (mul[0] == 0).all()
    for a in range(l):
        assert sorted(add[a]) == list(range(l))
        if a:
            assert sorted(mul[a]) == list(range(l))
    # associativity and distributivity on every triple
    A = add[add[:, :, None], e[None, None, :]]            # (a+b)+c
    B = add[e[:, None, None], add[None, :, :]]            # a+(b+c)
    assert np.array_equal(A, B)
    assert np.array_equal(mul[mul[:, :, None], e[None, None, :]], mul[e[:, None, None], mul[None, :, :]])
    assert np.array_equal(mul[e[:, None, None], add[None, :, :]], add[mul[:, :, None], mul[:, None, :]])
    # characteristic p: adding an element p times gives 0
    p = next(q for q in range(2, l + 1) if l % q == 0)
    x = np.zeros(l, int)
    for _ in range(p):
        x = add[x, e]
    assert (x == 0).all()


def test_textbook_fields():
    # prime l: arithmetic mod l;  l = 4, 8, 16: addition is XOR on the coefficient bits
    for l in (3, 5, 7):
        add, mul = oracle.field_tables(l)
        e = np.arange(l)
        assert np.array_equal(add, (e[:, None] + e[None, :]) % l) and np.array_equal(mul, (e[:, None] * e[None, :]) % l)
    for l in (4, 8, 16):
        add, _ = oracle.field_tables(l)
        e = np.arange(l)
        assert np.array_equal(add, e[:, None] ^ e[None, :])
    # GF(4) = {0, 1, x, x+1} with x^2 = x + 1: the multiplication table of every textbook
    _, mul = oracle.field_tables(4)
    assert mul.tolist() == [[0, 0, 0, 0], [0, 1, 2, 3], [0, 2, 3, 1], [0, 3, 1, 2]]
    # GF(8) with x^3 = x + 1: x has order 7 and its powers run 2, 4, 3, 6, 7, 5, 1
    _, mul = oracle.field_tables(8)
    powers, y = [], 1
    for _ in range(7):
        y = int(mul[y, 2])
        powers.append(y)
    assert powers == [2, 4, 3, 6, 7, 5, 1]
    # GF(9) with x^2 = -1: x (= 3) has order 4, x^2 = 2 = -1
    _, mul = oracle.field_tables(9)
    assert int(mul[3, 3]) == 2 and int(mul[2, 2]) == 1
    for l in (6, 10, 12, 1):
        with pytest.raises(ValueError):
            oracle.field_tables(l)


@pytest.mark.parametrize("l,r", [(4, 3), (8, 3), (8, 5), (8, 7), (9, 3), (9, 5)])
def test_prime_power_placement(l, r):
    wf, fw, mask = oracle.assign(l, r)
    K, f = r * l, l * l
    # the r squares L_alpha(i, j) = alpha*i + j are Latin and mutually orthogonal
    sq = np.zeros((r, l, l), int)
    for file in range(f):
        for k in range(r):
            sq[k, file // l, file % l] = fw[file, k] - k * l
    for k in range(r):
        for i in range(l):
            assert sorted(sq[k, i]) == list(range(l)) and sorted(sq[k, :, i]) == list(range(l))
        for k2 in range(k + 1, r):
            assert len({(sq[k, i, j], sq[k2, i, j]) for i in range(l) for j in range(l)}) == l * l
    # every file has r workers (one per class), every worker l files; workers of one class are
    # disjoint, workers of different classes share exactly one file (Sec. 4.1.2)
    H = np.zeros((K, f), int)
    for u in range(K):
        H[u, wf[u]] = 1
    assert (H.sum(0) == r).all() and (H.sum(1) == l).all()
    G = H @ H.T
    for u in range(K):
        for v in range(K):
            want = l if u == v else (0 if u // l == v // l else 1)
            assert G[u, v] == want
    # Lemma 2: the biadjacency matrix has singular values sqrt(r*l) once, sqrt(l) (r*(l-1) times), 0 otherwise
    ev = np.sort(np.linalg.eigvalsh(G.astype(float)))[::-1]
    assert abs(ev[0] - r * l) < 1e-9 and np.allclose(ev[1:1 + r * (l - 1)], l) and np.allclose(ev[1 + r * (l - 1):], 0, atol=1e-9)
    if f <= 64:
        for u in range(K):
            assert mask[u] == sum(1 << int(x) for x in wf[u])


def test_prime_power_claim_2_and_limits():
    # Claim 2 holds for every MOLS placement: r = 3 gives c_max = 0, 1, 3 for q = 1, 2, 3
    wf, _, _ = oracle.assign(4, 3)
    assert [oracle.worst_case(wf, 16, 3, q)[0] for q in (1, 2, 3)] == [0, 1, 3]
    wf, _, _ = oracle.assign(8, 5)
    assert [oracle.worst_case(wf, 64, 5, q)[0] for q in (2, 3, 4)] == [0, 1, 1]
    # Algorithm 2 offers l - 1 squares; r = l exists only through the bigraph of Sec. 4.2.1 (prime l)
    for l, r in [(4, 4), (8, 8), (9, 9), (6, 3), (12, 5)]:
        with pytest.raises(ValueError):
            oracle.assign(l, r)
