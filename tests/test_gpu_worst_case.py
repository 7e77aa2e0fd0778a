"""GPU parity of the exhaustive c_max^(q) search: the paper's printed tables (all rows, including
those too large for the CPU suite), the oracle's maximiser on the smaller clusters, Claim 2."""
import math

import pytest

import oracle
from conftest import read_golden_rows
from paper_2010_04902_b200 import binding as bz

pytestmark = pytest.mark.gpu


def _rows():
    return [tuple(int(x) for x in row[:6]) for row in read_golden_rows("cmax_tables.txt")]


@pytest.mark.parametrize("K,f,l,r,q,cmax", _rows())
def test_printed_tables(K, f, l, r, q, cmax):
    _, fw, mask = bz.assign_mols(l, r)
    got, arg, n = bz.worst_case(mask, f, r, q)
    assert got == cmax and n == math.comb(K, q)
    assert len(arg) == q and list(arg) == sorted(set(arg.tolist()))
    assert oracle.count_distorted(fw, arg) == cmax


@pytest.mark.parametrize("l,r,qs", [(5, 3, range(0, 9)), (5, 5, range(0, 9)), (7, 3, range(0, 8)), (7, 5, [1, 3, 5, 6]),
                                    (7, 7, [1, 4, 5]), (3, 3, range(0, 10)), (3, 1, [1, 2])])
def test_first_maximiser_matches_oracle(l, r, qs):
    wf, _, _ = oracle.assign(l, r)
    _, _, mask = bz.assign_mols(l, r)
    for q in qs:
        want, warg, wn = oracle.worst_case(wf, l * l, r, q)
        got, arg, n = bz.worst_case(mask, l * l, r, q)
        assert (got, n) == (want, wn) and arg.tolist() == warg.tolist(), (l, r, q)


def test_claim2_on_the_largest_cluster():
    # (K, f, l, r) = (49, 49, 7, 7): 0 for q < 4, 1 for 4 <= q < 7, 2 for q = 7 (85.9 million subsets)
    _, _, mask = bz.assign_mols(7, 7)
    for q, want in [(3, 0), (4, 1), (6, 1), (7, 2)]:
        assert bz.worst_case(mask, 49, 7, q)[0] == want


def test_budget():
    _, _, mask = bz.assign_mols(7, 5)
    with pytest.raises(bz.BzError) as e:
        bz.worst_case(mask, 49, 5, 17, max_subsets=10 ** 9)
    assert e.value.status == bz.ERR_BUDGET
    assert bz.worst_case(mask, 49, 5, 3, max_subsets=math.comb(35, 3))[0] == 1
