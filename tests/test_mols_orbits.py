"""Host logic of the symmetry-reduced worst-case search (Sec. 5.3.2 / Sec. 6.1 on the placements of
Algorithm 2): the translations of the file grid are automorphisms, and the number of worker sets the
search visits is the number of their orbits - checked against the oracle's placement, brute force and
the orbit-counting (Burnside) formula.  No GPU needed."""
import itertools
from math import comb

import numpy as np
import pytest

import oracle
from paper_2010_04902_b200 import binding as bz


def _translations(l, r):
    """For every (a, b): the worker permutation induced by moving file (i, j) to (i + a, j + b), read off
    the oracle's placement (asserting that the image of a worker's file set is again a worker's)."""
    wf, _, _ = oracle.assign(l, r)
    sets = {frozenset(int(x) for x in row): u for u, row in enumerate(wf)}
    perms = []
    for a in range(l):
        for b in range(l):
            perm = []
            for u in range(r * l):
                image = frozenset(((x // l + a) % l) * l + (x % l + b) % l for x in wf[u])
                assert image in sets, "a translation is not an automorphism of the placement"
                v = sets[image]
                assert v // l == u // l           # it stays inside the parallel class
                perm.append(v)
            perms.append(perm)
    return perms


def _burnside(l, r, q):
    K = r * l
    full_classes = comb(r, q // l) if q % l == 0 else 0                      # sets fixed when every class moves
    one_fixed = sum(comb(l, j) * comb(r - 1, (q - j) // l) for j in range(0, min(l, q) + 1) if (q - j) % l == 0)
    total = comb(K, q) + (l - 1) * full_classes + r * (l - 1) * one_fixed + (l - r) * (l - 1) * full_classes
    assert total % (l * l) == 0
    return total // (l * l)


@pytest.mark.parametrize("l,r", [(3, 3), (5, 3)])
def test_orbit_count_by_brute_force(l, r):
    perms = _translations(l, r)
    K = r * l
    for q in range(0, K + 1 if l == 3 else 6):
        seen = set()
        for S in itertools.combinations(range(K), q):
            seen.add(min(tuple(sorted(p[u] for u in S)) for p in perms))
        assert bz.mols_orbit_count(l, r, q) == len(seen) == _burnside(l, r, q), (l, r, q)


@pytest.mark.parametrize("l,r", [(5, 3), (5, 5), (7, 3), (7, 5), (7, 7)])
def test_orbit_count_matches_the_counting_formula(l, r):
    _translations(l, r)
    for q in range(0, r * l + 1):
        assert bz.mols_orbit_count(l, r, q) == _burnside(l, r, q), (l, r, q)
    # nearly l*l fewer sets than C(K, q) in the middle of the range
    K = r * l
    assert bz.mols_orbit_count(l, r, K // 2) * l * l < comb(K, K // 2) * 1.1


def test_distortion_is_invariant_under_translations():
    l, r = 5, 3
    perms = _translations(l, r)
    _, fw, _ = oracle.assign(l, r)
    rng = np.random.default_rng(0)
    for _ in range(20):
        S = rng.choice(r * l, size=int(rng.integers(2, 8)), replace=False)
        want = oracle.count_distorted(fw, np.sort(S).astype(np.int32))
        for p in perms:
            assert oracle.count_distorted(fw, np.sort([p[u] for u in S]).astype(np.int32)) == want


def test_argument_checks():
    with pytest.raises(bz.BzError) as e:
        bz.mols_orbit_count(4, 3, 2)         # l not prime
    assert e.value.status == bz.ERR_INVALID_ARG
    with pytest.raises(bz.BzError) as e:
        bz.mols_orbit_count(5, 4, 2)         # r even
    assert e.value.status == bz.ERR_INVALID_ARG
    with pytest.raises(bz.BzError) as e:
        bz.mols_orbit_count(11, 3, 2)        # more than 64 files
    assert e.value.status == bz.ERR_UNSUPPORTED
