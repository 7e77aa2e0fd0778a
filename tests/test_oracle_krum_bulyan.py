"""Pins for the oracle's pairwise distances, Krum / Multi-Krum and Bulyan.  CPU only.

The paper cites these aggregators without defining them, so the pins are: exact integer cases
worked by hand, reductions to library routines (plain mean, median, scipy distances), and
invariants of the definitions."""
import numpy as np
import pytest
from scipy.spatial.distance import cdist

import oracle
from paper_2010_04902_b200 import inputs


def _col(vals):
    return np.array(vals, np.float32).reshape(len(vals), 1)


# ------------------------------------------------------------------ distances

def test_pairdist_exact_on_integers():
    v = inputs.integer_gradients(9, 777, seed=4).numpy()
    D = oracle.pairdist(v)
    vi = v.astype(np.int64)
    want = ((vi[:, None, :] - vi[None, :, :]) ** 2).sum(-1)
    assert np.array_equal(D, want.astype(np.float64))
    assert np.array_equal(D, D.T) and (np.diag(D) == 0).all()


def test_pairdist_matches_scipy():
    v = inputs.true_gradients(25, 5000, seed=2).numpy()
    D = oracle.pairdist(v)
    want = cdist(v.astype(np.float64), v.astype(np.float64), "sqeuclidean")
    assert np.allclose(D, want, rtol=1e-12, atol=0)
    v[7] = v[3]
    assert oracle.pairdist(v)[3, 7] == 0.0


def test_pairdist_is_not_transposed():
    # a wrong stride (coordinates taken as rows) would not give these three numbers
    v = np.array([[0, 0, 0], [1, 2, 2], [4, 0, 3]], np.float32)
    D = oracle.pairdist(v)
    assert D[0, 1] == 9 and D[0, 2] == 25 and D[1, 2] == 9 + 4 + 1


# ------------------------------------------------------------------ Krum / Multi-Krum

def test_krum_five_points_on_a_line():
    # points 0,1,2,3,10 ; c = 1 -> nb = 5 - 1 - 2 = 2 nearest neighbours
    # squared distances:  0:{1,4,9,100} 1:{1,1,4,81} 2:{4,1,1,64} 3:{9,4,1,49} 10:{100,81,64,49}
    # scores:             0: 5          1: 2         2: 2         3: 5         10: 113
    v = _col([0, 1, 2, 3, 10])
    D = oracle.pairdist(v)
    assert list(oracle.krum_scores(D, 1)) == [5.0, 2.0, 2.0, 5.0, 113.0]
    assert list(oracle.multikrum_select(D, 1, 1)) == [1]                # Krum; tie 1 vs 2 -> lower index
    assert list(oracle.multikrum_select(D, 1, 3)) == [1, 2, 0]          # tie 0 vs 3 -> lower index
    out, sel, _ = oracle.multikrum(v, 1, 3)
    assert out[0] == np.float32(1.0)
    out4, sel4, _ = oracle.multikrum(v, 1, 4)
    assert list(sel4) == [1, 2, 0, 3] and out4[0] == np.float32(1.5)


def test_krum_two_dimensional_hand_case():
    # rows (0,0) (3,4) (0,1) (6,8) (1,0) (1,1) (50,50); c = 2 -> nb = 7 - 2 - 2 = 3
    v = np.array([[0, 0], [3, 4], [0, 1], [6, 8], [1, 0], [1, 1], [50, 50]], np.float32)
    D = oracle.pairdist(v)
    # from (0,0): 25, 1, 100, 1, 2, 5000 -> 1+1+2 = 4
    # from (3,4): 25, 18, 25, 20, 13, 4325 -> 13+18+20 = 51
    # from (0,1): 1, 18, 85, 2, 1, 4901 -> 1+1+2 = 4
    # from (6,8): 100, 25, 85, 89, 74, 3700 -> 25+74+85 = 184
    # from (1,0): 1, 20, 2, 89, 1, 4901 -> 1+1+2 = 4
    # from (1,1): 2, 13, 1, 74, 1, 4802 -> 1+1+2 = 4
    assert list(oracle.krum_scores(D, 2))[:6] == [4.0, 51.0, 4.0, 184.0, 4.0, 4.0]
    assert list(oracle.multikrum_select(D, 2, 5)) == [0, 2, 4, 5, 1]


def test_multikrum_c0_all_rows_is_the_plain_mean():
    v = inputs.true_gradients(25, 3000, seed=6).numpy()
    out, sel, _ = oracle.multikrum(v, 0, 25)
    assert sorted(sel.tolist()) == list(range(25))
    want = v.astype(np.float64).mean(0)
    assert np.linalg.norm(out - want) <= 1e-7 * np.linalg.norm(want)


def test_multikrum_identical_rows_and_translation():
    row = np.random.default_rng(0).standard_normal(100).astype(np.float32)
    v = np.tile(row, (9, 1))
    out, sel, D = oracle.multikrum(v, 2, 4)
    assert (D == 0).all() and list(sel) == [0, 1, 2, 3] and np.array_equal(out, row)
    vi = inputs.integer_gradients(11, 60, seed=8).numpy()
    s1 = oracle.multikrum_select(oracle.pairdist(vi), 3, 6)
    s2 = oracle.multikrum_select(oracle.pairdist(vi + 1000.0), 3, 6)
    assert list(s1) == list(s2)


def test_multikrum_rejects_what_the_paper_rules_out():
    D = np.zeros((7, 7))
    oracle.multikrum_select(D, 2, 1)          # 7 >= 2*2+3
    for c, m in [(3, 1), (-1, 1), (1, 0), (1, 8)]:
        with pytest.raises(ValueError):
            oracle.multikrum_select(D, c, m)


def test_multikrum_excludes_the_distorted_files():
    # config-3-like cluster: (l, r) = (7, 3), q = 5 at the worst-case placement distorts 8 files;
    # multi-Krum with c = 8 must select honest files only.
    wf, fw, _ = oracle.assign(7, 3)
    _, byz, _ = oracle.worst_case(wf, 49, 3, 5)
    g = inputs.true_gradients(49, 2000, seed=0)
    rep = inputs.build_replicas(g, fw, byz, "reversed").numpy()
    voted = oracle.vote(rep)
    bad = {i for i in range(49) if not np.array_equal(voted[i], g.numpy()[i])}
    assert len(bad) == 8
    out, sel, _ = oracle.multikrum(voted, 8, 41)
    assert not (set(sel.tolist()) & bad)


# ------------------------------------------------------------------ Bulyan

def test_bulyan_seven_points_worked_by_hand():
    # values 0,1,2,3,4,5,100 ; c = 1 -> theta = 5, beta = 3.  Picks (scores in the comments of
    # each round use nb = |R| - 3, floored at 1):
    #  R = all (nb 4): scores 30,15,10,10,15,30,* -> row 2
    #  R \ {2} (nb 3): 0:26 1:14 3:9 4:11 5:21      -> row 3
    #  R = {0,1,4,5,6} (nb 2): 0:17 1:10 4:10 5:17  -> row 1 (tie with 4)
    #  R = {0,4,5,6} (nb 1): 0:16 4:1 5:1           -> row 4 (tie with 5)
    #  R = {0,5,6} (nb 1): 0:25 5:25 6:9025         -> row 0 (tie with 5)
    v = _col([0, 1, 2, 3, 4, 5, 100])
    D = oracle.pairdist(v)
    assert list(oracle.bulyan_select(D, 1)) == [2, 3, 1, 4, 0]
    out, sel, _ = oracle.bulyan(v, 1)
    # sorted selection 0,1,2,3,4: median 2, window grows to 1 (tie -> lower side) then 3
    assert out[0] == np.float32(2.0)


def test_trimmed_mean_hand_cases():
    sel5 = np.arange(5, dtype=np.int32)
    assert oracle.trimmed_mean(_col([0, 10, 11, 12, 100]), sel5, 3)[0] == np.float32(11.0)
    assert oracle.trimmed_mean(_col([0, 1, 2, 50, 60]), sel5, 3)[0] == np.float32(1.0)
    assert oracle.trimmed_mean(_col([60, 2, 50, 0, 1]), sel5, 3)[0] == np.float32(1.0)   # unsorted input
    assert oracle.trimmed_mean(_col([0, 1, 2, 50, 60]), sel5, 5)[0] == np.float32(22.6)
    assert oracle.trimmed_mean(_col([0, 1, 2, 50, 60]), sel5, 1)[0] == np.float32(2.0)
    # a subset of the rows, in pick order
    assert oracle.trimmed_mean(_col([7, 0, 9, 1, 2, 8]), np.array([4, 1, 3], np.int32), 3)[0] == np.float32(1.0)
    # asymmetric growth: lower side on the tie, then the nearer upper value, then the lower one
    assert oracle.trimmed_mean(_col([4, 5, 6, 7, 100]), sel5, 4)[0] == np.float32(5.5)


def test_trimmed_mean_beta1_is_the_median_and_full_is_the_mean():
    v = inputs.true_gradients(25, 2000, seed=9).numpy()
    sel = np.array([3, 20, 7, 1, 14, 9, 22, 0, 11], np.int32)
    assert np.array_equal(oracle.trimmed_mean(v, sel, 1), np.median(v[sel], axis=0))
    assert np.array_equal(oracle.trimmed_mean(v, sel, 1), oracle.median(v[sel]))
    full = oracle.trimmed_mean(v, sel, len(sel))
    want = v[sel].astype(np.float64).mean(0)
    assert np.linalg.norm(full - want) <= 1e-7 * np.linalg.norm(want)


def test_bulyan_c0_is_the_plain_mean():
    v = inputs.true_gradients(25, 1500, seed=10).numpy()
    out, sel, _ = oracle.bulyan(v, 0)
    assert sorted(sel.tolist()) == list(range(25))
    want = v.astype(np.float64).mean(0)
    assert np.linalg.norm(out - want) <= 1e-7 * np.linalg.norm(want)


def test_bulyan_bounds_and_preconditions():
    # config-4-like cluster: (l, r) = (5, 5), q = 6 -> c_max = 4 distorted files (printed table)
    wf, fw, _ = oracle.assign(5, 5)
    _, byz, _ = oracle.worst_case(wf, 25, 5, 6)
    g = inputs.true_gradients(25, 3000, seed=0, heavy_tail_frac=0.01)
    rep = inputs.build_replicas(g, fw, byz, "constant").numpy()
    voted = oracle.vote(rep)
    bad = {i for i in range(25) if not np.array_equal(voted[i], g.numpy()[i])}
    assert len(bad) == 4
    out, sel, _ = oracle.bulyan(voted, 4)
    assert len(sel) == 17 and len(set(sel.tolist())) == 17
    # The late picks run on a set of 2c+1 rows where c identical colluders score zero, so the
    # first stage may admit up to c distorted rows; the trimmed mean is what removes them.
    assert len(set(sel.tolist()) & bad) <= 4
    honest = [i for i in range(25) if i not in bad]
    assert (out >= voted[honest].min(0)).all() and (out <= voted[honest].max(0)).all()
    assert (out >= voted[sel].min(0)).all() and (out <= voted[sel].max(0)).all()
    with pytest.raises(ValueError):          # 4*6+3 > 25: the case the paper calls inapplicable
        oracle.bulyan(voted, 6)
    with pytest.raises(ValueError):
        oracle.bulyan_select(np.zeros((6, 6)), 1)
