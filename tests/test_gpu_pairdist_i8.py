"""GPU parity of the integer (tensor-core) distance kernel against the CPU oracle.

BZ_PAIRDIST_PATH=i8 takes that kernel's result whatever its own error bound says, =fp32 / =fp64 keep the
distances on the binary32 / binary64 kernels; unset, the library decides.  Shapes here satisfy the kernel's
conditions (f in {25, 49}, 16-byte aligned rows, d >= 8192), so "i8" really runs it."""
import numpy as np
import pytest
import torch

import oracle
from paper_2010_04902_b200 import binding as bz
from paper_2010_04902_b200 import inputs

pytestmark = pytest.mark.gpu

DEV = "cuda"
DIST_TOL = 1e-7      # relative error of a squared distance, as for the binary32 kernels


def _voted(l, r, q, d, attack, seed=0, heavy=0.0):
    wf, fw, _ = oracle.assign(l, r)
    byz = oracle.worst_case(wf, l * l, r, q)[1]
    g = inputs.true_gradients(l * l, d, seed=seed, heavy_tail_frac=heavy)
    rep = inputs.build_replicas(g, fw, byz, attack)
    return rep, torch.from_numpy(oracle.vote(rep.numpy()))


def _check_close(got, want):
    assert np.array_equal(got, got.T) and (np.diag(got) == 0).all()
    off = ~np.eye(want.shape[0], dtype=bool)
    nz = off & (want > 0)
    assert (np.abs(got[nz] - want[nz]) <= DIST_TOL * want[nz]).all()
    assert (got[off & (want == 0)] == 0).all()     # identical (colluding) rows


@pytest.mark.parametrize("f,d", [(25, 8192), (49, 8192), (25, 70004), (49, 100000), (49, 1_000_004)])
def test_exact_on_integer_rows(f, d, monkeypatch):
    monkeypatch.setenv("BZ_PAIRDIST_PATH", "i8")
    v = inputs.integer_gradients(f, d, seed=f + d)
    want = oracle.pairdist(v.numpy())
    got = bz.pairdist(v.to(DEV)).cpu().numpy()
    assert np.array_equal(got, want)


@pytest.mark.parametrize("l,r,q,attack,d,heavy", [(5, 3, 3, "reversed", 50004, 0.0), (7, 3, 5, "alie", 50004, 0.0),
                                                  (5, 5, 6, "constant", 200000, 0.01), (7, 3, 5, "alie", 1_000_004, 0.0)])
def test_close_on_gradients(l, r, q, attack, d, heavy, monkeypatch):
    monkeypatch.setenv("BZ_PAIRDIST_PATH", "i8")
    _, v = _voted(l, r, q, d, attack, heavy=heavy)
    want = oracle.pairdist(v.numpy())
    got = bz.pairdist(v.to(DEV)).cpu().numpy()
    _check_close(got, want)
    assert np.array_equal(bz.pairdist(v.to(DEV)).cpu().numpy(), got)   # integer sums: the same bits every time


def test_outliers_late_in_a_row():
    # A CTA fixes a row's scale when it first meets the row.  Later values that do not fit it enter the
    # contraction as zero, are listed, and a small kernel adds what they really contribute: the integer kernel's
    # result stands (status 0) and is as accurate as without them.
    f, d = 49, 400_000
    g = inputs.true_gradients(f, d, seed=5).numpy()
    g[3, 150_000] = 3.0e4
    g[3, 300_000] = -7.0e8
    g[17, 222_222] = 55.0
    g[17, 222_223] = -1.0e3
    g[9, 222_222] = 77.0                # two rows with an outlier at the same coordinate
    g[21, 399_999] = 1.0e5              # the last coordinate
    g[40] *= 1.0e-6
    g[41] = g[40]
    want = oracle.pairdist(g)
    ws = bz.alloc_workspace(bz.OP_PAIRDIST, 0, f, d)
    got = bz.pairdist(torch.from_numpy(g).to(DEV), workspace=ws).cpu().numpy()
    assert bz.last_path() == bz.PATH_TENSOR and bz.pairdist_status(ws, f) == 0
    _check_close(got, want)
    off = ~np.eye(f, dtype=bool) & (want > 0)
    assert (np.abs(got[off] - want[off]) <= 2e-9 * want[off]).all()
    # the same through the vote
    rep = torch.from_numpy(np.stack([g, g, g]))
    rep[0, 17, 222_223] = 5.0e8         # outvoted
    voted, dist = bz.vote_pairdist(rep.to(DEV), workspace=ws)
    assert bz.pairdist_status(ws, f) == 0
    assert np.array_equal(voted.cpu().numpy().view(np.uint32), g.view(np.uint32))
    _check_close(dist.cpu().numpy(), want)


def test_outliers_where_a_cta_first_meets_a_row():
    # eight isolated values of very different sizes inside the first 256 coordinates (the first step of CTA 0): they
    # are peeled off two at a time before the row's scale is fixed, so the scale is that of the ordinary values and
    # nothing of the row is lost; a ninth would set the scale instead (the second case)
    f, d = 49, 300_000
    for extra in (0, 1):
        g = inputs.true_gradients(f, d, seed=31 + extra).numpy()
        for k, mag in enumerate([3.0e7, -2.0e7, 4.0e5, 3.5e5, -6.0e3, 5.0e3, 90.0, -80.0] + [40.0] * extra):
            g[12, 3 + 29 * k] = mag
        g[20, 5] = 1.0e4
        want = oracle.pairdist(g)
        ws = bz.alloc_workspace(bz.OP_PAIRDIST, 0, f, d)
        got = bz.pairdist(torch.from_numpy(g).to(DEV), workspace=ws).cpu().numpy()
        assert bz.last_path() == bz.PATH_TENSOR
        _check_close(got, want)
        if extra == 0:
            assert bz.pairdist_status(ws, f) == 0


def test_a_row_that_outgrows_its_scale():
    # more large values than a list holds (78 inside one tile; and a whole stretch of the row 300 times larger, the
    # way gradients change magnitude from layer to layer): the CTAs that meet them give the row a coarser scale
    # and read the accumulators back; the integer kernel still answers
    f, d = 49, 400_000
    g = inputs.true_gradients(f, d, seed=5).numpy()
    g[17, 222_222:222_300] *= 1.0e3
    g[:, 300_000:] *= 300.0
    g[5, 100_000:] *= 1.0e-3
    want = oracle.pairdist(g)
    ws = bz.alloc_workspace(bz.OP_PAIRDIST, 0, f, d)
    got = bz.pairdist(torch.from_numpy(g).to(DEV), workspace=ws).cpu().numpy()
    assert bz.last_path() == bz.PATH_TENSOR and bz.pairdist_status(ws, f) == 0
    _check_close(got, want)


def test_scale_changes_give_the_same_answer_every_launch():
    # the same rows as above, 30 launches: a change of scale involves every role of a CTA (converters, the MMA thread's
    # read-back request, the drain warps), so a hand-off that depended on timing would show as a launch that differs
    f, d = 49, 400_000
    g = inputs.true_gradients(f, d, seed=5).numpy()
    g[17, 222_222:222_300] *= 1.0e3
    g[:, 300_000:] *= 300.0
    g[5, 100_000:] *= 1.0e-3
    want = oracle.pairdist(g)
    ws = bz.alloc_workspace(bz.OP_PAIRDIST, 0, f, d)
    v = torch.from_numpy(g).to(DEV)
    first = bz.pairdist(v, workspace=ws).cpu().numpy()
    _check_close(first, want)
    for _ in range(30):
        again = bz.pairdist(v, workspace=ws).cpu().numpy()
        assert np.array_equal(again, first) and bz.pairdist_status(ws, f) == 0


@pytest.mark.parametrize("seed", range(8))
def test_randomised_scales_outliers_and_sparse_rows(seed):
    # rows whose magnitude changes from segment to segment (layers), single outliers, rows that start with zeros,
    # copies of rows: whatever mix of listing, rescaling and fall-back the kernel takes, every distance stays within
    # the tolerance and identical rows stay at exactly 0
    rng = np.random.default_rng(100 + seed)
    f = 25 if seed % 2 else 49
    d = int(rng.integers(9_000, 400_000)) // 4 * 4
    g = inputs.true_gradients(f, d, seed=seed).numpy()
    for _ in range(int(rng.integers(0, 5))):                      # layer-like segments, for all rows or for one
        j0 = int(rng.integers(0, d - 1000))
        j1 = int(rng.integers(j0 + 1, d))
        scale = float(10.0 ** rng.uniform(-4, 4))
        rows = slice(None) if rng.random() < 0.5 else int(rng.integers(0, f))
        g[rows, j0:j1] *= scale
    for _ in range(int(rng.integers(0, 40))):                     # isolated outliers
        g[int(rng.integers(0, f)), int(rng.integers(0, d))] *= float(10.0 ** rng.uniform(1, 6))
    if rng.random() < 0.5:                                        # a row that is zero at first
        g[int(rng.integers(0, f)), :int(rng.integers(1, d // 2))] = 0.0
    a, b = rng.choice(f, size=2, replace=False)
    g[a] = g[b]                                                   # colluding copies
    want = oracle.pairdist(g)
    ws = bz.alloc_workspace(bz.OP_PAIRDIST, 0, f, d)
    got = bz.pairdist(torch.from_numpy(g).to(DEV), workspace=ws).cpu().numpy()
    assert bz.last_path() == bz.PATH_TENSOR
    _check_close(got, want)
    if bz.pairdist_status(ws, f) == 0:      # the integer kernel's answer: far inside the tolerance
        off = ~np.eye(f, dtype=bool) & (want > 0)
        assert (np.abs(got[off] - want[off]) <= 2e-8 * want[off]).all()
    r = 3 if seed % 4 < 2 else 5
    rep = np.stack([g] * r)
    rep[int(rng.integers(0, r)), int(rng.integers(0, f))] = 7.0   # one Byzantine copy, outvoted
    voted, dist = bz.vote_pairdist(torch.from_numpy(rep).to(DEV), workspace=ws)
    assert np.array_equal(voted.cpu().numpy().view(np.uint32), g.view(np.uint32))
    _check_close(dist.cpu().numpy(), want)


def test_rounding_errors_lined_up_by_an_attacker():
    # Sec. 6.1's attacker knows the honest gradients.  Here it also knows the kernel: its row keeps every CTA's scale
    # for the row coarse (three values of 100 in every fourth 128-coordinate tile: too many to pass as outliers, too
    # frequent for the row to be moved to a finer scale) and places all its other values just short of half-way
    # between two fixed-point steps, on the side that makes each rounding error pull the distance to one honest row
    # the same way.  Independent rounding errors would cancel; lined up they add.  Whatever that does to the integer
    # kernel's sums, the bound it evaluates (Cauchy-Schwarz over the values it actually rounded) holds for this input
    # too: either it fits the tolerance and so does the result, or the binary64 kernel answers.
    f, d = 49, 11_200_000
    g = inputs.true_gradients(f, d, seed=12).numpy()
    b = g[7]
    step = 2.0 ** (8 - 30)                                   # |v| < 128 in a row's first step -> E = 8
    k = np.random.default_rng(1).integers(1, 2 ** 9, size=d).astype(np.float64)
    frac = np.where(b > 0, 15.0 / 32.0, 17.0 / 32.0)         # rounds down where b is above, up where b is below
    a = ((k + frac) * step).astype(np.float32)
    assert np.array_equal(a.astype(np.float64), (k + frac) * step)   # representable: the attack is exact
    for off in (0, 1, 2):
        a[off::4 * 128] = 100.0
    g[30] = a
    want = oracle.pairdist(g)
    ws = bz.alloc_workspace(bz.OP_PAIRDIST, 0, f, d)
    got = bz.pairdist(torch.from_numpy(g).to(DEV), workspace=ws).cpu().numpy()
    status = bz.pairdist_status(ws, f)
    _check_close(got, want)
    import os
    os.environ["BZ_PAIRDIST_PATH"] = "i8"
    try:
        forced = bz.pairdist(torch.from_numpy(g).to(DEV), workspace=ws).cpu().numpy()
    finally:
        del os.environ["BZ_PAIRDIST_PATH"]
    others = np.arange(f) != 30
    rel = np.abs(forced[30] - want[30])[others] / want[30][others]
    calm = np.abs(forced[0, 1:] - want[0, 1:]) / want[0, 1:]
    print("attacked row: relative error of the integer kernel %.3g (median over its pairs; pairs of an honest row: %.3g), "
          "status %d" % (float(np.median(rel)), float(np.median(calm[calm > 0])), status))
    assert status == bz.STATUS_RECOMPUTED or rel.max() <= DIST_TOL     # whenever it could have mattered, the guard fired
    assert rel.max() <= 1e-5                                           # and the unguarded result is still sane


@pytest.mark.parametrize("bad", [float("inf"), float("nan"), 3.0e38])
def test_values_without_a_fixed_point_scale(bad, monkeypatch):
    # the integer kernel marks them and the binary64 kernel's answer is what the caller gets
    v = inputs.true_gradients(25, 20_000, seed=9)
    v[4, 12_345] = bad
    ws = bz.alloc_workspace(bz.OP_PAIRDIST, 0, 25, 20_000)
    got = bz.pairdist(v.to(DEV), workspace=ws).cpu().numpy()
    assert bz.pairdist_status(ws, 25) == bz.STATUS_RECOMPUTED
    monkeypatch.setenv("BZ_PAIRDIST_PATH", "fp64")
    by_fp64 = bz.pairdist(v.to(DEV)).cpu().numpy()
    assert bz.last_path() == bz.PATH_FP64
    assert np.array_equal(got, by_fp64, equal_nan=True)
    want = oracle.pairdist(v.numpy())
    if bad == 3.0e38:
        assert (np.abs(got[4] - want[4])[np.arange(25) != 4] <= 1e-12 * want[4][np.arange(25) != 4]).all()
    if not np.isfinite(bad):
        assert np.array_equal(np.isnan(got), np.isnan(want)) and np.array_equal(np.isinf(got), np.isinf(want))
    clean = np.ones((25, 25), dtype=bool)
    clean[4, :] = clean[:, 4] = False
    clean &= ~np.eye(25, dtype=bool)
    assert (np.abs(got[clean] - want[clean]) <= DIST_TOL * want[clean]).all()


@pytest.mark.parametrize("l,r,q,attack,d", [(5, 3, 3, "reversed", 50004), (7, 3, 5, "alie", 100_000), (5, 5, 6, "constant", 40_000),
                                            (7, 5, 5, "alie", 20_000), (7, 7, 4, "reversed", 20_000)])
def test_vote_and_distances_in_one_pass(l, r, q, attack, d, monkeypatch):
    monkeypatch.setenv("BZ_PAIRDIST_PATH", "i8")
    rep, v = _voted(l, r, q, d, attack)
    voted, dist = bz.vote_pairdist(rep.to(DEV))
    assert np.array_equal(voted.cpu().numpy().view(np.uint32), v.numpy().view(np.uint32))
    _check_close(dist.cpu().numpy(), oracle.pairdist(v.numpy()))


def test_full_size_on_sampled_rows():
    # the benchmark's multi-Krum shape (r = 3, f = 49, d = 11.2 M) in the library's default configuration:
    # the oracle computes the distances among a sample of rows from copies of the same bytes
    l, r, q, d = 7, 3, 5, 11_200_000
    wf, fw, _ = oracle.assign(l, r)
    byz = oracle.worst_case(wf, l * l, r, q)[1]
    g = inputs.true_gradients(l * l, d, seed=0, device=DEV)
    rep = inputs.build_replicas(g, fw, byz, "alie")
    del g
    distorted = sorted({int(i) for i in range(l * l) if sum(int(w) in set(int(b) for b in byz) for w in fw[i]) >= 2})
    rows = sorted(set([0, 1, 17, 30, 48] + distorted[:2]))
    voted, dist = bz.vote_pairdist(rep)                      # vote in front of the integer kernel
    alone = bz.pairdist(voted)                               # the integer kernel on given rows
    torch.cuda.synchronize()
    sample = voted[rows].cpu().numpy()
    assert np.array_equal(sample.view(np.uint32), oracle.vote(rep[:, rows].cpu().numpy()).view(np.uint32))
    want = oracle.pairdist(sample)
    for got in (dist, alone):
        sub = got.cpu().numpy()[np.ix_(rows, rows)]
        _check_close(sub, want)
    # the two kernels fix a row's scale per step and their steps differ in size, so a few early tiles are
    # rounded on different grids: equal far below the tolerance, not bit for bit
    a, b = dist.cpu().numpy(), alone.cpu().numpy()
    assert np.array_equal(a == 0, b == 0)
    assert (np.abs(a - b) <= 1e-10 * np.maximum(a, b)).all()


def test_padded_rows_and_coordinate_slabs(monkeypatch):
    # rows with a leading dimension larger than d, and a coordinate slab of a larger allocation (the way
    # multi-GPU slabs and the 1e8-coordinate cells are passed): the kernel's conditions hold (16-byte
    # aligned start, ld a multiple of 4), so it runs; an unaligned slab takes the binary32 kernel
    monkeypatch.setenv("BZ_PAIRDIST_PATH", "i8")
    f, d_all = 49, 60_000
    g = inputs.true_gradients(f, d_all, seed=8)
    g[5] = -100.0 * g[5]
    buf = torch.zeros((f, d_all + 12), dtype=torch.float32, device=DEV)
    buf[:, :d_all] = g.to(DEV)
    for j0, d in [(0, 60_000), (4_000, 33_336), (8, 20_002)]:
        slab = buf[:, j0:j0 + d]
        want = oracle.pairdist(g[:, j0:j0 + d].contiguous().numpy())
        _check_close(bz.pairdist(slab).cpu().numpy(), want)
    # the same through the vote: replicas and voted rows as slabs of padded arrays
    r = 3
    rep_all = torch.zeros((r, f, d_all + 12), dtype=torch.float32, device=DEV)
    rep_all[:, :, :d_all] = g.to(DEV)[None]
    rep_all[0, 7, :d_all] = 3.0
    rep_all[1, 7, :d_all] = 3.0
    voted_all = torch.zeros((f, d_all + 12), dtype=torch.float32, device=DEV)
    j0, d = 4_000, 33_336
    voted, dist = bz.vote_pairdist(rep_all[:, :, j0:j0 + d], voted_all[:, j0:j0 + d])
    want_voted = oracle.vote(rep_all[:, :, j0:j0 + d].cpu().numpy())
    assert np.array_equal(voted.cpu().numpy().view(np.uint32), want_voted.view(np.uint32))
    assert (voted_all[:, :j0] == 0).all() and (voted_all[:, j0 + d:] == 0).all()      # nothing written outside the slab
    _check_close(dist.cpu().numpy(), oracle.pairdist(want_voted))
    monkeypatch.delenv("BZ_PAIRDIST_PATH")
    odd = buf[:, 1:50_001]                                                            # starts 4 bytes off a 16-byte boundary
    _check_close(bz.pairdist(odd).cpu().numpy(), oracle.pairdist(g[:, 1:50_001].contiguous().numpy()))
