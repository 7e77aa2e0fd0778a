"""GPU parity of the Krum family against the CPU oracle: distances, selection indices (bit-exact),
means (relative L2 <= 1e-5, the tolerance for averaged outputs in binary32)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2010_04902_b200 import binding as bz
from paper_2010_04902_b200 import inputs

pytestmark = pytest.mark.gpu

DEV = "cuda"
MEAN_TOL = 1e-5      # relative L2 of averaged outputs
DIST_TOL = 1e-7      # relative error of a squared distance (binary32 products, binary64 sums)


def _rel_l2(got, want):
    got = np.asarray(got, np.float64)
    want = np.asarray(want, np.float64)
    den = np.linalg.norm(want)
    return np.linalg.norm(got - want) / (den if den > 0 else 1.0)


def _voted(l, r, q, d, attack, seed=0, heavy=0.0):
    wf, fw, _ = oracle.assign(l, r)
    byz = oracle.worst_case(wf, l * l, r, q)[1]
    g = inputs.true_gradients(l * l, d, seed=seed, heavy_tail_frac=heavy)
    rep = inputs.build_replicas(g, fw, byz, attack)
    return torch.from_numpy(oracle.vote(rep.numpy()))


@pytest.mark.parametrize("f,d", [(25, 1), (25, 255), (25, 4097), (49, 3), (49, 1000), (49, 70001), (9, 513), (121, 300)])
def test_pairdist_exact_on_integer_rows(f, d):
    v = inputs.integer_gradients(f, d, seed=f + d)
    want = oracle.pairdist(v.numpy())
    got = bz.pairdist(v.to(DEV)).cpu().numpy()
    assert np.array_equal(got, want)


@pytest.mark.parametrize("l,r,q,attack,d", [(5, 3, 3, "reversed", 50001), (7, 3, 5, "alie", 50001),
                                            (5, 5, 6, "constant", 20000), (3, 3, 2, "alie", 999)])
def test_pairdist_close_on_gradients(l, r, q, attack, d):
    v = _voted(l, r, q, d, attack)
    want = oracle.pairdist(v.numpy())
    got = bz.pairdist(v.to(DEV)).cpu().numpy()
    assert np.array_equal(got, got.T) and (np.diag(got) == 0).all()
    off = ~np.eye(v.shape[0], dtype=bool)
    nz = off & (want > 0)
    assert (np.abs(got[nz] - want[nz]) <= DIST_TOL * want[nz]).all()
    assert (got[off & (want == 0)] == 0).all()     # identical (colluding) rows
    # twice the same call: fixed summation order
    assert np.array_equal(bz.pairdist(v.to(DEV)).cpu().numpy(), got)


@pytest.mark.parametrize("f,d", [(25, 4), (25, 1000), (49, 5000), (25, 300_000), (49, 200_004)])
def test_binary64_kernel_matches_the_oracle_to_the_last_digits(f, d, monkeypatch):
    # differences, squares and sums in double precision: only the order of the additions differs from the oracle's
    monkeypatch.setenv("BZ_PAIRDIST_PATH", "fp64")
    g = inputs.true_gradients(f, d, seed=f * d % 1000).numpy()
    g[1, ::7] *= 1.0e4
    g[f - 1] = g[0]
    want = oracle.pairdist(g)
    got = bz.pairdist(torch.from_numpy(g).to(DEV)).cpu().numpy()
    assert bz.last_path() == bz.PATH_FP64
    assert np.array_equal(got, got.T) and (np.diag(got) == 0).all() and got[0, f - 1] == 0
    nz = want > 0
    assert (np.abs(got[nz] - want[nz]) <= 1e-12 * want[nz]).all()
    assert np.array_equal(bz.pairdist(torch.from_numpy(g).to(DEV)).cpu().numpy(), got)
    # rows too short for the integer kernel take it by default
    if d < 8192:
        monkeypatch.delenv("BZ_PAIRDIST_PATH")
        assert np.array_equal(bz.pairdist(torch.from_numpy(g).to(DEV)).cpu().numpy(), got)
        assert bz.last_path() == bz.PATH_FP64


def test_pairdist_unaligned_rows():
    v = inputs.integer_gradients(25, 1003, seed=2)
    buf = torch.zeros((25, 1100), dtype=torch.float32, device=DEV)
    buf[:, 1:1004] = v.to(DEV)
    assert np.array_equal(bz.pairdist(buf[:, 1:1004]).cpu().numpy(), oracle.pairdist(v.numpy()))
    buf[:, 4:1007] = v.to(DEV)
    assert np.array_equal(bz.pairdist(buf[:, 4:1007]).cpu().numpy(), oracle.pairdist(v.numpy()))


@pytest.mark.parametrize("f", [25, 49])
@pytest.mark.parametrize("d,shift", [(150_002, 0), (150_001, 0), (150_003, 1), (150_000, 2), (150_000, 3), (1003, 1)])
@pytest.mark.parametrize("path", ["", "fp32"])
def test_pairdist_rows_on_8_and_4_byte_boundaries(f, d, shift, path, monkeypatch):
    # contiguous rows of a length that is not a multiple of 4 (every other row starts 8 or 4 bytes off a 16-byte
    # boundary) and rows shifted inside a buffer: the tiled kernels stage them with 8- or 4-byte copies.  By default the
    # binary64 kernel answers (the integer kernel needs 16-byte aligned rows); BZ_PAIRDIST_PATH=fp32 takes the binary32 one.
    if path:
        monkeypatch.setenv("BZ_PAIRDIST_PATH", path)
    g = inputs.true_gradients(f, d, seed=f + d % 100)
    g[f - 1] = g[2]
    buf = torch.zeros(f * d + 8, dtype=torch.float32, device=DEV)
    rows = buf[shift: shift + f * d].view(f, d)
    rows.copy_(g)
    want = oracle.pairdist(g.numpy())
    got = bz.pairdist(rows).cpu().numpy()
    assert bz.last_path() == (bz.PATH_FP32 if path else bz.PATH_FP64)
    assert np.array_equal(got, got.T) and (np.diag(got) == 0).all() and got[2, f - 1] == 0
    nz = want > 0
    tol = 1e-7 if path else 1e-12
    assert (np.abs(got[nz] - want[nz]) <= tol * want[nz]).all()


def test_krum_hand_cases_on_device():
    v = torch.tensor([[0.0], [1.0], [2.0], [3.0], [10.0]])
    D = bz.pairdist(v.to(DEV))
    assert bz.krum_select(D, 1, 1).cpu().tolist() == [1]
    assert bz.krum_select(D, 1, 3).cpu().tolist() == [1, 2, 0]
    out, sel = bz.multikrum(v.to(DEV), 1, 4)
    assert sel.cpu().tolist() == [1, 2, 0, 3] and float(out[0]) == 1.5
    v7 = torch.tensor([[0.0], [1.0], [2.0], [3.0], [4.0], [5.0], [100.0]])
    assert bz.bulyan_select(bz.pairdist(v7.to(DEV)), 1).cpu().tolist() == [2, 3, 1, 4, 0]
    out, sel = bz.bulyan(v7.to(DEV), 1)
    assert float(out[0]) == 2.0


@pytest.mark.parametrize("l,r,q,attack,d,c,m", [
    (7, 3, 5, "alie", 30011, 5, 44),        # benchmark parameters of the multi-Krum configuration
    (7, 3, 5, "alie", 30011, 8, 41),        # the paper's reading: c = c_max = 8 distorted files
    (5, 3, 3, "reversed", 12345, 3, 22),
    (5, 5, 6, "constant", 8000, 4, 1),      # Krum
    (3, 3, 2, "reversed", 777, 1, 5),       # generic (f = 9) path
])
def test_multikrum_parity(l, r, q, attack, d, c, m):
    v = _voted(l, r, q, d, attack)
    want_out, want_sel, want_D = oracle.multikrum(v.numpy(), c, m)
    out, sel, D = bz.multikrum(v.to(DEV), c, m, want_dist=True)
    assert sel.cpu().tolist() == want_sel.tolist()
    assert _rel_l2(out.cpu().numpy(), want_out) <= MEAN_TOL
    # stage by stage through the separate entry points
    sel2 = bz.krum_select(torch.from_numpy(want_D).to(DEV), c, m)
    assert sel2.cpu().tolist() == want_sel.tolist()
    out2 = bz.mean_rows(v.to(DEV), sel2)
    assert np.array_equal(out2.cpu().numpy(), want_out)        # same binary64 sums, same order


def test_multikrum_c0_is_plain_mean():
    v = inputs.true_gradients(25, 5001, seed=6)
    out, sel = bz.multikrum(v.to(DEV), 0, 25)
    assert sorted(sel.cpu().tolist()) == list(range(25))
    assert _rel_l2(out.cpu().numpy(), v.double().mean(0).numpy()) <= MEAN_TOL


@pytest.mark.parametrize("l,r,q,attack,d,c,heavy", [
    (5, 5, 6, "constant", 30011, 4, 0.01),   # benchmark parameters of the Bulyan configuration
    (7, 3, 5, "alie", 9001, 8, 0.0),
    (7, 3, 3, "reversed", 4000, 11, 0.0),    # largest c for f = 49: theta = 27, beta = 5
    (5, 3, 2, "alie", 4000, 0, 0.0),         # c = 0: theta = beta = f
    (3, 3, 2, "reversed", 600, 1, 0.0),      # generic (f = 9) path, theta = 7
])
def test_bulyan_parity(l, r, q, attack, d, c, heavy):
    v = _voted(l, r, q, d, attack, heavy=heavy)
    want_out, want_sel, want_D = oracle.bulyan(v.numpy(), c)
    out, sel = bz.bulyan(v.to(DEV), c)
    assert sel.cpu().tolist() == want_sel.tolist()
    assert _rel_l2(out.cpu().numpy(), want_out) <= MEAN_TOL
    sel2 = bz.bulyan_select(torch.from_numpy(want_D).to(DEV), c)
    assert sel2.cpu().tolist() == want_sel.tolist()


@pytest.mark.parametrize("theta,beta", [(5, 3), (7, 5), (9, 9), (9, 1), (15, 5), (17, 9), (19, 13), (23, 21), (25, 25),
                                        (27, 5), (29, 9), (37, 25), (47, 45), (49, 49),          # register kernels
                                        (7, 1), (25, 17), (49, 1), (8, 3), (12, 12), (11, 5), (13, 7)])  # generic
def test_trimmed_mean_parity(theta, beta):
    # (theta, beta) pairs with a register kernel and pairs that take the generic one; many duplicates and ties
    rng = np.random.default_rng(theta * 64 + beta)
    f = max(theta, 25)
    v = rng.standard_normal((f, 2049)).astype(np.float32)
    v[:, :512] = np.round(v[:, :512] * 2) / 2
    sel = rng.permutation(f)[:theta].astype(np.int32)
    want = oracle.trimmed_mean(v, sel, beta)
    got = bz.trimmed_mean(torch.from_numpy(v).to(DEV), torch.from_numpy(sel).to(DEV), beta)
    assert np.array_equal(got.cpu().numpy(), want)


@pytest.mark.parametrize("theta,beta", [(17, 9), (23, 21), (39, 29), (49, 49)])
@pytest.mark.parametrize("d,ld,shift,out_shift", [
    (4100, 4100, 0, 0),   # 16-byte aligned rows: four coordinates per thread for theta <= 25
    (4099, 4100, 0, 0),   # ... with three coordinates left for the last group
    (4098, 4098, 0, 0),   # 8-byte aligned rows: two coordinates per thread
    (4097, 4100, 0, 0),   # odd d in even rows: the last group holds one coordinate
    (4097, 4100, 1, 0),   # rows start 4 bytes off: one coordinate per thread
    (4098, 4100, 0, 1),   # output 4 bytes off
    (4098, 4100, 2, 2),   # rows and output 8 bytes off
    (1, 2, 0, 0), (2, 2, 0, 0), (3, 4, 0, 0),
])
def test_trimmed_mean_layouts(theta, beta, d, ld, shift, out_shift):
    rng = np.random.default_rng(theta * 1000 + d + shift)
    f = 49
    v = rng.standard_normal((f, d)).astype(np.float32)
    v[:, : d // 3] = np.round(v[:, : d // 3] * 2) / 2
    sel = rng.permutation(f)[:theta].astype(np.int32)
    want = oracle.trimmed_mean(v, sel, beta)
    buf = torch.full((f * ld + 8,), float("nan"), dtype=torch.float32, device=DEV)
    rows = buf[shift: shift + f * ld].view(f, ld)[:, :d]
    rows.copy_(torch.from_numpy(v))
    out_buf = torch.full((d + 4,), -7.0, dtype=torch.float32, device=DEV)
    out = out_buf[out_shift: out_shift + d]
    bz.trimmed_mean(rows, torch.from_numpy(sel).to(DEV), beta, out=out)
    assert np.array_equal(out.cpu().numpy(), want)
    assert (out_buf[:out_shift] == -7.0).all() and (out_buf[out_shift + d:] == -7.0).all()


@pytest.mark.parametrize("theta,beta", [(17, 9), (15, 5), (23, 21), (39, 29), (11, 5)])
def test_trimmed_mean_with_infinities_and_nans(theta, beta):
    # Columns holding +-inf or NaN: distances to the median can be NaN, and the window then follows the stepwise
    # rule (a false comparison takes the upper neighbour).  NaN results compare equal whatever their payload.
    rng = np.random.default_rng(theta * 7 + beta)
    f, d = max(theta, 25), 4096
    v = rng.standard_normal((f, d)).astype(np.float32)
    specials = np.array([np.inf, -np.inf, np.nan, -np.nan, 3.0e38, -3.0e38], dtype=np.float32)
    for j in range(0, d, 2):                       # every other column: 1 .. theta special values
        n = 1 + (j // 2) % theta
        rows = rng.permutation(f)[:n]
        v[rows, j] = specials[rng.integers(0, len(specials), n)]
    v[:, 1::64] = np.inf                            # whole columns of one infinity
    sel = rng.permutation(f)[:theta].astype(np.int32)
    want = oracle.trimmed_mean(v, sel, beta)
    got = bz.trimmed_mean(torch.from_numpy(v).to(DEV), torch.from_numpy(sel).to(DEV), beta).cpu().numpy()
    assert np.array_equal(np.isnan(got), np.isnan(want))
    ok = ~np.isnan(want)
    assert np.array_equal(got[ok].view(np.uint32), want[ok].view(np.uint32))
    assert (~np.isfinite(v[sel])).any(axis=0).sum() > 1000 and np.isinf(want).sum() > 10   # the stepwise path ran


def test_preconditions_reported():
    v = torch.zeros((25, 16), dtype=torch.float32, device=DEV)
    with pytest.raises(bz.BzError) as e:
        bz.bulyan(v, 6)          # 4*6+3 > 25: the case the paper calls inapplicable
    assert e.value.status == bz.ERR_PRECONDITION
    with pytest.raises(bz.BzError) as e:
        bz.multikrum(v, 12, 1)   # 2*12+3 > 25
    assert e.value.status == bz.ERR_PRECONDITION
