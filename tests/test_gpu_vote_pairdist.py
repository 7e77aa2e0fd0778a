"""GPU parity of the single-pass vote + pairwise distances (Eq. 3 feeding the Krum family of Sec. 1.2)
and of Multi-Krum / Bulyan run from the replicas: voted rows and selections bit for bit, distances and
averaged outputs within the tolerances of the two-call path."""
import numpy as np
import pytest
import torch

import oracle
from paper_2010_04902_b200 import binding as bz
from paper_2010_04902_b200 import inputs

pytestmark = pytest.mark.gpu

DEV = "cuda"


def _bits(a):
    if isinstance(a, torch.Tensor):
        a = a.detach().cpu().numpy()
    return np.ascontiguousarray(a, np.float32).view(np.uint32)


def _case(l, r, d, seed, attack, q=None):
    K, f = l * r, l * l
    _, fw, _ = oracle.assign(l, r)
    q = q if q is not None else max(1, (K - 1) // 3)
    byz = [(i * K) // q for i in range(q)]
    g = inputs.true_gradients(f, d, seed=seed)
    return inputs.build_replicas(g, fw, byz, attack), fw, byz


def _dist_close(D, want, tol=1e-7):
    D = D.cpu().numpy()
    nz = want > 0
    return bool((np.abs(D[nz] - want[nz]) <= tol * want[nz]).all()) and bool((D[~nz] == 0).all())


@pytest.mark.parametrize("l,r,d,attack", [(5, 3, 100_003, "reversed"), (5, 3, 1_048_576, "alie"), (7, 3, 50_001, "alie"),
                                          (5, 5, 70_000, "constant"), (7, 5, 30_011, "reversed"), (7, 7, 20_002, "alie")])
def test_voted_rows_and_distances(l, r, d, attack):
    rep, _, _ = _case(l, r, d, seed=d % 97, attack=attack)
    want_voted = oracle.vote(rep.numpy())
    want_D = oracle.pairdist(want_voted)
    voted, D = bz.vote_pairdist(rep.to(DEV))
    assert np.array_equal(_bits(voted), _bits(want_voted))
    assert _dist_close(D, want_D)
    assert np.array_equal(D.cpu().numpy(), D.cpu().numpy().T)
    # the two-call path sums the same terms; it may group them differently across CTAs
    D2 = bz.pairdist(bz.vote(rep.to(DEV)))
    assert np.allclose(D.cpu().numpy(), D2.cpu().numpy(), rtol=2e-7, atol=0)


@pytest.mark.parametrize("l,r,d,attack", [(5, 3, 100_004, "reversed"), (7, 3, 50_000, "alie"), (5, 5, 70_000, "constant"),
                                          (7, 5, 30_012, "reversed"), (7, 7, 20_000, "alie"), (5, 3, 2_000_000, "alie")])
def test_binary32_single_pass_on_every_compiled_shape(l, r, d, attack, monkeypatch):
    # BZ_PAIRDIST_PATH=fp32 puts the vote in front of the binary32 distance kernel (the default is the integer one)
    monkeypatch.setenv("BZ_PAIRDIST_PATH", "fp32")
    rep, _, _ = _case(l, r, d, seed=d % 89, attack=attack)
    want_voted = oracle.vote(rep.numpy())
    want_D = oracle.pairdist(want_voted)
    ws = bz.alloc_workspace(bz.OP_PAIRDIST, 0, l * l, d)
    voted, D = bz.vote_pairdist(rep.to(DEV), workspace=ws)
    assert bz.last_path() == bz.PATH_FP32_FUSED
    assert bz.pairdist_status(ws, l * l) == 0
    assert np.array_equal(_bits(voted), _bits(want_voted))
    assert _dist_close(D, want_D)
    assert np.array_equal(D.cpu().numpy(), D.cpu().numpy().T) and (np.diag(D.cpu().numpy()) == 0).all()
    monkeypatch.delenv("BZ_PAIRDIST_PATH")
    voted, D = bz.vote_pairdist(rep.to(DEV), workspace=ws)
    assert bz.last_path() == bz.PATH_TENSOR
    assert np.array_equal(_bits(voted), _bits(want_voted)) and _dist_close(D, want_D)


def test_two_calls_in_a_row_agree_bit_for_bit():
    rep, _, _ = _case(5, 3, 300_000, seed=1, attack="alie")
    rep_dev = rep.to(DEV)
    ws = bz.alloc_workspace(bz.OP_PAIRDIST, 0, 25, 300_000)
    v1, D1 = bz.vote_pairdist(rep_dev, workspace=ws)
    D1 = D1.clone()
    v2, D2 = bz.vote_pairdist(rep_dev, workspace=ws)
    assert torch.equal(D1, D2) and torch.equal(v1, v2)


def test_shapes_without_a_fused_kernel():
    # odd offsets (unaligned rows), a short array, a shape with no specialisation: the two-call path answers
    full, _, _ = _case(5, 3, 20_001, seed=2, attack="reversed")
    rep_dev = full.to(DEV)[:, :, 1:]
    want_voted = oracle.vote(np.ascontiguousarray(full[:, :, 1:].numpy()))
    voted, D = bz.vote_pairdist(rep_dev)
    assert np.array_equal(_bits(voted), _bits(want_voted)) and _dist_close(D, oracle.pairdist(want_voted))
    for l, r, d in [(5, 3, 300), (3, 3, 4_000)]:
        rep, _, _ = _case(l, r, d, seed=3, attack="constant", q=2)
        want_voted = oracle.vote(rep.numpy())
        voted, D = bz.vote_pairdist(rep.to(DEV))
        # a few hundred binary32 terms per sum: their rounding is not averaged out over many blocks
        assert np.array_equal(_bits(voted), _bits(want_voted)) and _dist_close(D, oracle.pairdist(want_voted), 2e-6)
    # a padded destination (ld_voted > d) on the fused path
    rep, _, _ = _case(5, 3, 10_000, seed=4, attack="alie")
    buf = torch.full((25, 10_240), 7.0, device=DEV)
    voted, D = bz.vote_pairdist(rep.to(DEV), voted=buf[:, :10_000])
    assert np.array_equal(_bits(voted), _bits(oracle.vote(rep.numpy())))
    assert float((buf[:, 10_000:] - 7.0).abs().sum()) == 0.0


@pytest.mark.parametrize("l,r,d", [(5, 3, 120_001), (7, 3, 60_000), (5, 5, 40_003)])
def test_multikrum_and_bulyan_from_the_replicas(l, r, d):
    rep, fw, byz = _case(l, r, d, seed=11, attack="alie")
    f = l * l
    c = oracle.count_distorted(fw, np.array(byz, np.int32))
    want_voted = oracle.vote(rep.numpy())
    rep_dev = rep.to(DEV)
    if f >= 2 * c + 3:
        m = f - c
        want_out, want_sel, _ = oracle.multikrum(want_voted, c, m)
        out, sel, voted = bz.vote_multikrum(rep_dev, c, m)
        assert np.array_equal(_bits(voted), _bits(want_voted))
        assert sel.cpu().tolist() == want_sel.tolist()
        assert np.linalg.norm(out.cpu().numpy().astype(np.float64) - want_out) <= 1e-5 * np.linalg.norm(want_out)
    cb = min(c, (f - 3) // 4)
    want_out, want_sel, _ = oracle.bulyan(want_voted, cb)
    out, sel, voted = bz.vote_bulyan(rep_dev, cb)
    assert np.array_equal(_bits(voted), _bits(want_voted))
    assert sel.cpu().tolist() == want_sel.tolist()
    assert np.linalg.norm(out.cpu().numpy().astype(np.float64) - want_out) <= 1e-5 * np.linalg.norm(want_out)


def test_argument_errors():
    rep = torch.zeros((3, 25, 1024), device=DEV)
    with pytest.raises(bz.BzError) as e:
        bz.vote_pairdist(rep, workspace=torch.empty(256, dtype=torch.uint8, device=DEV))
    assert e.value.status == bz.ERR_WORKSPACE
    with pytest.raises(bz.BzError) as e:
        bz.vote_multikrum(rep, 12, 5)
    assert e.value.status == bz.ERR_PRECONDITION
    with pytest.raises(bz.BzError) as e:
        bz.vote_bulyan(rep, 6)
    assert e.value.status == bz.ERR_PRECONDITION
    ws = bz.alloc_workspace(bz.OP_PAIRDIST, 0, 25, 1024)
    D = torch.empty((25, 25), dtype=torch.float64, device=DEV)
    voted = torch.empty((25, 1024), device=DEV)
    st = bz.lib().bz_vote_pairdist(rep.data_ptr(), 4, 25, 1024, 1024, 25 * 1024, voted.data_ptr(), 1024, D.data_ptr(),
                                   ws.data_ptr(), ws.numel(), None)
    assert st == bz.ERR_INVALID_ARG        # even replication
