"""GPU parity of the aggregation fused with the model update (Eq. 1, Algorithm 1's last step; momentum
of Sec. 6.1) against the oracle: the aggregate bit for bit, the updated state within the rounding of
the two single-precision multiply-adds."""
import numpy as np
import pytest
import torch

import oracle
from paper_2010_04902_b200 import binding as bz
from paper_2010_04902_b200 import inputs

pytestmark = pytest.mark.gpu

DEV = "cuda"
ETA, MU = 0.05, 0.9


def _bits(a):
    if isinstance(a, torch.Tensor):
        a = a.detach().cpu().numpy()
    return np.ascontiguousarray(a, np.float32).view(np.uint32)


def _close(got, want, slack):
    """|got - want| within two units in the last place of want plus `slack` (what one unit in the last
    place of the other operand contributes)."""
    got = got.cpu().numpy() if isinstance(got, torch.Tensor) else got
    tol = 2 * np.spacing(np.abs(want)) + slack
    return bool((np.abs(got.astype(np.float64) - want.astype(np.float64)) <= tol).all())


def _case(l, r, d, seed, attack="reversed", q=None):
    K, f = l * r, l * l
    wf, fw, _ = oracle.assign(l, r)
    q = q if q is not None else max(1, (K - 1) // 4)
    byz = [(i * K) // q for i in range(q)]
    g = inputs.true_gradients(f, d, seed=seed)
    return inputs.build_replicas(g, fw, byz, attack)


@pytest.mark.parametrize("l,r,d", [(5, 3, 200_003), (7, 3, 70_001), (5, 5, 66_000), (7, 7, 40_001), (3, 3, 5_000)])
def test_three_steps_with_momentum(l, r, d):
    rng = np.random.default_rng(d)
    w_ref = rng.standard_normal(d).astype(np.float32)
    v_ref = np.zeros(d, np.float32)
    w = torch.from_numpy(w_ref.copy()).to(DEV)
    v = torch.zeros(d, device=DEV)
    out = torch.empty(d, device=DEV)
    for step in range(3):
        rep = _case(l, r, d, seed=100 + step, attack=["reversed", "alie", "constant"][step])
        g_ref = oracle.vote_median(rep.numpy())
        bz.vote_median_update(rep.to(DEV), w, ETA, v, MU, out)
        assert np.array_equal(_bits(out), _bits(g_ref))
        w_ref, v_ref = oracle.model_update(w_ref, g_ref, ETA, v_ref, MU)
        # the two sides carry their own state: a last-place difference in v feeds eta * that into w
        slack_v = step * 2 * np.spacing(np.abs(v_ref))
        assert _close(v, v_ref, slack_v)
        assert _close(w, w_ref, (step + 1) * ETA * 2 * np.spacing(np.abs(v_ref)) + step * 2 * np.spacing(np.abs(w_ref)))
    rel = np.linalg.norm(w.cpu().numpy().astype(np.float64) - w_ref) / np.linalg.norm(w_ref)
    assert rel <= 1e-6


def test_plain_step_without_output():
    d = 150_000
    rep = _case(5, 3, d, seed=7)
    g_ref = oracle.vote_median(rep.numpy())
    w0 = np.linspace(-1, 1, d).astype(np.float32)
    w = torch.from_numpy(w0.copy()).to(DEV)
    bz.vote_median_update(rep.to(DEV), w, ETA)
    want, _ = oracle.model_update(w0, g_ref, ETA)
    assert _close(w, want, 0)
    # eta = 0 leaves the parameters bit for bit
    w2 = torch.from_numpy(w0.copy()).to(DEV)
    bz.vote_median_update(rep.to(DEV), w2, 0.0)
    assert np.array_equal(_bits(w2), _bits(w0))


def test_unaligned_views_and_small_inputs():
    # odd offsets take the scalar register path; d < 512 skips the staged path
    for d, off in [(30_001, 1), (300, 0), (5, 3)]:
        full = _case(5, 3, d + off, seed=d)
        rep_dev = full.to(DEV)[:, :, off:]
        g_ref = oracle.vote_median(np.ascontiguousarray(full[:, :, off:].numpy()))
        w0 = np.full(d, 0.5, np.float32)
        v0 = np.full(d, -0.25, np.float32)
        wbuf = torch.zeros(d + 8, device=DEV)
        vbuf = torch.zeros(d + 8, device=DEV)
        w, v = wbuf[1:1 + d], vbuf[3:3 + d]
        w.copy_(torch.from_numpy(w0))
        v.copy_(torch.from_numpy(v0))
        out = torch.empty(d, device=DEV)
        bz.vote_median_update(rep_dev, w, ETA, v, MU, out)
        assert np.array_equal(_bits(out), _bits(g_ref))
        w_ref, v_ref = oracle.model_update(w0, g_ref, ETA, v0, MU)
        assert _close(v, v_ref, 0) and _close(w, w_ref, ETA * 2 * np.spacing(np.abs(v_ref)))
        # nothing outside the views was touched
        assert float(wbuf[0]) == 0.0 and float(wbuf[1 + d:].abs().sum()) == 0.0
        assert float(vbuf[:3].abs().sum()) == 0.0 and float(vbuf[3 + d:].abs().sum()) == 0.0


def test_generic_shape_and_standalone_update():
    # f = 9 (l = 3) with r = 9 replicas has no specialised kernel
    d = 4_097
    g = inputs.true_gradients(9, d, seed=5)
    rep = g.unsqueeze(0).repeat(9, 1, 1).contiguous()
    rep[:4, 2] = -rep[:4, 2]                       # four of nine copies of file 2 are wrong: the vote repairs it
    g_ref = oracle.vote_median(rep.numpy())
    w0 = np.ones(d, np.float32)
    w = torch.ones(d, device=DEV)
    v = torch.zeros(d, device=DEV)
    bz.vote_median_update(rep.to(DEV), w, ETA, v, MU)
    w_ref, v_ref = oracle.model_update(w0, g_ref, ETA, np.zeros(d, np.float32), MU)
    assert _close(v, v_ref, 0) and _close(w, w_ref, ETA * 2 * np.spacing(np.abs(v_ref)))
    # the standalone update on an aggregate already in memory (a Multi-Krum output here)
    voted = oracle.vote(rep.numpy())
    agg, _, _ = oracle.multikrum(voted, 1, 7)
    agg32 = agg.astype(np.float32)
    w2 = torch.ones(d, device=DEV)
    v2 = torch.full((d,), 0.125, device=DEV)
    bz.model_update(torch.from_numpy(agg32).to(DEV), w2, ETA, v2, MU)
    w_ref2, v_ref2 = oracle.model_update(w0, agg32, ETA, np.full(d, 0.125, np.float32), MU)
    assert _close(v2, v_ref2, 0) and _close(w2, w_ref2, ETA * 2 * np.spacing(np.abs(v_ref2)))


def test_argument_errors_and_empty_input():
    rep = torch.zeros((3, 25, 16), device=DEV)
    st = bz.lib().bz_vote_median_update(rep.data_ptr(), 3, 25, 16, 16, 400, None, None, 0.1, 0.0, None, None)
    assert st == bz.ERR_INVALID_ARG
    w = torch.ones(0, device=DEV)
    bz.vote_median_update(torch.zeros((3, 25, 0), device=DEV), w, 0.1)
    with pytest.raises(TypeError):
        bz.vote_median_update(rep, torch.ones(15, device=DEV), 0.1)
