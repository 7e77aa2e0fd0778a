"""GPU parity on the sweep cells: every feasible (l, r) of l in {5, 7}, r in {3, 5, 7}, several numbers
of Byzantine workers, d = 1 M (full comparison) and one 100 M-coordinate case (sampled columns, exercises
indices beyond 2^32 elements)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2010_04902_b200 import binding as bz
from paper_2010_04902_b200 import inputs

pytestmark = pytest.mark.gpu

DEV = "cuda"
CELLS = [(5, 3), (5, 5), (7, 3), (7, 5), (7, 7)]       # (5, 7) is infeasible: r > l


def _bits(a):
    if isinstance(a, torch.Tensor):
        a = a.detach().cpu().numpy()
    return np.ascontiguousarray(a, np.float32).view(np.uint32)


def _spread_workers(K, q):
    """q distinct workers spread over the classes (a fixed, assignment-independent choice)."""
    return [(i * K) // q for i in range(q)]


def test_infeasible_cell_is_refused():
    with pytest.raises(bz.BzError) as e:
        bz.assign_mols(5, 7)
    assert e.value.status == bz.ERR_INVALID_ARG


@pytest.mark.parametrize("l,r", CELLS)
@pytest.mark.parametrize("qsel", ["one", "mid", "max"])
def test_vote_median_and_multikrum_at_1m(l, r, qsel):
    K, f, d = l * r, l * l, 1_000_000
    qmax = (K - 1) // 2
    q = {"one": 1, "mid": max(1, qmax // 2), "max": qmax}[qsel]
    _, fw, _ = oracle.assign(l, r)
    byz = _spread_workers(K, q)
    g = inputs.true_gradients(f, d, seed=l * 10 + r)
    rep = inputs.build_replicas(g, fw, byz, "alie" if qsel != "max" else "reversed")
    rep_dev = rep.to(DEV)
    want_voted = oracle.vote(rep.numpy())
    want_med = oracle.median(want_voted)
    assert np.array_equal(_bits(bz.vote_median(rep_dev)), _bits(want_med))
    voted = bz.vote(rep_dev)
    assert np.array_equal(_bits(voted), _bits(want_voted))
    c = oracle.count_distorted(fw, np.array(byz, np.int32))
    if f >= 2 * c + 3:
        m = f - c
        want_out, want_sel, want_D = oracle.multikrum(want_voted, c, m)
        out, sel, D = bz.multikrum(voted, c, m, want_dist=True)
        assert sel.cpu().tolist() == want_sel.tolist()
        got = out.cpu().numpy().astype(np.float64)
        assert np.linalg.norm(got - want_out) <= 1e-5 * np.linalg.norm(want_out)
        Dg = D.cpu().numpy()
        nz = want_D > 0
        assert (np.abs(Dg[nz] - want_D[nz]) <= 1e-7 * want_D[nz]).all()
    else:
        with pytest.raises(bz.BzError) as e:
            bz.multikrum(voted, c, max(1, f - c))
        assert e.value.status == bz.ERR_PRECONDITION


def test_ramanujan_clusters():
    from conftest import read_golden_rows
    # Case 1, (m, s) = (3, 5): the printed (15,25,5,3) table holds for this graph too (Sec. 5.3.2)
    wf, fw, mask = bz.assign_ramanujan(3, 5)
    for K, f, l, r, q, cmax, _ in read_golden_rows("cmax_tables.txt"):
        if (K, f, l, r) == ("15", "25", "5", "3"):
            got, arg, _ = bz.worst_case(mask, 25, 3, int(q))
            assert got == int(cmax) and oracle.count_distorted(fw, arg) == int(cmax)
            want, warg, _ = oracle.worst_case(oracle.assign_ramanujan(3, 5)[0], 25, 3, int(q))
            assert arg.tolist() == warg.tolist()
    # Case 2 with m > s, (m, s) = (10, 5): K = 25 workers, f = 50 files (even: two middle values), r = 5
    wf, fw, mask = bz.assign_ramanujan(10, 5)
    cmax, byz, _ = bz.worst_case(mask, 50, 5, 6)
    ocmax, obyz, _ = oracle.worst_case(oracle.assign_ramanujan(10, 5)[0], 50, 5, 6)
    assert (cmax, byz.tolist()) == (ocmax, obyz.tolist())
    g = inputs.true_gradients(50, 30_001, seed=3)
    rep = inputs.build_replicas(g, fw, byz, "constant")
    want_voted = oracle.vote(rep.numpy())
    assert np.array_equal(_bits(bz.vote(rep.to(DEV))), _bits(want_voted))
    assert np.array_equal(_bits(bz.vote_median(rep.to(DEV))), _bits(oracle.median(want_voted)))
    out, sel = bz.multikrum(torch.from_numpy(want_voted).to(DEV), cmax, 50 - cmax)
    want_out, want_sel, _ = oracle.multikrum(want_voted, cmax, 50 - cmax)
    assert sel.cpu().tolist() == want_sel.tolist()
    assert np.linalg.norm(out.cpu().numpy().astype(np.float64) - want_out) <= 1e-5 * np.linalg.norm(want_out)


@pytest.mark.parametrize("l,r,q", [(4, 3, 3), (8, 3, 4), (8, 5, 5)])
def test_prime_power_clusters(l, r, q):
    # squares over the field F_l (Sec. 4.1.1): f = 16 and f = 64 files
    K, f, d = l * r, l * l, 20_001
    wf, fw, mask = bz.assign_mols(l, r)
    owf, ofw, _ = oracle.assign(l, r)
    assert np.array_equal(wf, owf) and np.array_equal(fw, ofw)
    cmax, byz, n = bz.worst_case(mask, f, r, q)
    ocmax, obyz, on = oracle.worst_case(owf, f, r, q)
    assert (cmax, n, byz.tolist()) == (ocmax, on, obyz.tolist())
    g = inputs.true_gradients(f, d, seed=l)
    rep = inputs.build_replicas(g, fw, byz, "alie")
    want_voted = oracle.vote(rep.numpy())
    assert sum(not np.array_equal(_bits(want_voted[i]), _bits(g[i])) for i in range(f)) == cmax   # Sec. 2 / Sec. 5.3.2
    assert np.array_equal(_bits(bz.vote(rep.to(DEV))), _bits(want_voted))
    assert np.array_equal(_bits(bz.vote_median(rep.to(DEV))), _bits(oracle.median(want_voted)))   # even f: two middle values
    voted, win = bz.vote_vectorwise(rep.to(DEV))
    assert np.array_equal(_bits(voted), _bits(want_voted)) and win.cpu().tolist() == oracle.vote_vectorwise(rep.numpy()).tolist()
    c = cmax
    out, sel = bz.multikrum(torch.from_numpy(want_voted).to(DEV), c, f - c)
    want_out, want_sel, _ = oracle.multikrum(want_voted, c, f - c)
    assert sel.cpu().tolist() == want_sel.tolist()
    assert np.linalg.norm(out.cpu().numpy().astype(np.float64) - want_out) <= 1e-5 * np.linalg.norm(want_out)


def test_hundred_million_coordinates():
    # (l, r) = (5, 3), d = 1e8: 30 GB of replicas, 7.5e9 elements - offsets need 64 bits
    l, r, q, d = 5, 3, 3, 100_000_000
    wf, fw, _ = oracle.assign(l, r)
    byz = oracle.worst_case(wf, l * l, r, q)[1]
    g = inputs.true_gradients(l * l, d, seed=0, device=DEV)
    rep = inputs.build_replicas(g, fw, byz, "reversed")
    del g
    out = bz.vote_median(rep)
    torch.cuda.synchronize()
    rng = np.random.default_rng(1)
    idx = np.unique(np.concatenate([np.arange(0, 300), np.arange(d - 300, d), rng.integers(0, d, size=20000),
                                    np.arange(2 ** 26 - 64, 2 ** 26 + 64)]))
    idx_dev = torch.from_numpy(idx).to(DEV)
    want = oracle.vote_median(rep[:, :, idx_dev].cpu().numpy())
    assert np.array_equal(_bits(out[idx_dev]), _bits(want))
    # the last file of the last class sits beyond 2^32 elements: check the vote on a slab of it
    slab = slice(d - 4096, d)
    voted_tail = bz.vote(rep[:, :, slab])
    assert np.array_equal(_bits(voted_tail), _bits(oracle.vote(rep[:, :, slab].cpu().numpy())))
    del rep, out
    torch.cuda.empty_cache()
