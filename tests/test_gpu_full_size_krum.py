"""The Krum-family configurations at their configured size, end to end against the CPU oracle on ALL rows:
K = 21, (l, r) = (7, 3), f = 49, d = 11.2 M, q = 5 workers with the ALIE payload, Multi-Krum with
(c, m) = (5, 44) and with the paper's operand count (8, 41) (Sec. 6.1: c counts corrupted operands,
c_max^(5) = 8 in the appendix table); and K = 25, (l, r) = (5, 5), f = 25, d = 25 M with 1 % heavy-tailed
coordinates, q = 6 workers sending a constant, Bulyan with c = c_max^(6) = 4.

Bars: voted rows and selection indices bit-exact, every distance within 1e-7 relative, averaged outputs
within 1e-5 relative L2 (trimmed mean bit-exact).  Each test also reports the oracle's smallest relative
score gap at every selection boundary beside the GPU's largest relative distance error - the index parity
holds because the second is orders of magnitude below the first - and, when the environment variable
BZ_REPORT_DIR names a folder, writes the figures to krum_full_size_report.json there.

Also here: run-to-run determinism of every shipped instance of the integer distance kernel at full size, and
the repair path after bounded waits that ran out.
"""
import json
import os

import numpy as np
import pytest
import torch

import oracle
from conftest import ROOT
from paper_2010_04902_b200 import binding as bz
from paper_2010_04902_b200 import inputs

pytestmark = pytest.mark.gpu

DEV = "cuda"
DIST_TOL = 1e-7
MEAN_TOL = 1e-5
# The integer kernel's only error is the rounding of a value to its row's fixed-point grid; on these gradients
# that is ~1e-11 relative.  A wrong power-of-two scale on even one 128-coordinate tile would show at ~1e-5/d*128
# and above, so the full-size tests also hold the kernel to this sharper figure.
I8_SHARP = 2e-9


def _report(name, rec):
    print(name, json.dumps(rec))
    out_dir = os.environ.get("BZ_REPORT_DIR", "")
    if not out_dir:
        return
    try:
        os.makedirs(out_dir, exist_ok=True)
        path = os.path.join(out_dir, "krum_full_size_report.json")
        data = {}
        if os.path.exists(path):
            with open(path) as fh:
                data = json.load(fh)
        data[name] = rec
        with open(path, "w") as fh:
            json.dump(data, fh, indent=1, sort_keys=True)
    except OSError:
        pass


def _cluster(l, r, q, d, attack, heavy=0.0):
    wf, fw, _ = oracle.assign(l, r)
    byz = oracle.worst_case(wf, l * l, r, q)[1]
    g = inputs.true_gradients(l * l, d, seed=0, heavy_tail_frac=heavy, device=DEV)
    rep = inputs.build_replicas(g, fw, byz, attack)
    del g
    return rep


def _oracle_vote_by_files(rep, step=7):
    """Eq. (3) on the CPU, a few files at a time (the vote is independent per file; this bounds host memory)."""
    r, f, d = rep.shape
    voted = np.empty((f, d), np.float32)
    for i0 in range(0, f, step):
        voted[i0:i0 + step] = oracle.vote(rep[:, i0:i0 + step].cpu().numpy())
    return voted


def _dist_errors(got, want):
    assert np.array_equal(got, got.T) and (np.diag(got) == 0).all()
    off = ~np.eye(want.shape[0], dtype=bool)
    nz = off & (want > 0)
    assert (got[off & (want == 0)] == 0).all()          # colluding rows are identical: exactly 0
    rel = np.abs(got[nz] - want[nz]) / want[nz]
    return float(rel.max())


def _rel_l2(got, want):
    got, want = np.asarray(got, np.float64), np.asarray(want, np.float64)
    return float(np.linalg.norm(got - want) / np.linalg.norm(want))


def _multikrum_gap(D, c, m):
    """Smallest relative gap between the scores on the two sides of the selection boundary."""
    s = np.sort(oracle.krum_scores(D, c), kind="stable")
    if m >= len(s):
        return float("inf")
    return float((s[m] - s[m - 1]) / s[m]) if s[m] > 0 else 0.0


def _bulyan_gaps(D, c, selected):
    """Per pick: relative gap between the best and the second-best score among the rows still in play
    (scores as the first stage defines them: clamp(|R| - c - 2, 1, |R| - 1) nearest rows inside R).
    Written out here only to REPORT the margin; the picks themselves are the oracle's."""
    f = D.shape[0]
    left = list(range(f))
    gaps = []
    for pick in selected:
        if len(left) > 1:
            nb = min(max(len(left) - c - 2, 1), len(left) - 1)
            sc = []
            for a in left:
                row = np.sort(np.array([D[a, b] for b in left if b != a]))
                sc.append(float(np.sum(row[:nb])))
            order = np.argsort(np.array(sc), kind="stable")
            assert left[order[0]] == int(pick)
            best, second = sc[order[0]], sc[order[1]]
            gaps.append((second - best) / second if second > 0 else 0.0)
        left.remove(int(pick))
    return gaps


@pytest.mark.parametrize("c,m", [(5, 44), (8, 41)])
def test_multikrum_config_on_all_rows(c, m):
    l, r, q, d = 7, 3, 5, 11_200_000
    f = l * l
    rep = _cluster(l, r, q, d, "alie")
    dist = torch.empty((f, f), dtype=torch.float64, device=DEV)
    ws = bz.alloc_workspace(bz.OP_MULTIKRUM, 0, f, d, c, m)
    out, sel, voted = bz.vote_multikrum(rep, c, m, workspace=ws, dist=dist)
    assert bz.pairdist_status(ws, f) == 0                  # the tensor-core kernel's distances stood
    want_voted = _oracle_vote_by_files(rep)
    del rep
    assert np.array_equal(voted.cpu().numpy().view(np.uint32), want_voted.view(np.uint32))
    want_out, want_sel, want_D = oracle.multikrum(want_voted, c, m)
    err = _dist_errors(dist.cpu().numpy(), want_D)
    gap = _multikrum_gap(want_D, c, m)
    _report("multikrum_r3_f49_d11.2M_c%d_m%d" % (c, m),
            {"oracle_min_rel_score_gap_at_boundary": gap, "gpu_max_rel_error_in_D": err,
             "selected_equal": sel.cpu().tolist() == want_sel.tolist()})
    assert err <= DIST_TOL and err <= I8_SHARP
    assert sel.cpu().tolist() == want_sel.tolist()
    assert _rel_l2(out.cpu().numpy(), want_out) <= MEAN_TOL
    assert np.array_equal(out.cpu().numpy(), want_out)     # binary64 sums in `selected` order on both sides
    # the given-rows instance of the kernel on the same rows
    alone = bz.pairdist(voted).cpu().numpy()
    err_alone = _dist_errors(alone, want_D)
    assert err_alone <= I8_SHARP


def test_bulyan_config_on_all_rows():
    l, r, q, d, c = 5, 5, 6, 25_000_000, 4
    f = l * l
    rep = _cluster(l, r, q, d, "constant", heavy=0.01)
    ws = bz.alloc_workspace(bz.OP_BULYAN, 0, f, d, c)
    out, sel, voted = bz.vote_bulyan(rep, c, workspace=ws)
    assert bz.pairdist_status(ws, f) == 0
    voted2, dist = bz.vote_pairdist(rep)                   # the same first stage, to look at D itself
    assert torch.equal(voted2.view(torch.int32), voted.view(torch.int32))
    want_voted = _oracle_vote_by_files(rep, step=5)
    del rep, voted2
    assert np.array_equal(voted.cpu().numpy().view(np.uint32), want_voted.view(np.uint32))
    want_out, want_sel, want_D = oracle.bulyan(want_voted, c)
    err = _dist_errors(dist.cpu().numpy(), want_D)
    gaps = _bulyan_gaps(want_D, c, want_sel)
    # colluding rows are identical, so some picks are exact ties (both sides then take the lower index)
    _report("bulyan_r5_f25_d25M_c4",
            {"oracle_min_nonzero_rel_score_gap_over_picks": float(min(g for g in gaps if g > 0)),
             "picks_decided_by_index_on_exactly_equal_scores": int(sum(1 for g in gaps if g == 0)),
             "gpu_max_rel_error_in_D": err,
             "selected_equal": sel.cpu().tolist() == want_sel.tolist()})
    assert err <= DIST_TOL and err <= I8_SHARP
    assert sel.cpu().tolist() == want_sel.tolist()
    got = out.cpu().numpy()
    assert _rel_l2(got, want_out) <= MEAN_TOL
    assert np.array_equal(got.view(np.uint32), want_out.view(np.uint32))
    with pytest.raises(bz.BzError) as e:                   # c = q = 6 violates f >= 4c + 3 (Sec. 6.1)
        bz.vote_bulyan(torch.zeros((5, 25, 64), device=DEV), 6)
    assert e.value.status == bz.ERR_PRECONDITION


SHIPPED = [  # (l, r, d): every instance of the integer kernel the library dispatches to, at a full-size d
    (5, 3, 11_200_000), (7, 3, 11_200_000), (5, 5, 25_000_000), (7, 5, 11_200_000), (7, 7, 11_200_000)]


@pytest.mark.parametrize("l,r,d", SHIPPED)
def test_fifty_launches_give_the_same_bits(l, r, d, monkeypatch):
    # integer sums do not depend on the order in which tiles, CTAs or warps get there
    monkeypatch.setenv("BZ_PAIRDIST_PATH", "i8")
    f = l * l
    wf, fw, _ = oracle.assign(l, r)
    byz = oracle.worst_case(wf, f, r, 3)[1]
    g = inputs.true_gradients(f, d, seed=3, device=DEV)
    rep = inputs.build_replicas(g, fw, byz, "reversed")
    del g
    voted = torch.empty((f, d), dtype=torch.float32, device=DEV)
    ws = bz.alloc_workspace(bz.OP_PAIRDIST, 0, f, d)
    first = None
    for it in range(50):
        dist = torch.empty((f, f), dtype=torch.float64, device=DEV)
        bz.vote_pairdist(rep, voted=voted, workspace=ws, dist=dist)
        if first is None:
            first = dist.clone()
            first_voted = voted.clone()
        else:
            assert torch.equal(dist, first), "launch %d differs" % it
    assert torch.equal(voted.view(torch.int32), first_voted.view(torch.int32))
    assert bz.pairdist_status(ws, f) == 0
    if r == 3 or (l, r) == (5, 5):                         # the two given-rows instances (f = 25 at 25 M, f = 49 at 11.2 M)
        del rep
        first = None
        for it in range(50):
            dist = torch.empty((f, f), dtype=torch.float64, device=DEV)
            bz.pairdist(voted, workspace=ws, dist=dist)
            if first is None:
                first = dist.clone()
            else:
                assert torch.equal(dist, first), "launch %d differs" % it


@pytest.mark.expired_waits
@pytest.mark.parametrize("l,r", [(7, 3), (5, 5)])
def test_results_are_repaired_after_waits_that_ran_out(l, r):
    # The loader threads are told to issue nothing, so every CTA's first bounded wait expires (about a second)
    # and the kernel ends early with its outputs incomplete.  The call must still deliver: the vote kernel
    # rebuilds the voted rows, the binary32 kernel the distances; status and counter say what happened.
    f, d = l * l, 120_004
    wf, fw, _ = oracle.assign(l, r)
    byz = oracle.worst_case(wf, f, r, 3)[1]
    rep = inputs.build_replicas(inputs.true_gradients(f, d, seed=11), fw, byz, "alie")
    want_voted = oracle.vote(rep.numpy())
    want_D = oracle.pairdist(want_voted)
    rep_dev = rep.to(DEV)
    ws = bz.alloc_workspace(bz.OP_MULTIKRUM, 0, f, d, 3, f - 3)
    voted = torch.full((f, d), float("nan"), dtype=torch.float32, device=DEV)
    before = bz.pipeline_timeouts()
    bz.debug_stall_pipeline(True)
    try:
        _, dist = bz.vote_pairdist(rep_dev, voted=voted, workspace=ws)
        status = bz.pairdist_status(ws, f)
        alone = bz.pairdist(voted, workspace=ws)
        status_alone = bz.pairdist_status(ws, f)
    finally:
        bz.debug_stall_pipeline(False)
    assert status == bz.STATUS_RECOMPUTED | bz.STATUS_STOPPED_EARLY == status_alone
    assert bz.pipeline_timeouts() > before
    assert np.array_equal(voted.cpu().numpy().view(np.uint32), want_voted.view(np.uint32))
    for got in (dist, alone):
        assert _dist_errors(got.cpu().numpy(), want_D) <= DIST_TOL
    # the whole aggregator on top of a stalled first stage, then a healthy call on the same workspace
    bz.debug_stall_pipeline(True)
    try:
        out, sel, _ = bz.vote_multikrum(rep_dev, 3, f - 3, workspace=ws)
        torch.cuda.synchronize()
    finally:
        bz.debug_stall_pipeline(False)
    want_out, want_sel, _ = oracle.multikrum(want_voted, 3, f - 3)
    assert sel.cpu().tolist() == want_sel.tolist() and _rel_l2(out.cpu().numpy(), want_out) <= MEAN_TOL
    mid = bz.pipeline_timeouts()
    _, dist = bz.vote_pairdist(rep_dev, voted=voted, workspace=ws)
    assert bz.pairdist_status(ws, f) == 0 and bz.pipeline_timeouts() == mid
    assert _dist_errors(dist.cpu().numpy(), want_D) <= I8_SHARP
