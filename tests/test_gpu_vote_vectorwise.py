"""GPU parity of the whole-vector vote (Eq. 3 as stated in Sec. 2) against the CPU oracle: winners and
voted rows bit-exact."""
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


def _check(rep):
    want_win = oracle.vote_vectorwise(rep.numpy())
    voted, win = bz.vote_vectorwise(rep.to(DEV))
    assert win.cpu().tolist() == want_win.tolist()
    want = np.stack([rep.numpy()[want_win[i], i] for i in range(rep.shape[1])])
    assert np.array_equal(_bits(voted), _bits(want))
    return voted, win


@pytest.mark.parametrize("l,r,q,attack,d", [(5, 3, 3, "reversed", 40_000), (7, 3, 5, "alie", 30_001), (5, 5, 6, "constant", 20_002),
                                            (7, 5, 5, "independent", 10_003), (7, 7, 4, "reversed", 8_000), (3, 3, 2, "alie", 7)])
def test_clusters(l, r, q, attack, d):
    wf, fw, _ = oracle.assign(l, r)
    byz = oracle.worst_case(wf, l * l, r, q)[1]
    g = inputs.true_gradients(l * l, d, seed=l + r)
    rep = inputs.build_replicas(g, fw, byz, attack)
    voted, _ = _check(rep)
    if attack != "independent":
        # colluding attackers: the paper's whole-vector vote and the element-wise vote give the same rows
        assert np.array_equal(_bits(voted), _bits(bz.vote(rep.to(DEV))))


def test_copies_that_differ_in_one_coordinate():
    # the difference sits in the first, a middle or the very last coordinate (tail of an odd length)
    rng = np.random.default_rng(0)
    r, f, d = 5, 6, 100_003
    g = rng.standard_normal((f, d)).astype(np.float32)
    rep = np.repeat(g[None], r, axis=0).copy()
    rep[0, 0, 0] += 1.0                    # file 0: copy 0 alone differs -> copies 1..4 agree, winner k = 1
    rep[1, 1, d // 2] += 1.0               # file 1: copy 1 alone
    rep[4, 2, d - 1] += 1.0                # file 2: copy 4 alone, last coordinate
    rep[0, 3, 5] = 7.0
    rep[1, 3, 5] = 7.0                     # file 3: copies (0, 1) agree, (2, 3, 4) agree -> k = 2
    rep[0, 4, 9] = 1.0
    rep[1, 4, 9] = 2.0
    rep[2, 4, 9] = 3.0
    rep[3, 4, 9] = 4.0                     # file 4: all five differ -> k = 0
    rep[:, 5, 77] = np.float32(-0.0)
    rep[2, 5, 77] = np.float32(0.0)        # file 5: +0 against four -0: bit patterns differ
    _, win = _check(torch.from_numpy(rep))
    assert win.cpu().tolist() == [1, 0, 0, 2, 0, 0]


def test_other_r_and_layouts():
    rng = np.random.default_rng(5)
    # r = 9 and r = 11: the generic kernel (more than 32 pairs of copies)
    for r, f, d in [(9, 4, 5_000), (11, 3, 2_001), (1, 5, 300)]:
        pool = rng.standard_normal((3, f, d)).astype(np.float32)
        pick = rng.integers(0, 3, size=(r, f))
        rep = np.stack([np.stack([pool[pick[k, i], i] for i in range(f)]) for k in range(r)])
        _check(torch.from_numpy(rep))
    # padded rows and an unaligned start (leading dimensions not multiples of 4)
    g = torch.from_numpy(rng.standard_normal((25, 1001)).astype(np.float32))
    rep = g[None].repeat(3, 1, 1).clone()
    rep[2, 7] = -rep[2, 7]
    rep[0, 8] = 0.5
    rep[1, 8] = 0.5
    big = torch.zeros((3, 25, 1007), dtype=torch.float32, device=DEV)
    big[:, :, 3:1004] = rep.to(DEV)
    voted, win = bz.vote_vectorwise(big[:, :, 3:1004])
    want_win = oracle.vote_vectorwise(rep.numpy())
    assert win.cpu().tolist() == want_win.tolist()
    assert np.array_equal(_bits(voted), _bits(np.stack([rep.numpy()[want_win[i], i] for i in range(25)])))


def test_two_calls_share_the_workspace():
    # the pair bits of one call must not leak into the next
    g = inputs.true_gradients(25, 4096, seed=1)
    rep_a = g[None].repeat(3, 1, 1).clone()
    rep_a[0] += 1.0                                   # copy 0 differs everywhere -> winners k = 1
    rep_b = g[None].repeat(3, 1, 1).clone()           # all agree -> winners k = 0
    ws = bz.alloc_workspace(bz.OP_VOTE_VECTORWISE, 3, 25, 4096)
    _, win_a = bz.vote_vectorwise(rep_a.to(DEV), workspace=ws)
    _, win_b = bz.vote_vectorwise(rep_b.to(DEV), workspace=ws)
    assert win_a.cpu().tolist() == [1] * 25 and win_b.cpu().tolist() == [0] * 25


def test_full_size_cluster():
    # K = 15, r = 3, f = 25, d = 11.2 M on the device; the oracle checks the winners from the worker
    # placement (a file's winner is its first honest copy when at most one holder is Byzantine, else
    # the first Byzantine copy: colluders send one vector) and sampled columns of the voted rows
    l, r, q, d = 5, 3, 3, 11_200_000
    wf, fw, _ = oracle.assign(l, r)
    byz = set(int(u) for u in oracle.worst_case(wf, l * l, r, q)[1])
    g = inputs.true_gradients(l * l, d, seed=0, device=DEV)
    rep = inputs.build_replicas(g, fw, sorted(byz), "reversed")
    voted, win = bz.vote_vectorwise(rep)
    torch.cuda.synchronize()
    want_win = []
    for i in range(l * l):
        bad = [int(fw[i][k]) in byz for k in range(r)]
        want_win.append(bad.index(True) if sum(bad) >= 2 else bad.index(False))
    assert win.cpu().tolist() == want_win
    idx = torch.from_numpy(np.unique(np.concatenate([np.arange(0, 64), np.arange(d - 64, d),
                                                     np.random.default_rng(2).integers(0, d, 5000)]))).to(DEV)
    sample = rep[:, :, idx].cpu().numpy()
    assert oracle.vote_vectorwise(sample).tolist() == want_win      # the sample separates the copies as well
    assert np.array_equal(_bits(voted[:, idx]), _bits(np.stack([sample[want_win[i], i] for i in range(l * l)])))


# ---- agreement up to a tolerance ----------------------------------------------------------------------

def _check_clusters(rep, abs_tol, rel_tol):
    want_win = oracle.vote_clusters(rep.numpy(), abs_tol, rel_tol)
    voted, win = bz.vote_clusters(rep.to(DEV), abs_tol, rel_tol)
    assert win.cpu().tolist() == want_win.tolist()
    assert np.array_equal(_bits(voted), _bits(np.stack([rep.numpy()[want_win[i], i] for i in range(rep.shape[1])])))
    return win.cpu().tolist()


@pytest.mark.parametrize("l,r,q,d", [(5, 3, 3, 30_000), (7, 3, 5, 10_001), (5, 5, 6, 8_002), (7, 7, 4, 4_000)])
def test_noisy_honest_copies(l, r, q, d):
    wf, fw, _ = oracle.assign(l, r)
    byz = set(int(u) for u in oracle.worst_case(wf, l * l, r, q)[1])
    g = inputs.true_gradients(l * l, d, seed=l * r)
    rep = inputs.build_replicas(g, fw, sorted(byz), "reversed").numpy().copy()
    rng = np.random.default_rng(l)
    noise = (1.0 + rng.integers(-2, 3, size=rep.shape) * 2.0 ** -23).astype(np.float32)
    honest = np.array([[int(fw[i][k]) not in byz for i in range(l * l)] for k in range(r)])
    rep = torch.from_numpy(np.where(honest[:, :, None], rep * noise, rep).astype(np.float32))
    win = _check_clusters(rep, 0.0, 1e-5)
    rp = (r + 1) // 2
    for i in range(l * l):
        assert honest[win[i], i] == (honest[:, i].sum() >= rp)       # Sec. 2's guarantee, carried over
    # tolerances on either side of the noise, and the exact vote as the zero-tolerance case
    _check_clusters(rep, 0.0, 1e-8)
    _check_clusters(rep, 1e-3, 0.0)
    assert _check_clusters(rep, 0.0, 0.0) == oracle.vote_vectorwise(rep.numpy()).tolist()


def test_cluster_vote_edge_values_and_generic_r():
    rng = np.random.default_rng(9)
    # values at the edge of the bound, NaN and infinities, r = 9 (generic kernel), odd length
    r, f, d = 9, 5, 1_003
    base = rng.standard_normal((f, d)).astype(np.float32)
    rep = np.repeat(base[None], r, axis=0).copy()
    rep[1:4, 0] += np.float32(0.25)                 # three copies shifted by exactly the absolute tolerance
    rep[4:, 1] *= np.float32(1.0 + 2.0 ** -10)      # five copies scaled to the edge of the relative tolerance
    rep[0, 2, 17] = np.nan
    rep[1, 2, 17] = np.nan
    rep[2, 3, 5] = np.inf
    rep[3, 3, 5] = np.inf
    rep[4, 3, 5] = -np.inf
    rep = torch.from_numpy(rep)
    for abs_tol, rel_tol in [(0.25, 0.0), (0.2499, 0.0), (0.0, 2.0 ** -10), (0.0, 2.0 ** -11), (0.1, 0.01)]:
        _check_clusters(rep, abs_tol, rel_tol)


@pytest.mark.parametrize("r", [3, 5, 7])
def test_cluster_vote_edge_values_vector_kernels(r):
    # the same edge cases through the 128-bit kernels (d a multiple of 4): bound met exactly, one step
    # beyond it, equal and unequal NaNs, infinities of either sign, signed zeros, one bad coordinate per file
    rng = np.random.default_rng(90 + r)
    f, d = 12, 2_048
    base = rng.standard_normal((f, d)).astype(np.float32)
    rep = np.repeat(base[None], r, axis=0).copy()
    rep[1, 0] += np.float32(0.25)                                   # exactly the absolute tolerance away
    rep[1, 1] = np.nextafter(rep[1, 1] + np.float32(0.25), np.float32(np.inf))   # mostly one step beyond it
    rep[r - 1, 2] *= np.float32(1.0 + 2.0 ** -10)                   # edge of the relative tolerance
    rep[0, 3, 17] = np.nan                                          # a NaN in one copy only
    rep[:, 4, 33] = np.nan                                          # the same NaN everywhere: copies agree
    rep[0, 5, 5] = np.inf                                           # infinity against finite values
    rep[:, 6, 6] = np.inf                                           # equal infinities agree
    rep[0, 7, 7], rep[1:, 7, 7] = np.inf, -np.inf
    rep[0, 8, 8], rep[1:, 8, 8] = 0.0, -0.0
    rep[0, 9, 1023] = rep[0, 9, 1023] + np.float32(1.0)             # one coordinate off in copy 0
    rep[r // 2, 10, 2047] = np.float32(3e38)                        # the last coordinate of the middle copy
    rep[:, 11] = 0.0                                                # all zero
    rep = torch.from_numpy(rep)
    for abs_tol, rel_tol in [(0.25, 0.0), (0.2499, 0.0), (0.0, 2.0 ** -10), (0.0, 2.0 ** -11), (0.1, 0.01), (0.0, 0.0),
                             (1e30, 0.0), (0.0, 1.0)]:
        _check_clusters(rep, abs_tol, rel_tol)
