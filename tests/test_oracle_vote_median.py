"""Pins for the oracle's majority vote (Eq. 3) and coordinate-wise median.  CPU only."""
import struct
from collections import Counter

import numpy as np
import pytest
import torch

import oracle
from paper_2010_04902_b200 import inputs


def _f(bits):
    return struct.unpack("<f", struct.pack("<I", bits))[0]


def _bits(a):
    return np.ascontiguousarray(a, np.float32).view(np.uint32)


def _cluster(l, r, q, d, attack, seed=0, **kw):
    wf, fw, _ = oracle.assign(l, r)
    _, byz, _ = oracle.worst_case(wf, l * l, r, q)
    g = inputs.true_gradients(l * l, d, seed=seed)
    rep = inputs.build_replicas(g, fw, byz, attack, **kw)
    return g.numpy(), rep.numpy(), fw, byz


# ------------------------------------------------------------------ vote

def test_vote_hand_cases():
    # one file, one coordinate each; columns are the r copies in order k = 0..r-1
    a, b, c = 1.5, -2.25, 7.0
    cases = [
        ([a, a, a], a), ([a, b, a], a), ([b, a, a], a), ([a, a, b], a),
        ([a, b, c], a),                       # three-way tie: first occurrence
        ([a, b, b, a, c], a),                 # 2-2 tie: value first seen at k = 0
        ([b, a, a, b, b], b), ([c, a, b, a, a], a),
        ([a, b, c, c, b, a, a], a), ([a, b, b, c, c, c, b], b),  # 3-3 tie at r = 7
    ]
    for copies, want in cases:
        rep = np.array(copies, np.float32).reshape(len(copies), 1, 1)
        assert oracle.vote(rep)[0, 0] == np.float32(want), copies


def test_vote_is_bitwise():
    pz, nz = _f(0x00000000), _f(0x80000000)
    n1, n2 = _f(0x7FC00001), _f(0x7FC00002)  # two NaNs with different payloads
    cases = [([pz, nz, nz], 0x80000000), ([nz, pz, pz], 0x00000000), ([pz, nz, 1.0], 0x00000000),
             ([n1, n2, n2], 0x7FC00002), ([n1, n1, n2], 0x7FC00001), ([1.0, n1, n1], 0x7FC00001)]
    for copies, want_bits in cases:
        rep = np.array([_bits(np.float32(x)) for x in copies], np.uint32).view(np.float32).reshape(3, 1, 1)
        assert int(_bits(oracle.vote(rep))[0, 0]) == want_bits


def test_vote_against_counter_brute_force():
    rng = np.random.default_rng(5)
    for r in (1, 3, 5, 7):
        # few distinct values so that ties and pluralities of every shape occur
        rep = rng.integers(0, 3, size=(r, 4, 200)).astype(np.float32)
        got = oracle.vote(rep)
        for i in range(4):
            for j in range(200):
                col = [float(x) for x in rep[:, i, j]]
                cnt = Counter(col)
                top = max(cnt.values())
                want = next(x for x in col if cnt[x] == top)
                assert got[i, j] == want


def test_vote_r1_is_identity():
    rep = np.random.default_rng(0).standard_normal((1, 9, 33)).astype(np.float32)
    assert np.array_equal(_bits(oracle.vote(rep)), _bits(rep[0]))


@pytest.mark.parametrize("l,r,q,attack,want_distorted", [
    (5, 3, 2, "alie", 1),       # table (15,25,5,3), q = 2
    (5, 3, 3, "reversed", 3),   # q = 3
    (7, 3, 5, "alie", 8),       # table (21,49,7,3), q = 5
    (5, 5, 6, "constant", 4),   # table (25,25,5,5), q = 6
])
def test_vote_count_identity_at_worst_case_placement(l, r, q, attack, want_distorted):
    # Sec. 2: a file's gradient is distorted only if at least r' of its copies are Byzantine; at
    # the worst-case placement the number of such files is the printed c_max.
    g, rep, fw, byz = _cluster(l, r, q, 257, attack)
    voted = oracle.vote(rep)
    distorted = [i for i in range(l * l) if not np.array_equal(_bits(voted[i]), _bits(g[i]))]
    assert len(distorted) == want_distorted
    rp = (r + 1) // 2
    for i in range(l * l):
        n_byz = sum(1 for u in fw[i] if u in set(byz.tolist()))
        assert (i in distorted) == (n_byz >= rp)
    # colluding attackers: the element-wise vote equals the whole-vector vote of the paper
    win = oracle.vote_vectorwise(rep)
    for i in range(l * l):
        assert np.array_equal(_bits(voted[i]), _bits(rep[win[i], i]))


def test_vote_minority_corruption_is_harmless():
    # q < r' Byzantine workers cannot change any winner (Sec. 2).
    wf, fw, _ = oracle.assign(5, 3)
    g = inputs.true_gradients(25, 101, seed=3)
    for byz in ([4], [7], [13]):
        for attack in ("alie", "reversed", "constant", "independent"):
            rep = inputs.build_replicas(g, fw, byz, attack).numpy()
            assert np.array_equal(_bits(oracle.vote(rep)), _bits(g.numpy()))


def test_vote_independent_attackers_plurality():
    # Honest copies in the minority and Byzantine copies all different: the honest value wins a
    # file only where it is the earliest of the equally frequent patterns.
    wf, fw, _ = oracle.assign(5, 5)
    g = inputs.true_gradients(25, 64, seed=1)
    byz = [0, 5, 10, 15]           # four of the five holders of file 0 (one per class)
    assert all(0 in wf[u] for u in byz)
    rep = inputs.build_replicas(g, fw, byz, "independent").numpy()
    voted = oracle.vote(rep)
    # file 0: copies k = 0..3 are distinct random vectors, k = 4 is honest -> all counts are 1,
    # the copy of class 0 wins
    assert np.array_equal(_bits(voted[0]), _bits(rep[0, 0]))
    for i in range(1, 25):
        n_byz = sum(1 for u in fw[i] if u in byz)
        assert n_byz <= 1
        assert np.array_equal(_bits(voted[i]), _bits(g.numpy()[i]))


# ------------------------------------------------------------------ median

def test_median_hand_cases():
    cases = [([3, 1, 2], 2.0), ([5, 5, 5], 5.0), ([1, 9, 2, 8, 3], 3.0), ([-1, -7, 4, 0, 2, 2, -3], 0.0),
             ([1, 2, 3, 4], 2.5), ([4, 1], 2.5), ([6], 6.0)]
    for vals, want in cases:
        v = np.array(vals, np.float32).reshape(len(vals), 1)
        assert oracle.median(v)[0] == np.float32(want), vals


def test_median_total_order_on_zeros_and_nans():
    pz, nz = 0x00000000, 0x80000000
    pnan, nnan = 0x7FC00000, 0xFFC00000
    one, two = 0x3F800000, 0x40000000
    cases = [([nz, pz, pz], pz), ([nz, nz, pz], nz), ([pz, nz, one], pz), ([pnan, one, two], two),
             ([nnan, one, two], one), ([pnan, pnan, one], pnan), ([nnan, nnan, pnan], nnan)]
    for bits, want in cases:
        v = np.array(bits, np.uint32).view(np.float32).reshape(3, 1)
        assert int(_bits(oracle.median(v))[0]) == want, [hex(b) for b in bits]


@pytest.mark.parametrize("f", [1, 3, 5, 9, 25, 49, 63])
def test_median_matches_numpy(f):
    v = np.random.default_rng(f).standard_normal((f, 1000)).astype(np.float32)
    v[:, :50] = np.round(v[:, :50]) + np.float32(0.0)  # many duplicates; "+ 0" turns -0.0 into +0.0
    want = np.median(v, axis=0)      # odd count: numpy returns the middle element itself
    assert np.array_equal(_bits(oracle.median(v)), _bits(want))
    want2 = np.sort(v, axis=0)[(f - 1) // 2]
    assert np.array_equal(_bits(oracle.median(v)), _bits(want2))


@pytest.mark.parametrize("f", [2, 4, 16, 64])
def test_median_even_count(f):
    v = np.random.default_rng(f).standard_normal((f, 500)).astype(np.float32)
    s = np.sort(v, axis=0)
    want = np.float32(0.5) * s[f // 2 - 1] + np.float32(0.5) * s[f // 2]
    assert np.array_equal(_bits(oracle.median(v)), _bits(want))


def test_median_permutation_invariant_and_constant():
    rng = np.random.default_rng(2)
    v = rng.standard_normal((25, 300)).astype(np.float32)
    base = oracle.median(v)
    for _ in range(3):
        assert np.array_equal(_bits(oracle.median(v[rng.permutation(25)])), _bits(base))
    c = np.full((25, 17), -3.75, np.float32)
    assert (oracle.median(c) == np.float32(-3.75)).all()


@pytest.mark.parametrize("l,r,q,attack", [(5, 3, 2, "alie"), (5, 3, 3, "reversed"), (5, 3, 5, "constant"),
                                          (7, 3, 5, "alie"), (5, 5, 6, "constant")])
def test_median_stays_in_honest_range(l, r, q, attack):
    # With fewer than f/2 distorted files the median lies between the smallest and the largest
    # honest value of every coordinate - the property the defence relies on (Sec. 6.1).
    g, rep, fw, byz = _cluster(l, r, q, 513, attack)
    voted = oracle.vote(rep)
    honest = [i for i in range(l * l) if np.array_equal(_bits(voted[i]), _bits(g[i]))]
    assert len(honest) > (l * l) / 2
    out = oracle.median(voted)
    assert (out >= g[honest].min(0)).all() and (out <= g[honest].max(0)).all()
    assert np.array_equal(_bits(oracle.vote_median(rep)), _bits(out))


def test_inputs_are_seeded():
    a = inputs.true_gradients(25, 1000, seed=0)
    b = inputs.true_gradients(25, 1000, seed=0)
    c = inputs.true_gradients(25, 1000, seed=1)
    assert torch.equal(a, b) and not torch.equal(a, c)
    # per-coordinate spread sigma = 0.1 around a shared N(0,1) mean
    assert abs(float(a.std(dim=0, unbiased=True).mean()) - 0.1) < 0.01
    assert abs(float(a.mean(dim=0).std()) - 1.0) < 0.1
    h = inputs.true_gradients(25, 200000, seed=0, heavy_tail_frac=0.01)
    dev = (h - h.median(dim=0).values).abs().max(dim=0).values
    frac_wide = float((dev > 0.6).float().mean())   # 6 sigma: only heavy-tailed coordinates get there
    assert 0.002 < frac_wide < 0.012


# ---- Eq. (3) on whole vectors (the paper's own statement of the vote) --------------------------------

def test_vectorwise_vote_hand_cases():
    # file 0: copies (A, B, A) -> A wins, first at k = 0;  file 1: (A, B, B) -> k = 1;
    # file 2: three different vectors -> every count is 1, the earliest copy wins
    A = np.array([1.0, 2.0, 3.0, 4.0], np.float32)
    B = np.array([1.0, 2.0, 3.0, 4.5], np.float32)   # differs from A in the last coordinate only
    C = np.array([9.0, 2.0, 3.0, 4.0], np.float32)   # differs in the first coordinate only
    rep = np.stack([np.stack([A, A, A]), np.stack([B, B, B]), np.stack([A, B, C])])   # [k][file]
    assert oracle.vote_vectorwise(rep).tolist() == [0, 1, 0]
    # r = 5: (A, B, B, A, C) is a 2-2 tie -> the vector seen first (k = 0); (C, B, B, A, B) -> B at k = 1
    rep5 = np.stack([np.stack([A, C]), np.stack([B, B]), np.stack([B, B]), np.stack([A, A]), np.stack([C, B])])
    assert oracle.vote_vectorwise(rep5).tolist() == [0, 1]
    # equality is on bit patterns: +0 and -0 are different vectors, a NaN equals itself
    Z = np.array([0.0, 1.0], np.float32)
    N = np.array([-0.0, 1.0], np.float32)
    Q = np.array([np.nan, 1.0], np.float32)
    rep3 = np.stack([np.stack([Z, Q]), np.stack([N, Q]), np.stack([N, Z])])
    assert oracle.vote_vectorwise(rep3).tolist() == [1, 0]


def test_vectorwise_vote_against_counter():
    # brute force: the most common byte string among a file's copies, ties to the one seen first
    from collections import Counter
    rng = np.random.default_rng(11)
    for r, f, d in [(3, 6, 5), (5, 9, 3), (7, 4, 2)]:
        pool = rng.integers(-2, 3, size=(3, d)).astype(np.float32)    # few distinct vectors -> many agreements
        pick = rng.integers(0, 3, size=(r, f))
        rep = pool[pick]
        win = oracle.vote_vectorwise(rep)
        for i in range(f):
            keys = [rep[k, i].tobytes() for k in range(r)]
            cnt = Counter(keys)
            best = max(cnt.values())
            first = next(k for k in range(r) if cnt[keys[k]] == best)
            assert win[i] == first


def test_vectorwise_and_elementwise_votes_differ_only_without_an_agreeing_majority():
    # A file with honest copies in the minority and Byzantine copies that disagree among themselves:
    # element by element the honest value can still win coordinates where two attackers happen to
    # agree with it, while no whole vector has a majority (the case Sec. 2 leaves open).
    g = np.array([[1.0, 2.0, 3.0]], np.float32)
    b1 = np.array([[1.0, 7.0, 8.0]], np.float32)
    b2 = np.array([[5.0, 2.0, 9.0]], np.float32)
    rep = np.stack([b1, b2, g])                      # k = 0, 1 Byzantine, k = 2 honest
    assert oracle.vote_vectorwise(rep).tolist() == [0]           # all counts 1: first copy
    assert oracle.vote(rep)[0].tolist() == [1.0, 2.0, 8.0]       # per coordinate: 1 (b1, g), 2 (b2, g), tie -> first
    # with a true majority both rules return the honest vector
    rep = np.stack([g, b2, g])
    assert oracle.vote_vectorwise(rep).tolist() == [0]
    assert np.array_equal(oracle.vote(rep)[0], g[0])


# ---- agreement up to a tolerance (Sec. 2: clusters of nearly equal copies) --------------------------

def test_cluster_vote_reduces_to_the_exact_vote():
    rng = np.random.default_rng(3)
    pool = rng.standard_normal((3, 6)).astype(np.float32)
    rep = pool[rng.integers(0, 3, size=(5, 8))]
    assert oracle.vote_clusters(rep, 0.0, 0.0).tolist() == oracle.vote_vectorwise(rep).tolist()


def test_cluster_vote_hand_cases():
    one = np.float32(1.0)
    up = np.nextafter(one, np.float32(2.0))          # 1 + 2^-23
    A = np.array([1.0, 100.0], np.float32)
    A1 = np.array([up, 100.0], np.float32)           # A with one ulp of noise
    Bz = np.array([1.0, -100.0], np.float32)
    # exact vote: three different vectors -> first copy; with a relative tolerance of 1e-6 the two honest
    # copies agree and the earlier of them wins although the Byzantine copy comes first
    rep = np.stack([Bz, A, A1])[:, None, :]
    assert oracle.vote_vectorwise(rep).tolist() == [0]
    assert oracle.vote_clusters(rep, 0.0, 1e-6).tolist() == [1]
    assert oracle.vote_clusters(rep, 0.0, 1e-8).tolist() == [0]      # tolerance below one ulp: nothing agrees
    # agreement is not transitive: 0.0 ~ 0.6 ~ 1.2 with abs_tol 0.7, but 0.0 !~ 1.2 -> the middle copy agrees with all
    rep = np.array([[[0.0]], [[1.2]], [[0.6]]], np.float32)
    assert oracle.vote_clusters(rep, 0.7, 0.0).tolist() == [2]
    # the bound is abs_tol + rel_tol * max(|a|, |b|): 10 vs 11 agree at rel_tol 0.1 (bound 1.1), not at 0.05;
    # with abs_tol 0.5 added the second bound is 1.05 and they agree again
    rep = np.array([[[10.0]], [[11.0]], [[50.0]]], np.float32)
    assert oracle.vote_clusters(rep, 0.0, 0.1).tolist() == [0]
    rep3 = np.array([[[50.0]], [[10.0]], [[11.0]]], np.float32)
    assert oracle.vote_clusters(rep3, 0.0, 0.1).tolist() == [1]
    assert oracle.vote_clusters(rep3, 0.0, 0.05).tolist() == [0]
    assert oracle.vote_clusters(rep3, 0.5, 0.05).tolist() == [1]
    # one coordinate out of tolerance breaks the agreement of the whole vector
    C = np.array([1.0, 2.0, 3.0], np.float32)
    C1 = np.array([1.0, 2.0, 3.5], np.float32)
    rep = np.stack([C1, C, C])[:, None, :]
    assert oracle.vote_clusters(rep, 0.1, 0.0).tolist() == [1]
    # NaN agrees only with the same bit pattern; infinities of equal sign are equal bit patterns
    N = np.array([np.nan, 1.0], np.float32)
    I = np.array([np.inf, 1.0], np.float32)
    rep = np.stack([N, I, I])[:, None, :]
    assert oracle.vote_clusters(rep, 1.0, 1.0).tolist() == [1]
    rep = np.stack([N, N, I])[:, None, :]
    assert oracle.vote_clusters(rep, 1.0, 1.0).tolist() == [0]


def test_cluster_vote_recovers_noisy_honest_copies():
    # honest copies differ by rounding noise (a few ulps), Byzantine copies collude: the exact vote is
    # lost on every file (all copies differ), the cluster vote picks an honest copy wherever honest copies
    # are in the majority - the guarantee of Sec. 2 carried over
    wf, fw, _ = oracle.assign(5, 3)
    byz = oracle.worst_case(wf, 25, 3, 3)[1]
    g = inputs.true_gradients(25, 300, seed=4)
    rep = inputs.build_replicas(g, fw, byz, "reversed").numpy().copy()
    rng = np.random.default_rng(0)
    noise = (1.0 + rng.integers(-2, 3, size=rep.shape) * 2.0 ** -23).astype(np.float32)
    honest = np.ones(rep.shape[:2], bool)
    for i in range(25):
        for k in range(3):
            honest[k, i] = int(fw[i][k]) not in set(int(b) for b in byz)
    rep = np.where(honest[:, :, None], rep * noise, rep)
    win = oracle.vote_clusters(rep, 0.0, 1e-5)
    for i in range(25):
        if honest[:, i].sum() >= 2:
            assert honest[win[i], i] and win[i] == int(np.argmax(honest[:, i]))
        else:
            assert not honest[win[i], i]
