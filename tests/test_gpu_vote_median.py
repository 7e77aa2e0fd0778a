"""GPU parity: majority vote, coordinate-wise median and the fused pass against the CPU oracle,
bit for bit, through the C ABI."""
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


def _cluster(l, r, q, d, attack, seed=0):
    wf, fw, _ = oracle.assign(l, r)
    byz = oracle.worst_case(wf, l * l, r, q)[1] if q > 0 else []
    g = inputs.true_gradients(l * l, d, seed=seed)
    return inputs.build_replicas(g, fw, byz, attack)


def _check_all(rep_cpu, rep_dev=None):
    rep_dev = rep_cpu.to(DEV) if rep_dev is None else rep_dev
    want_voted = oracle.vote(rep_cpu.numpy())
    want_out = oracle.median(want_voted)
    voted = bz.vote(rep_dev)
    assert np.array_equal(_bits(voted), _bits(want_voted))
    assert np.array_equal(_bits(bz.median(voted)), _bits(want_out))
    assert np.array_equal(_bits(bz.vote_median(rep_dev)), _bits(want_out))


# sizes: below one vector, ragged tails, several CTAs' worth with a ragged tail
@pytest.mark.parametrize("d", [1, 3, 4, 5, 127, 1025, 70001])
@pytest.mark.parametrize("l,r,q,attack", [(5, 3, 3, "reversed"), (5, 5, 6, "constant"), (7, 3, 5, "alie"),
                                          (7, 5, 6, "alie"), (7, 7, 5, "reversed"), (3, 3, 2, "constant")])
def test_parity_specialised_and_generic_shapes(l, r, q, attack, d):
    _check_all(_cluster(l, r, q, d, attack))


@pytest.mark.parametrize("d", [2, 6, 1026, 70002])
@pytest.mark.parametrize("l,r,q,attack", [(5, 3, 3, "reversed"), (5, 5, 6, "constant"), (7, 3, 5, "alie"), (7, 7, 5, "reversed")])
def test_rows_on_8_byte_boundaries(l, r, q, attack, d):
    # d = 2 (mod 4): contiguous rows start on 8-byte, not 16-byte boundaries - the 64-bit load kernels
    rep = _cluster(l, r, q, d, attack)
    _check_all(rep)
    assert bz.last_path() == bz.PATH_REGISTERS
    # the same values in a window that starts 8 bytes into a padded allocation
    buf = torch.zeros((r, l * l, d + 10), dtype=torch.float32, device=DEV)
    buf[:, :, 2:2 + d] = rep.to(DEV)
    _check_all(rep, buf[:, :, 2:2 + d])


def test_config1_vote_then_median():
    # K=15, r=3, l=5, f=25, d=100000, q=2 at the worst-case placement, ALIE with z=1
    _check_all(_cluster(5, 3, 2, 100000, "alie", seed=0))


@pytest.mark.parametrize("r,f", [(3, 25), (5, 25), (7, 49), (5, 9), (9, 25), (3, 7)])
def test_plurality_rule_on_ties(r, f):
    # few distinct values: every count pattern and tie occurs; honest majority does not exist
    rng = np.random.default_rng(r * 100 + f)
    rep = torch.from_numpy(rng.integers(0, 3, size=(r, f, 1531)).astype(np.float32))
    _check_all(rep)


def test_independent_attackers():
    wf, fw, _ = oracle.assign(5, 5)
    g = inputs.true_gradients(25, 2049, seed=1)
    _check_all(inputs.build_replicas(g, fw, [0, 5, 10, 15, 7], "independent"))


def test_signed_zeros_nans_infinities():
    rng = np.random.default_rng(11)
    special = np.array([0x00000000, 0x80000000, 0x7FC00000, 0xFFC00000, 0x7FC00001, 0x7F800000, 0xFF800000,
                        0x00000001, 0x80000001, 0x3F800000, 0xBF800000], np.uint32)
    for r, f in [(3, 25), (5, 49), (3, 9)]:
        rep = special[rng.integers(0, len(special), size=(r, f, 777))].view(np.float32)
        _check_all(torch.from_numpy(rep.copy()))


@pytest.mark.parametrize("r,f", [(3, 25), (3, 49), (5, 9)])
def test_unaligned_base_and_padded_rows(r, f):
    d, ld = 1001, 1032
    big = torch.zeros((r, f, ld), dtype=torch.float32)
    big[:, :, :d] = torch.from_numpy(np.random.default_rng(3).integers(-2, 3, size=(r, f, d)).astype(np.float32))
    dev = big.to(DEV)
    # padded rows, aligned base
    _check_all(big[:, :, :d].contiguous(), dev[:, :, :d])
    # base shifted by one element: the scalar path
    _check_all(big[:, :, 1:d].contiguous(), dev[:, :, 1:d])
    # output into an unaligned slice
    out = torch.zeros(d + 1, dtype=torch.float32, device=DEV)
    bz.vote_median(dev[:, :, :d], out[1:])
    assert np.array_equal(_bits(out[1:]), _bits(oracle.vote_median(big[:, :, :d].contiguous().numpy())))
    voted = torch.zeros((f, ld), dtype=torch.float32, device=DEV)
    bz.vote(dev[:, :, :d], voted[:, 3:3 + d])
    assert np.array_equal(_bits(voted[:, 3:3 + d]), _bits(oracle.vote(big[:, :, :d].contiguous().numpy())))


@pytest.mark.parametrize("f", [1, 2, 4, 9, 25, 49, 64, 121])
def test_median_only_any_f(f):
    v = torch.from_numpy(np.random.default_rng(f).standard_normal((f, 3001)).astype(np.float32))
    v[:, :64] = torch.round(v[:, :64])
    assert np.array_equal(_bits(bz.median(v.to(DEV))), _bits(oracle.median(v.numpy())))


# ---- the TMA-staged kernels: every compiled (r, f), at sizes and layouts that really take them -------------------
STAGED_SHAPES = [(3, 25), (3, 49), (5, 25), (5, 49), (7, 49), (1, 25), (1, 49)]
_SPECIAL = np.array([0x00000000, 0x80000000, 0x7FC00000, 0xFFC00000, 0x7FC00001, 0x7F800000, 0xFF800000,
                     0x00000001, 0x80000001, 0x3F800000, 0xBF800000], np.uint32)


def _staged_inputs(kind, r, f, d, rng):
    if kind == "ties":          # three distinct values: every count pattern, no honest majority
        return rng.integers(0, 3, size=(r, f, d)).astype(np.float32)
    if kind == "special":       # signed zeros, NaN payloads, infinities, denormals
        return _SPECIAL[rng.integers(0, len(_SPECIAL), size=(r, f, d))].view(np.float32).copy()
    if kind == "independent":   # every copy a different vector except a common base: plurality decides
        base = rng.standard_normal((1, f, d)).astype(np.float32)
        rep = np.repeat(base, r, axis=0)
        lie = rng.random((r, f, d)) < 0.4
        rep[lie] = rng.standard_normal(int(lie.sum())).astype(np.float32)
        return rep
    raise ValueError(kind)


def _check_staged(rep_np, rep_dev):
    """Fused pass (or the median alone for r = 1) on the staged kernel, bit for bit against the oracle."""
    r = rep_np.shape[0]
    want = oracle.median(oracle.vote(rep_np))
    if r == 1:
        got = bz.median(rep_dev[0])
    else:
        got = bz.vote_median(rep_dev)
    assert bz.last_path() == bz.PATH_STAGED        # not the register kernels
    assert np.array_equal(_bits(got), _bits(want))


@pytest.mark.parametrize("kind", ["ties", "special", "independent"])
@pytest.mark.parametrize("r,f", STAGED_SHAPES)
def test_edge_values_through_the_staged_kernels(r, f, kind):
    rng = np.random.default_rng(1000 * r + f + len(kind))
    # aligned, several tiles per CTA... a size that ends in a ragged tile (multiple of 4, not of 128), and the smallest
    for d in (512, 4484, 148 * 128 * 2 + 36):
        rep = _staged_inputs(kind, r, f, d, rng)
        _check_staged(rep, torch.from_numpy(rep).to(DEV))
    # rows padded to a leading dimension that is a multiple of 4, window starting 16 bytes into the allocation
    d, ld = 3076, 3100
    rep = _staged_inputs(kind, r, f, d, rng)
    buf = torch.full((r, f, ld), float("nan"), dtype=torch.float32, device=DEV)
    buf[:, :, 4:4 + d] = torch.from_numpy(rep).to(DEV)
    _check_staged(rep, buf[:, :, 4:4 + d])


@pytest.mark.parametrize("kind", ["ties", "special", "independent"])
@pytest.mark.parametrize("r,f", [(3, 25), (3, 49), (5, 25), (5, 49), (7, 49)])
def test_vote_alone_through_the_staged_kernel(r, f, kind, monkeypatch):
    # bz_vote through the fused kernel's ring (the default where it applies): the winners,
    # bit for bit, on aligned sizes, a ragged last tile, padded replica rows and an output with its own leading dimension
    monkeypatch.setenv("BZ_VOTE_PATH", "staged")
    rng = np.random.default_rng(77 * r + f + len(kind))
    for d in (512, 4484, 148 * 128 + 36):
        rep = _staged_inputs(kind, r, f, d, rng)
        got = bz.vote(torch.from_numpy(rep).to(DEV))
        assert bz.last_path() == bz.PATH_STAGED
        assert np.array_equal(_bits(got), _bits(oracle.vote(rep)))
    d, ld = 3076, 3100
    rep = _staged_inputs(kind, r, f, d, rng)
    buf = torch.full((r, f, ld), float("nan"), dtype=torch.float32, device=DEV)
    buf[:, :, 4:4 + d] = torch.from_numpy(rep).to(DEV)
    out_buf = torch.full((f, d + 7), -7.0, dtype=torch.float32, device=DEV)
    out = out_buf[:, 3:3 + d]                       # rows 12 bytes off, leading dimension d + 7: 32-bit stores do not mind
    bz.vote(buf[:, :, 4:4 + d], out)
    assert bz.last_path() == bz.PATH_STAGED
    assert np.array_equal(_bits(out), _bits(oracle.vote(rep)))
    assert (out_buf[:, :3] == -7.0).all() and (out_buf[:, 3 + d:] == -7.0).all()
    # the register kernel on request
    monkeypatch.setenv("BZ_VOTE_PATH", "registers")
    got = bz.vote(torch.from_numpy(rep).to(DEV))
    assert bz.last_path() == bz.PATH_REGISTERS and np.array_equal(_bits(got), _bits(oracle.vote(rep)))
    # by default: the register kernel for an input this small, the staged one from ~100 MB of replicas up
    monkeypatch.delenv("BZ_VOTE_PATH")
    bz.vote(torch.from_numpy(rep).to(DEV))
    assert bz.last_path() == bz.PATH_REGISTERS
    if kind == "ties":
        d_big = (128 * 1024 * 1024) // (4 * r * f) // 128 * 128 + 128
        big = torch.from_numpy(rng.integers(0, 3, size=(r, f, d_big)).astype(np.float32))
        got = bz.vote(big.to(DEV))
        assert bz.last_path() == bz.PATH_STAGED
        sample = np.concatenate([np.arange(0, 300), np.arange(d_big - 300, d_big), rng.integers(0, d_big, 5000)])
        assert np.array_equal(_bits(got[:, sample]), _bits(oracle.vote(big[:, :, sample].numpy())))


@pytest.mark.parametrize("f", [25, 49])
def test_median_of_given_rows_on_the_staged_kernel(f):
    # Gaussian rows with a block of rounded values (many equal keys), at a size with many tiles per CTA
    d = 600_004
    v = torch.from_numpy(np.random.default_rng(f).standard_normal((f, d)).astype(np.float32))
    v[:, :4096] = torch.round(v[:, :4096])
    got = bz.median(v.to(DEV))
    assert bz.last_path() == bz.PATH_STAGED
    assert np.array_equal(_bits(got), _bits(oracle.median(v.numpy())))
    # an odd size takes the register kernels and must agree
    got = bz.median(v[:, :d - 1].to(DEV))
    assert bz.last_path() == bz.PATH_REGISTERS
    assert np.array_equal(_bits(got), _bits(oracle.median(v[:, :d - 1].contiguous().numpy())))


def test_empty_input():
    rep = torch.zeros((3, 25, 0), dtype=torch.float32, device=DEV)
    assert bz.vote_median(rep).numel() == 0
    assert bz.vote(rep).shape == (25, 0)


def test_host_entry_point():
    rep = _cluster(5, 3, 3, 200003, "reversed", seed=4)
    want = oracle.vote_median(rep.numpy())
    pinned = rep.pin_memory()
    out = torch.empty(200003, dtype=torch.float32).pin_memory()
    small = bz.alloc_workspace(bz.OP_VOTE_MEDIAN_HOST, 3, 25, 200003)       # several slabs
    bz.vote_median_host(pinned, out, small)
    assert np.array_equal(_bits(out), _bits(want))
    out.zero_()
    whole = torch.empty(76 * 200064 * 4 + 256, dtype=torch.uint8, device=DEV)  # one slab
    bz.vote_median_host(pinned, out, whole)
    assert np.array_equal(_bits(out), _bits(want))
    out2 = torch.empty(200003, dtype=torch.float32)
    bz.vote_median_host(rep, out2, small)                                    # pageable memory also works
    assert np.array_equal(_bits(out2), _bits(want))


_REGISTER_PATH_SCRIPT = r"""
import numpy as np, torch, oracle
from paper_2010_04902_b200 import binding as bz, inputs
n0 = bz.kernel_launch_count()
for (l, r, q, attack, d) in [(5, 3, 3, "reversed", 70001), (7, 3, 5, "alie", 33333), (5, 5, 6, "constant", 20480),
                             (7, 7, 5, "reversed", 9999)]:
    wf, fw, _ = oracle.assign(l, r)
    byz = oracle.worst_case(wf, l * l, r, q)[1]
    rep = inputs.build_replicas(inputs.true_gradients(l * l, d, seed=2), fw, byz, attack)
    got = bz.vote_median(rep.cuda()).cpu().numpy()
    assert np.array_equal(got.view(np.uint32), oracle.vote_median(rep.numpy()).view(np.uint32)), (l, r)
assert bz.pipeline_timeouts() == 0
print("register path ok", bz.kernel_launch_count() - n0)
"""


def test_register_path_at_sizes_the_staged_path_normally_takes():
    # the fused pass has two implementations; the environment switch pins the register one
    import os
    import subprocess
    import sys
    from conftest import ROOT
    env = dict(os.environ, BZ_VOTE_MEDIAN_PATH="registers", PYTHONPATH=ROOT)
    res = subprocess.run([sys.executable, "-c", _REGISTER_PATH_SCRIPT], env=env, cwd=ROOT, capture_output=True, text=True)
    assert res.returncode == 0 and "register path ok" in res.stdout, res.stdout + res.stderr


def _sampled_columns(d, n, rng):
    return np.unique(np.concatenate([np.arange(0, 600), np.arange(d - 600, d), rng.integers(0, d, size=n)]))


@pytest.mark.parametrize("l,r,q,attack,d", [(5, 3, 3, "reversed", 11_200_000), (7, 3, 5, "alie", 11_200_000)])
def test_full_size_sampled_columns(l, r, q, attack, d):
    # benchmark-size input in the benchmark's launch configuration; the oracle recomputes a sample
    # of coordinates (both ends and 20000 random ones) one by one
    wf, fw, _ = oracle.assign(l, r)
    byz = oracle.worst_case(wf, l * l, r, q)[1]
    g = inputs.true_gradients(l * l, d, seed=0, device=DEV)
    rep = inputs.build_replicas(g, fw, byz, attack)
    out = bz.vote_median(rep)
    torch.cuda.synchronize()
    idx = _sampled_columns(d, 20000, np.random.default_rng(0))
    idx_dev = torch.from_numpy(idx).to(DEV)
    cols = rep[:, :, idx_dev].cpu()
    want = oracle.vote_median(cols.numpy())
    assert np.array_equal(_bits(out[idx_dev]), _bits(want))
    # a property that holds at every coordinate: with fewer than f/2 distorted files the median
    # lies inside the honest range
    byz_set = set(byz.tolist())
    bad = torch.tensor([sum(1 for u in fw[i] if int(u) in byz_set) >= (r + 1) // 2 for i in range(l * l)])
    honest = g[(~bad).to(DEV)]
    assert bool((out >= honest.min(dim=0).values).all()) and bool((out <= honest.max(dim=0).values).all())
