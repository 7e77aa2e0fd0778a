"""bz_pairdist_static: the distance matrix for callers that cannot allocate device memory.

Some users of the library run where cudaMalloc is off limits: an operator inside a framework whose
memory plan was fixed before the run, a latency-bound loop that cannot risk the device-wide stall an
allocation may bring, a job held to a fixed memory budget on a shared GPU.  The entry point tested here
gives them the pairwise distances with the scratch taken from a 4 MiB array that is part of the library
itself; they hand in inputs and outputs only.

The file sorts last so that a run stopping at the first failure has already executed every other test.
It must pass on its own in a fresh process as well as after the rest of the suite.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2010_04902_b200 import binding as bz
from paper_2010_04902_b200 import inputs

pytestmark = pytest.mark.gpu

DEV = "cuda"
DIST_TOL = 1e-7   # the relative tolerance the distance tests use


SHORT_TOL = 2e-6  # rows of a few hundred to a few thousand coordinates: few binary32 blocks, their rounding does not average out


def _close(got, want, tol=DIST_TOL):
    got = got.cpu().numpy()
    want = want.cpu().numpy() if isinstance(want, torch.Tensor) else want
    assert np.array_equal(got, got.T) and (np.diag(got) == 0).all()
    assert (np.abs(got - want) <= tol * np.abs(want)).all()


def _free_bytes():
    torch.cuda.synchronize()
    return torch.cuda.mem_get_info()[0]


def test_two_calls_in_a_row_match_the_workspace_entry_point():
    # first call: f = 25 (register-tiled kernel), many tiles, ragged tail
    v1 = inputs.true_gradients(25, 300_003, seed=21).to(DEV)
    want1 = bz.pairdist(v1)
    got1 = torch.empty((25, 25), dtype=torch.float64, device=DEV)     # outputs exist before the call
    # second call, straight after, on a much smaller input: fewer CTAs write the shared array, so
    # anything the first call left behind must not leak into the result
    v2 = inputs.integer_gradients(25, 517, seed=22).to(DEV)
    want2 = bz.pairdist(v2)
    got2 = torch.empty((25, 25), dtype=torch.float64, device=DEV)
    warm = torch.empty((25, 25), dtype=torch.float64, device=DEV)
    bz.pairdist_static(v1, warm)                                      # the device's first call resolves the array's address
    bz.pairdist_static(v2, warm)                                      # (and the runtime has loaded both kernels' code)
    before_torch, before_free = torch.cuda.memory_allocated(), _free_bytes()
    bz.pairdist_static(v1, got1)
    bz.pairdist_static(v2, got2)
    # neither through torch's allocator nor behind its back: the device's free memory is what it was
    assert torch.cuda.memory_allocated() == before_torch and _free_bytes() == before_free
    _close(got1, want1)
    _close(got2, want2)
    assert torch.equal(got2, want2)                                   # integer rows: exact on both paths
    # and against the CPU oracle, not only against the library's other entry point
    _close(got1, oracle.pairdist(v1.cpu().numpy()))
    assert np.array_equal(got2.cpu().numpy(), oracle.pairdist(v2.cpu().numpy()))


def test_other_shapes_and_a_third_call():
    # generic kernel (f = 9 and the largest f that fits), unaligned rows, then f = 25 again
    for f, d in [(9, 4001), (84, 700), (49, 30_001)]:
        v = inputs.true_gradients(f, d, seed=f).to(DEV)
        got = torch.empty((f, f), dtype=torch.float64, device=DEV)
        bz.pairdist_static(v, got)
        _close(got, bz.pairdist(v))
        _close(got, oracle.pairdist(v.cpu().numpy()), DIST_TOL if d >= 30_000 else SHORT_TOL)
    buf = torch.zeros((25, 2100), dtype=torch.float32, device=DEV)
    buf[:, 1:2002] = inputs.true_gradients(25, 2001, seed=5).to(DEV)
    got = torch.empty((25, 25), dtype=torch.float64, device=DEV)
    bz.pairdist_static(buf[:, 1:2002], got)
    _close(got, bz.pairdist(buf[:, 1:2002]))
    v = inputs.true_gradients(25, 70_000, seed=6).to(DEV)
    bz.pairdist_static(v, got)
    _close(got, bz.pairdist(v))


def test_shapes_beyond_the_built_in_scratch_are_refused():
    for f in (85, 100, 121):
        v = torch.zeros((f, 64), dtype=torch.float32, device=DEV)
        out = torch.full((f, f), -1.0, dtype=torch.float64, device=DEV)
        assert bz.workspace_bytes(bz.OP_PAIRDIST, 0, f, 64) > bz.STATIC_SCRATCH_BYTES
        with pytest.raises(bz.BzError) as e:
            bz.pairdist_static(v, out)
        assert e.value.status == bz.ERR_STATIC_LIMIT
        assert "built-in" in str(e.value)
        assert bool((out == -1.0).all())                              # refused before anything ran
    assert bz.workspace_bytes(bz.OP_PAIRDIST, 0, 25, 64) <= bz.STATIC_SCRATCH_BYTES
    assert bz.workspace_bytes(bz.OP_PAIRDIST, 0, 84, 64) <= bz.STATIC_SCRATCH_BYTES
