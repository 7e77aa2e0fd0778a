"""GPU parity for gradients kept in the workers' own buffers (a table of row pointers instead of one
strided array): vote and fused vote + median, bit-exact against the CPU oracle."""
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


def _worker_buffers(rep, wf, fw, pad=0, shift=0):
    """What each worker sent: buffer u holds the copies of worker u's files, in the order of wf[u].
    pad / shift give rows that are padded or start at an odd element (unaligned)."""
    r, f, d = rep.shape
    K, l = wf.shape
    bufs = []
    for u in range(K):
        k = u // l
        buf = torch.zeros((l, d + pad + shift), dtype=torch.float32, device=DEV)
        for slot, i in enumerate(wf[u]):
            assert int(fw[int(i)][k]) == u
            buf[slot, shift:shift + d] = rep[k, int(i)].to(DEV)
        bufs.append(buf[:, shift:shift + d])
    return bufs


@pytest.mark.parametrize("l,r,q,attack,d,pad,shift", [
    (5, 3, 3, "reversed", 40_000, 0, 0), (7, 3, 5, "alie", 30_001, 3, 0), (5, 5, 6, "constant", 20_002, 0, 1),
    (7, 5, 5, "independent", 8_003, 5, 0), (7, 7, 4, "reversed", 4_000, 0, 0), (3, 3, 2, "alie", 1_001, 0, 0),
    (4, 3, 3, "alie", 5_000, 0, 0)])
def test_vote_and_median_from_worker_buffers(l, r, q, attack, d, pad, shift):
    wf, fw, _ = oracle.assign(l, r)
    byz = oracle.worst_case(wf, l * l, r, q)[1]
    g = inputs.true_gradients(l * l, d, seed=l + r)
    rep = inputs.build_replicas(g, fw, byz, attack)
    bufs = _worker_buffers(rep, wf, fw, pad, shift)
    table = bz.row_table(bufs, fw, wf)
    want_voted = oracle.vote(rep.numpy())
    want_med = oracle.median(want_voted)
    assert np.array_equal(_bits(bz.vote_median_rows(table, r, l * l, d)), _bits(want_med))
    assert np.array_equal(_bits(bz.vote_rows(table, r, l * l, d)), _bits(want_voted))
    # an unaligned output takes the scalar kernel as well
    out = torch.zeros(d + 1, dtype=torch.float32, device=DEV)
    bz.vote_median_rows(table, r, l * l, d, out[1:])
    assert np.array_equal(_bits(out[1:]), _bits(want_med))


def test_full_size_from_worker_buffers():
    # the benchmark's cluster (K = 15, r = 3, f = 25, d = 11.2 M): same result as the strided kernel,
    # which is itself checked against the oracle, and sampled columns against the oracle directly
    l, r, q, d = 5, 3, 3, 11_200_000
    wf, fw, _ = oracle.assign(l, r)
    byz = oracle.worst_case(wf, l * l, r, q)[1]
    g = inputs.true_gradients(l * l, d, seed=0, device=DEV)
    rep = inputs.build_replicas(g, fw, byz, "reversed")
    del g
    bufs = []
    for u in range(l * r):
        bufs.append(torch.stack([rep[u // l, int(i)] for i in wf[u]]))
    table = bz.row_table(bufs, fw, wf)
    out = bz.vote_median_rows(table, r, l * l, d)
    assert torch.equal(out.view(torch.int32), bz.vote_median(rep).view(torch.int32))
    idx = torch.from_numpy(np.unique(np.concatenate([np.arange(0, 128), np.arange(d - 128, d),
                                                     np.random.default_rng(1).integers(0, d, 20000)]))).to(DEV)
    assert np.array_equal(_bits(out[idx]), _bits(oracle.vote_median(rep[:, :, idx].cpu().numpy())))
    ms = []
    for fn in (lambda: bz.vote_median_rows(table, r, l * l, d, out), lambda: bz.vote_median(rep, out)):
        for _ in range(3):
            fn()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(10):
            fn()
        e1.record()
        torch.cuda.synchronize()
        ms.append(e0.elapsed_time(e1) / 10)
    print("vote+median from worker buffers %.3f ms, strided %.3f ms" % tuple(ms))
