"""The coordinate-sharded Krum family with the CUDA binding as the per-rank operations (the default wiring of
sharding.py): two ranks, each on its own slab of the replicas, one all-reduce of the distance matrix.

Both ranks run on the one GPU this test gets and exchange the 49 x 49 matrix through gloo (NCCL refuses two ranks
on one device); nothing on the device waits for the other rank - each rank's kernels are ordinary launches and the
exchange is a host-side collective between them - so sharing the GPU is safe.  The multi-GPU run differs only in
the backend."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.multiprocessing as mp

import oracle
from paper_2010_04902_b200 import inputs

pytestmark = pytest.mark.gpu


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _rank(rank, world, port, l, r, q, d, c, ret):
    import torch.distributed as dist

    from paper_2010_04902_b200 import binding as bz
    from paper_2010_04902_b200 import sharding
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    torch.cuda.set_device(0)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        f = l * l
        wf, fw, _ = oracle.assign(l, r)
        byz = oracle.worst_case(wf, f, r, q)[1]
        rep = inputs.build_replicas(inputs.true_gradients(f, d, seed=3), fw, byz, "alie")
        j0, j1 = sharding.coordinate_slab(d, rank, world)
        slab = rep[:, :, j0:j1].cuda()                 # a view with the full rows' leading dimensions would do as well
        before = bz.pipeline_timeouts()
        out, sel, D, voted = sharding.vote_multikrum(slab, c, f - c)
        path_mk = bz.last_path()
        b_out, b_sel, _, _ = sharding.vote_bulyan(slab, min(c, (f - 3) // 4))
        med = sharding.vote_median(slab)
        _, _, mask = bz.assign_mols(l, r)
        wc = [sharding.worst_case(mask, f, r, qq) for qq in (2, q)]    # the exhaustive search, dealt to the two ranks
        torch.cuda.synchronize()
        ret[rank] = dict(j=(j0, j1), out=out.cpu().numpy(), sel=sel.cpu().numpy(), D=D.cpu().numpy(),
                         voted=voted.cpu().numpy(), b_out=b_out.cpu().numpy(), b_sel=b_sel.cpu().numpy(),
                         med=med.cpu().numpy(), timeouts=bz.pipeline_timeouts() - before, path=path_mk, wc=wc)
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("l,r,q,d,c", [(7, 3, 5, 200_008, 8), (5, 5, 6, 120_000, 4)])
def test_two_ranks_with_the_cuda_binding(l, r, q, d, c):
    world = 2
    ctx = mp.get_context("spawn")
    mgr = ctx.Manager()
    ret = mgr.dict()
    port = _free_port()
    procs = [ctx.Process(target=_rank, args=(rk, world, port, l, r, q, d, c, ret)) for rk in range(world)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(300)
        assert p.exitcode == 0
    f = l * l
    wf, fw, _ = oracle.assign(l, r)
    byz = oracle.worst_case(wf, f, r, q)[1]
    rep = inputs.build_replicas(inputs.true_gradients(f, d, seed=3), fw, byz, "alie").numpy()
    voted = oracle.vote(rep)
    want_out, want_sel, want_D = oracle.multikrum(voted, c, f - c)
    cb = min(c, (f - 3) // 4)
    want_b, want_bsel, _ = oracle.bulyan(voted, cb)
    want_med = oracle.median(voted)
    parts = [ret[rk] for rk in range(world)]
    assert parts[0]["j"] == (0, parts[1]["j"][0]) and parts[1]["j"][1] == d
    from paper_2010_04902_b200 import binding as bz
    for p in parts:
        assert p["timeouts"] == 0 and p["path"] == bz.PATH_TENSOR      # slabs of 100 000 and 60 000 coordinates: the integer kernel
        assert p["sel"].tolist() == want_sel.tolist() and p["b_sel"].tolist() == want_bsel.tolist()
        nz = want_D > 0
        assert (np.abs(p["D"][nz] - want_D[nz]) <= 1e-7 * want_D[nz]).all() and (p["D"][~nz] == 0).all()
    for k, qq in enumerate((2, q)):
        want_c, want_set, want_n = oracle.worst_case(wf, f, r, qq)
        for p in parts:
            assert p["wc"][k] == (want_c, want_set.tolist(), want_n)
    for key, want in (("voted", voted), ("out", want_out), ("b_out", want_b), ("med", want_med)):
        got = np.concatenate([p[key] for p in parts], axis=-1)
        assert np.array_equal(got.view(np.uint32), np.ascontiguousarray(want).view(np.uint32)), key
