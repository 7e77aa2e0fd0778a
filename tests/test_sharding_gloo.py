"""The multi-rank path on CPU: two gloo ranks, each aggregating its coordinate slab with the CPU
checker standing in for the per-rank kernels, must reproduce the single-rank result - no exchange
for vote/median, one all-reduce of the distance matrix for the Krum family."""
import os
import socket
import types

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2010_04902_b200 import inputs, sharding


def test_coordinate_slabs_partition_the_range():
    for d in [0, 1, 3, 4, 5, 1000, 1001, 11_200_000, 11_173_962]:
        for world in [1, 2, 3, 4, 8]:
            ends = [sharding.coordinate_slab(d, rk, world) for rk in range(world)]
            assert ends[0][0] == 0 and ends[-1][1] == d
            for (a0, a1), (b0, b1) in zip(ends, ends[1:]):
                assert a1 == b0 and a0 <= a1
            for a0, a1 in ends:
                assert a0 % 4 == 0 or a0 == d
            sizes = [b - a for a, b in ends]
            assert max(sizes) - min(sizes) < 8
    with pytest.raises(ValueError):
        sharding.coordinate_slab(10, 2, 2)


def _oracle_ops():
    """Per-rank operations backed by the CPU checker, with the binding's signatures."""
    t = torch.from_numpy
    return types.SimpleNamespace(
        vote_median=lambda rep: t(oracle.vote_median(rep.numpy())),
        pairdist=lambda v: t(oracle.pairdist(v.numpy())),
        krum_select=lambda D, c, m: t(oracle.multikrum_select(D.numpy(), c, m)),
        mean_rows=lambda v, sel: t(oracle.mean_rows(v.numpy(), sel.numpy())),
        bulyan_select=lambda D, c: t(oracle.bulyan_select(D.numpy(), c)),
        trimmed_mean=lambda v, sel, beta: t(oracle.trimmed_mean(v.numpy(), sel.numpy(), beta)),
    )


def _recording_ops(calls):
    """The same stand-ins, but every call is first bound against the CUDA binding's own signature (so the
    arguments the sharding layer passes are the ones the default `ops=None` wiring would hand to the kernels)
    and its name is recorded."""
    import inspect
    from paper_2010_04902_b200 import binding
    base = _oracle_ops()
    base.vote_pairdist = lambda rep: (lambda v: (torch.from_numpy(v), torch.from_numpy(oracle.pairdist(v))))(oracle.vote(rep.numpy()))

    def wrap(name):
        fn = getattr(base, name)
        sig = inspect.signature(getattr(binding, name))

        def call(*a, **kw):
            sig.bind(*a, **kw)
            calls.append(name)
            return fn(*a, **kw)
        return call
    return types.SimpleNamespace(**{n: wrap(n) for n in ("vote_median", "pairdist", "vote_pairdist", "krum_select", "mean_rows",
                                                         "bulyan_select", "trimmed_mean")})


def test_default_ops_is_the_cuda_binding():
    from paper_2010_04902_b200 import binding
    ops = sharding._ops(None)
    assert ops is binding
    for name in ("vote_median", "pairdist", "vote_pairdist", "krum_select", "mean_rows", "bulyan_select", "trimmed_mean"):
        assert callable(getattr(ops, name))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, d, ret):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        ops = _oracle_ops()
        wf, fw, _ = oracle.assign(5, 3)
        _, byz, _ = oracle.worst_case(wf, 25, 3, 3)
        g = inputs.true_gradients(25, d, seed=0)
        rep = inputs.build_replicas(g, fw, byz, "reversed")
        j0, j1 = sharding.coordinate_slab(d, rank, world)
        rep_slab = rep[:, :, j0:j1].contiguous()
        med = sharding.vote_median(rep_slab, ops=ops)
        voted_slab = torch.from_numpy(oracle.vote(rep_slab.numpy()))
        mk_out, mk_sel, D = sharding.multikrum(voted_slab, 3, 22, ops=ops)
        bu_out, bu_sel, _ = sharding.bulyan(voted_slab, 3, ops=ops)
        # the single-pass forms, through stand-ins that check the binding's signatures and record the order
        calls = []
        rec = _recording_ops(calls)
        v_out, v_sel, v_D, v_voted = sharding.vote_multikrum(rep_slab, 3, 22, ops=rec)
        order_mk = list(calls)
        del calls[:]
        b_out, b_sel, _, _ = sharding.vote_bulyan(rep_slab, 3, ops=rec)
        order_bu = list(calls)
        assert order_mk == ["vote_pairdist", "krum_select", "mean_rows"]
        assert order_bu == ["vote_pairdist", "bulyan_select", "trimmed_mean"]
        assert torch.equal(v_voted, voted_slab) and torch.equal(v_sel, mk_sel) and torch.equal(v_out, mk_out)
        assert torch.equal(v_D, D) and torch.equal(b_sel, bu_sel) and torch.equal(b_out, bu_out)
        ret[rank] = dict(j=(j0, j1), med=med.numpy(), mk_out=mk_out.numpy(), mk_sel=mk_sel.numpy(), D=D.numpy(),
                         bu_out=bu_out.numpy(), bu_sel=bu_sel.numpy())
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("d", [4001, 1026])
def test_two_ranks_reproduce_the_single_rank_result(d):
    world = 2
    ctx = mp.get_context("spawn")
    mgr = ctx.Manager()
    ret = mgr.dict()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(rk, world, port, d, ret)) for rk in range(world)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(180)
        assert p.exitcode == 0
    wf, fw, _ = oracle.assign(5, 3)
    _, byz, _ = oracle.worst_case(wf, 25, 3, 3)
    g = inputs.true_gradients(25, d, seed=0)
    rep = inputs.build_replicas(g, fw, byz, "reversed").numpy()
    voted = oracle.vote(rep)
    want_med = oracle.median(voted)
    want_mk, want_mk_sel, want_D = oracle.multikrum(voted, 3, 22)
    want_bu, want_bu_sel, _ = oracle.bulyan(voted, 3)
    parts = [ret[rk] for rk in range(world)]
    assert parts[0]["j"][1] == parts[1]["j"][0] and parts[1]["j"][1] == d
    assert np.array_equal(np.concatenate([p["med"] for p in parts]).view(np.uint32), want_med.view(np.uint32))
    for p in parts:
        assert np.allclose(p["D"], want_D, rtol=1e-12, atol=0)           # summed in two pieces
        assert p["mk_sel"].tolist() == want_mk_sel.tolist() and p["bu_sel"].tolist() == want_bu_sel.tolist()
    assert np.array_equal(np.concatenate([p["mk_out"] for p in parts]), want_mk)
    assert np.array_equal(np.concatenate([p["bu_out"] for p in parts]), want_bu)


# ---- the exhaustive worst-case search dealt to the ranks ------------------------------------------------

def _brute_force_part(worker_files, f, r, q, part, parts):
    """A stand-in for bz_worst_case_part with its signature: every q-subset in lexicographic order, subset number n
    going to share n % parts; returns (c_max, argmax, n_subsets) of the share, c_max = -1 if it is empty."""
    import itertools
    K = len(worker_files)
    need = (r + 1) // 2
    best, best_set, n = -1, [0] * q, 0
    for n, S in enumerate(itertools.combinations(range(K), q)):
        if n % parts != part:
            continue
        holders = np.zeros(f, np.int64)
        for u in S:
            holders[list(worker_files[u])] += 1
        c = int((holders >= need).sum())
        if c > best:
            best, best_set = c, list(S)
    return best, np.array(best_set, np.int32), n + 1


def test_best_of_shares_rules():
    assert sharding.best_of_shares([(3, [0, 5, 9]), (4, [1, 2, 3]), (-1, [0, 0, 0])]) == (4, [1, 2, 3])
    assert sharding.best_of_shares([(4, [1, 2, 4]), (4, [1, 2, 3]), (4, [2, 3, 4])]) == (4, [1, 2, 3])   # first in lexicographic order
    assert sharding.best_of_shares([(-1, [0]), (0, [7])]) == (0, [7])
    with pytest.raises(ValueError):
        sharding.best_of_shares([(-1, [0]), (-1, [0])])


def test_shares_of_the_search_combine_to_the_whole():
    wf, _, _ = oracle.assign(5, 3)
    for q in (1, 2, 3, 4):
        want_c, want_set, _ = oracle.worst_case(wf, 25, 3, q)
        for parts in (1, 2, 3, 7, 40):     # q = 1 has 15 subsets: with 40 shares most are empty
            shares = [_brute_force_part(wf, 25, 3, q, p, parts)[:2] for p in range(parts)]
            assert sharding.best_of_shares(shares) == (want_c, [int(u) for u in want_set])
            if q == 1 and parts == 40:
                assert sum(c < 0 for c, _ in shares) == 25


def _wc_worker(rank, world, port, ret):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        import inspect
        from paper_2010_04902_b200 import binding
        wf, _, _ = oracle.assign(5, 3)
        sig = inspect.signature(binding.worst_case_part)

        def part(mask, f, r, q, p, parts, max_subsets=0):
            sig.bind(mask, f, r, q, p, parts, max_subsets)      # what the default wiring would hand to the binding
            assert (p, parts) == (rank, world)
            return _brute_force_part(wf, f, r, q, p, parts)
        ops = types.SimpleNamespace(worst_case_part=part)
        ret[rank] = [sharding.worst_case(None, 25, 3, q, ops=ops) for q in (2, 3, 4)]
    finally:
        dist.destroy_process_group()


def test_two_ranks_share_the_worst_case_search():
    world = 2
    ctx = mp.get_context("spawn")
    ret = ctx.Manager().dict()
    port = _free_port()
    procs = [ctx.Process(target=_wc_worker, args=(rk, world, port, ret)) for rk in range(world)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(180)
        assert p.exitcode == 0
    wf, _, _ = oracle.assign(5, 3)
    for k, q in enumerate((2, 3, 4)):
        want_c, want_set, want_n = oracle.worst_case(wf, 25, 3, q)
        for rk in range(world):
            c, arg, n = ret[rk][k]
            assert (c, arg, n) == (want_c, [int(u) for u in want_set], want_n)
