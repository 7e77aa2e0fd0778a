"""The C-ABI library loads, exports every symbol include/bz.h declares, and its host-side logic
(assignment, validation, workspace sizes, status strings) behaves as the header states.
No kernel is launched here: every call returns from host-side validation."""
import ctypes
import os
import re
import subprocess
import sys

import numpy as np
import pytest

import oracle
from conftest import ROOT, read_golden_rows
from paper_2010_04902_b200 import binding as bz
from paper_2010_04902_b200 import build as bz_build


@pytest.fixture(scope="module")
def lib():
    bz_build.build()
    return bz.lib()


def _declared():
    text = open(os.path.join(ROOT, "include", "bz.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(bz_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared()
    assert len(names) >= 17
    for name in names:
        assert hasattr(lib, name), name
    assert sorted(bz.EXPORTS) == names


def test_status_strings(lib):
    seen = set()
    for code in range(0, -7, -1):
        s = bz.status_string(code)
        assert s and s != "unknown status"
        seen.add(s)
    assert len(seen) == 7
    assert bz.status_string(-99) == "unknown status"
    assert bz.last_cuda_error() == ""


def test_assign_matches_printed_table_and_oracle(lib):
    wf, fw, mask = bz.assign_mols(5, 3)
    for row in read_golden_rows("assignment_l5_r3.txt"):
        assert list(wf[int(row[0])]) == [int(x) for x in row[1:]]
    # primes, and prime powers over F_l (the library and the checker build the field in different ways)
    for l, r in [(3, 2), (5, 3), (5, 5), (7, 3), (7, 5), (7, 7), (11, 4), (13, 13),
                 (4, 3), (8, 3), (8, 7), (9, 5), (16, 15), (25, 4), (27, 3), (32, 5), (49, 2), (81, 3)]:
        wf, fw, mask = bz.assign_mols(l, r)
        owf, ofw, omask = oracle.assign(l, r)
        assert np.array_equal(wf, owf) and np.array_equal(fw, ofw)
        if l * l <= 64:
            assert np.array_equal(mask, omask)
        else:
            assert mask is None


@pytest.mark.parametrize("l,r", [(4, 4), (6, 3), (9, 9), (10, 2), (2048, 3), (5, 6), (5, 7), (5, 0), (1, 1), (0, 0), (-3, 1)])
def test_assign_rejects(lib, l, r):
    with pytest.raises(bz.BzError) as e:
        bz.assign_mols(l, r)
    assert e.value.status == bz.ERR_INVALID_ARG


def test_assign_mask_needs_at_most_64_files(lib):
    buf = np.zeros(11 * 4, np.uint64)
    assert lib.bz_assign_mols(11, 4, None, None, buf.ctypes.data) == bz.ERR_INVALID_ARG
    assert lib.bz_assign_mols(11, 4, None, None, None) == bz.OK


def test_workspace_sizes(lib):
    for f in (9, 25, 49, 121):
        pd = bz.workspace_bytes(bz.OP_PAIRDIST, 0, f, 1000)
        mk = bz.workspace_bytes(bz.OP_MULTIKRUM, 0, f, 1000, 2, 3)
        bu = bz.workspace_bytes(bz.OP_BULYAN, 0, f, 1000, 1)
        assert pd > 0 and pd % 256 == 0 and mk >= pd + f * f * 8 and bu == mk
    assert bz.workspace_bytes(bz.OP_WORST_CASE, 3, 25) > 0
    assert bz.workspace_bytes(bz.OP_VOTE_VECTORWISE, 3, 25, 1000) >= 25 * 20
    small = bz.workspace_bytes(bz.OP_VOTE_MEDIAN_HOST, 3, 25, 1000)
    big = bz.workspace_bytes(bz.OP_VOTE_MEDIAN_HOST, 3, 25, 10 ** 7)
    assert 76 * 1000 * 4 <= small <= big <= 76 * 65536 * 4 + 256
    assert bz.workspace_bytes(99, 3, 25, 1000) == 0 and bz.workspace_bytes(bz.OP_PAIRDIST, 0, 500, 10) == 0


def test_validation_runs_before_any_launch(lib):
    n0 = bz.kernel_launch_count()
    fake = ctypes.c_void_p(256)  # never dereferenced: each call below fails validation first
    L = lib
    # vote / median family
    assert L.bz_vote_median(None, 3, 25, 10, 10, 250, fake, None) == bz.ERR_INVALID_ARG
    assert L.bz_vote_median(fake, 4, 25, 10, 10, 250, fake, None) == bz.ERR_INVALID_ARG      # r even
    assert L.bz_vote_median(fake, 3, 25, -1, 10, 250, fake, None) == bz.ERR_INVALID_ARG
    assert L.bz_vote_median(fake, 3, 25, 10, 9, 250, fake, None) == bz.ERR_INVALID_ARG       # ld_file < d
    assert L.bz_vote_median(fake, 3, 25, 10, 10, 5, fake, None) == bz.ERR_INVALID_ARG        # ld_replica < d
    assert L.bz_vote_median(fake, 17, 25, 10, 10, 250, fake, None) == bz.ERR_UNSUPPORTED
    assert L.bz_vote_median(fake, 3, 129, 10, 10, 2000, fake, None) == bz.ERR_UNSUPPORTED
    assert L.bz_vote_median(fake, 3, 25, 10, 10, 250, None, None) == bz.ERR_INVALID_ARG
    assert L.bz_vote_median(fake, 3, 25, 0, 0, 0, fake, None) == bz.OK                       # d == 0: no-op
    assert L.bz_vote(fake, 3, 25, 10, 10, 250, None, 10, None) == bz.ERR_INVALID_ARG
    assert L.bz_vote(fake, 3, 25, 10, 10, 250, fake, 9, None) == bz.ERR_INVALID_ARG
    assert L.bz_vote(fake, 3, 25, 0, 0, 0, fake, 0, None) == bz.OK
    # whole-vector vote: bz_vote's rules, then its outputs and workspace
    assert L.bz_vote_vectorwise(None, 3, 25, 10, 10, 250, fake, 10, fake, fake, 1 << 20, None) == bz.ERR_INVALID_ARG
    assert L.bz_vote_vectorwise(fake, 4, 25, 10, 10, 250, fake, 10, fake, fake, 1 << 20, None) == bz.ERR_INVALID_ARG
    assert L.bz_vote_vectorwise(fake, 17, 25, 10, 10, 250, fake, 10, fake, fake, 1 << 20, None) == bz.ERR_UNSUPPORTED
    assert L.bz_vote_vectorwise(fake, 3, 25, 10, 10, 5, fake, 10, fake, fake, 1 << 20, None) == bz.ERR_INVALID_ARG
    assert L.bz_vote_vectorwise(fake, 3, 25, 10, 10, 250, None, 10, None, fake, 1 << 20, None) == bz.ERR_INVALID_ARG   # no output
    assert L.bz_vote_vectorwise(fake, 3, 25, 10, 10, 250, fake, 9, fake, fake, 1 << 20, None) == bz.ERR_INVALID_ARG    # ld_voted < d
    assert L.bz_vote_vectorwise(fake, 3, 25, 10, 10, 250, fake, 10, fake, None, 1 << 20, None) == bz.ERR_WORKSPACE
    assert L.bz_vote_vectorwise(fake, 3, 25, 10, 10, 250, fake, 10, fake, fake, 16, None) == bz.ERR_WORKSPACE
    assert L.bz_vote_vectorwise(fake, 3, 25, 10, 10, 250, fake, 10, fake, ctypes.c_void_p(264), 1 << 20, None) == bz.ERR_WORKSPACE
    assert L.bz_vote_clusters(fake, 3, 25, 10, 10, 250, -1.0, 0.0, fake, 10, fake, fake, 1 << 20, None) == bz.ERR_INVALID_ARG
    assert L.bz_vote_clusters(fake, 3, 25, 10, 10, 250, 0.0, float('nan'), fake, 10, fake, fake, 1 << 20, None) == bz.ERR_INVALID_ARG
    assert L.bz_vote_clusters(fake, 3, 25, 10, 10, 250, 0.0, 1e-6, fake, 10, fake, None, 0, None) == bz.ERR_WORKSPACE
    assert L.bz_vote_median_rows(None, 3, 25, 10, fake, None) == bz.ERR_INVALID_ARG
    assert L.bz_vote_median_rows(fake, 2, 25, 10, fake, None) == bz.ERR_INVALID_ARG
    assert L.bz_vote_median_rows(fake, 3, 25, 10, None, None) == bz.ERR_INVALID_ARG
    assert L.bz_vote_median_rows(fake, 3, 200, 10, fake, None) == bz.ERR_UNSUPPORTED
    assert L.bz_vote_median_rows(fake, 3, 25, 0, None, None) == bz.OK
    assert L.bz_vote_rows(fake, 3, 25, 10, fake, 9, None) == bz.ERR_INVALID_ARG
    assert L.bz_vote_rows(fake, 3, 25, 10, None, 10, None) == bz.ERR_INVALID_ARG
    assert L.bz_median(None, 25, 10, 10, fake, None) == bz.ERR_INVALID_ARG
    assert L.bz_median(fake, 0, 10, 10, fake, None) == bz.ERR_INVALID_ARG
    assert L.bz_median(fake, 25, 0, 0, fake, None) == bz.OK
    assert L.bz_vote_median_host(fake, 3, 25, 10, fake, None, 0, None) == bz.ERR_WORKSPACE
    assert L.bz_vote_median_host(fake, 3, 25, 10, fake, ctypes.c_void_p(264), 1 << 30, None) == bz.ERR_WORKSPACE
    assert L.bz_vote_median_host(fake, 3, 25, 10, fake, fake, 16, None) == bz.ERR_WORKSPACE
    # Krum family: the operand requirements of Sec. 6.1
    assert L.bz_krum_select(fake, 7, 3, 1, fake, None) == bz.ERR_PRECONDITION                # 7 < 2*3+3
    assert L.bz_krum_select(fake, 7, 2, 0, fake, None) == bz.ERR_PRECONDITION
    assert L.bz_krum_select(fake, 7, 2, 8, fake, None) == bz.ERR_PRECONDITION
    assert L.bz_krum_select(fake, 7, -1, 1, fake, None) == bz.ERR_PRECONDITION
    assert L.bz_krum_select(None, 7, 2, 1, fake, None) == bz.ERR_INVALID_ARG
    assert L.bz_bulyan_select(fake, 25, 6, fake, None) == bz.ERR_PRECONDITION                # 25 < 4*6+3
    assert L.bz_bulyan_select(fake, 6, 1, fake, None) == bz.ERR_PRECONDITION
    assert L.bz_multikrum(fake, 49, 10, 10, 24, 1, fake, fake, None, fake, 1 << 30, None) == bz.ERR_PRECONDITION
    assert L.bz_multikrum(fake, 49, 10, 10, 5, 44, fake, fake, None, fake, 16, None) == bz.ERR_WORKSPACE
    assert L.bz_multikrum(fake, 49, 10, 10, 5, 44, fake, fake, None, None, 1 << 30, None) == bz.ERR_WORKSPACE
    assert L.bz_bulyan(fake, 25, 10, 10, 6, fake, fake, fake, 1 << 30, None) == bz.ERR_PRECONDITION
    assert L.bz_bulyan(fake, 25, 10, 10, 4, fake, fake, fake, 16, None) == bz.ERR_WORKSPACE
    assert L.bz_pairdist(fake, 25, 10, 10, None, fake, 1 << 30, None) == bz.ERR_INVALID_ARG
    assert L.bz_pairdist(fake, 25, 10, 9, fake, fake, 1 << 30, None) == bz.ERR_INVALID_ARG
    assert L.bz_mean_rows(fake, 25, 10, 10, fake, 0, fake, None) == bz.ERR_PRECONDITION
    assert L.bz_mean_rows(fake, 25, 0, 0, fake, 3, fake, None) == bz.OK
    assert L.bz_trimmed_mean(fake, 25, 10, 10, fake, 17, 18, fake, None) == bz.ERR_PRECONDITION
    assert L.bz_trimmed_mean(fake, 25, 10, 10, fake, 26, 3, fake, None) == bz.ERR_PRECONDITION
    # worst case
    mask = np.zeros(15, np.uint64)
    out = ctypes.c_int32(0)
    po = ctypes.addressof(out)
    assert L.bz_worst_case(None, 15, 25, 3, 2, 0, po, None, None, fake, 1 << 20, None) == bz.ERR_INVALID_ARG
    assert L.bz_worst_case(mask.ctypes.data, 15, 25, 3, 16, 0, po, None, None, fake, 1 << 20, None) == bz.ERR_INVALID_ARG
    assert L.bz_worst_case(mask.ctypes.data, 15, 25, 4, 2, 0, po, None, None, fake, 1 << 20, None) == bz.ERR_INVALID_ARG
    assert L.bz_worst_case(mask.ctypes.data, 15, 65, 3, 2, 0, po, None, None, fake, 1 << 20, None) == bz.ERR_UNSUPPORTED
    assert L.bz_worst_case(mask.ctypes.data, 15, 25, 9, 2, 0, po, None, None, fake, 1 << 20, None) == bz.ERR_UNSUPPORTED
    assert L.bz_worst_case(mask.ctypes.data, 15, 25, 3, 2, 0, po, None, None, None, 0, None) == bz.ERR_WORKSPACE
    bad = mask.copy()
    bad[3] = np.uint64(1) << np.uint64(40)  # a file index >= f
    assert L.bz_worst_case(bad.ctypes.data, 15, 25, 3, 2, 0, po, None, None, fake, 1 << 20, None) == bz.ERR_INVALID_ARG
    # the calls added around the distance stage: status, probe, path
    st = ctypes.c_int32(0)
    assert L.bz_pairdist_status(None, 25, ctypes.addressof(st), None) == bz.ERR_INVALID_ARG
    assert L.bz_pairdist_status(fake, 25, None, None) == bz.ERR_INVALID_ARG
    assert L.bz_pairdist_status(fake, 0, ctypes.addressof(st), None) == bz.ERR_INVALID_ARG
    assert L.bz_pairdist_status(fake, 129, ctypes.addressof(st), None) == bz.ERR_UNSUPPORTED
    assert L.bz_stream_probe(fake, 64, 0, None, None) == bz.ERR_INVALID_ARG
    assert L.bz_stream_probe(None, 64, 1, fake, None) == bz.ERR_INVALID_ARG
    assert L.bz_stream_probe(ctypes.c_void_p(264), 64, 0, fake, None) == bz.ERR_INVALID_ARG      # 16-byte alignment
    assert L.bz_stream_probe(fake, 60, 1, fake, None) == bz.ERR_INVALID_ARG                      # whole 64-bit words
    assert L.bz_last_path() in range(8)
    assert bz.kernel_launch_count() == n0


def test_binding_refuses_cpu_tensors(lib):
    import torch
    with pytest.raises(TypeError):
        bz.vote_median(torch.zeros((3, 25, 8)))
    with pytest.raises(ValueError):
        bz.vote_median(torch.zeros((3, 25, 8))[:, :, ::2])


def test_no_path_between_the_library_and_the_checker():
    # the product path must not reach the CPU checker, and the checker must not use the library
    pkg = os.path.join(ROOT, "paper_2010_04902_b200")
    for dirpath, _, files in os.walk(pkg):
        for name in files:
            if name.endswith((".py", ".cu", ".cuh", ".h", ".inc", ".cpp")):
                text = open(os.path.join(dirpath, name)).read()
                assert "import oracle" not in text and "from oracle" not in text and "bz_oracle" not in text, name
    for name in os.listdir(os.path.join(ROOT, "oracle")):
        if name.endswith((".py", ".cpp")):
            text = open(os.path.join(ROOT, "oracle", name)).read()
            assert "paper_2010_04902_b200" not in text and "libbz.so" not in text, name


def test_networks_file_is_current_and_correct():
    gen = os.path.join(ROOT, "paper_2010_04902_b200", "csrc", "gen_networks.py")
    res = subprocess.run([sys.executable, gen, "--check"], capture_output=True, text=True)
    assert res.returncode == 0, res.stdout + res.stderr
