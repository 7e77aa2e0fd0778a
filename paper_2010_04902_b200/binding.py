"""Thin ctypes binding over libbz.so: one Python function per C entry point, same names minus the
``bz_`` prefix.  It only marshals arguments (pointers, sizes, the current CUDA stream) - every step
of the aggregation runs in the library's kernels.  There is no fallback: a missing library or a
non-zero status raises.

Device arrays are torch CUDA tensors (torch is used for allocation and streams only).
"""
from __future__ import annotations

import ctypes
import os

import numpy as np
import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libbz.so")

OK = 0
ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_PRECONDITION, ERR_WORKSPACE, ERR_BUDGET, ERR_CUDA = -1, -2, -3, -4, -5, -6
OP_PAIRDIST, OP_MULTIKRUM, OP_BULYAN, OP_WORST_CASE, OP_VOTE_MEDIAN_HOST, OP_WORST_CASE_MOLS, OP_VOTE_VECTORWISE = 1, 2, 3, 4, 5, 6, 7
MAX_R, MAX_F = 15, 128
STATUS_RECOMPUTED, STATUS_STOPPED_EARLY = 1, 2
PATH_NONE, PATH_STAGED, PATH_REGISTERS, PATH_GENERIC, PATH_TENSOR, PATH_FP32, PATH_FP32_FUSED, PATH_FP64 = range(8)


class BzError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        msg = "%s failed: %s (%d)" % (what, status_string(status), status)
        if status == ERR_CUDA:
            msg += " - " + last_cuda_error()
        super().__init__(msg)


_lib = None

_c_int, _c_i64, _c_sz, _c_vp, _c_u64 = ctypes.c_int, ctypes.c_int64, ctypes.c_size_t, ctypes.c_void_p, ctypes.c_uint64

_SIGNATURES = {
    "bz_assign_mols": (_c_int, [_c_int, _c_int, _c_vp, _c_vp, _c_vp]),
    "bz_assign_ramanujan": (_c_int, [_c_int, _c_int, _c_vp, _c_vp, _c_vp]),
    "bz_vote": (_c_int, [_c_vp, _c_int, _c_int, _c_i64, _c_i64, _c_i64, _c_vp, _c_i64, _c_vp]),
    "bz_vote_median_rows": (_c_int, [_c_vp, _c_int, _c_int, _c_i64, _c_vp, _c_vp]),
    "bz_vote_rows": (_c_int, [_c_vp, _c_int, _c_int, _c_i64, _c_vp, _c_i64, _c_vp]),
    "bz_vote_vectorwise": (_c_int, [_c_vp, _c_int, _c_int, _c_i64, _c_i64, _c_i64, _c_vp, _c_i64, _c_vp, _c_vp, _c_sz, _c_vp]),
    "bz_vote_clusters": (_c_int, [_c_vp, _c_int, _c_int, _c_i64, _c_i64, _c_i64, ctypes.c_float, ctypes.c_float, _c_vp, _c_i64, _c_vp, _c_vp, _c_sz, _c_vp]),
    "bz_median": (_c_int, [_c_vp, _c_int, _c_i64, _c_i64, _c_vp, _c_vp]),
    "bz_vote_median": (_c_int, [_c_vp, _c_int, _c_int, _c_i64, _c_i64, _c_i64, _c_vp, _c_vp]),
    "bz_vote_median_host": (_c_int, [_c_vp, _c_int, _c_int, _c_i64, _c_vp, _c_vp, _c_sz, _c_vp]),
    "bz_vote_median_update": (_c_int, [_c_vp, _c_int, _c_int, _c_i64, _c_i64, _c_i64, _c_vp, _c_vp, ctypes.c_float,
                                       ctypes.c_float, _c_vp, _c_vp]),
    "bz_model_update": (_c_int, [_c_vp, _c_i64, _c_vp, _c_vp, ctypes.c_float, ctypes.c_float, _c_vp]),
    "bz_pairdist": (_c_int, [_c_vp, _c_int, _c_i64, _c_i64, _c_vp, _c_vp, _c_sz, _c_vp]),
    "bz_pairdist_static": (_c_int, [_c_vp, _c_int, _c_i64, _c_i64, _c_vp, _c_vp]),
    "bz_krum_select": (_c_int, [_c_vp, _c_int, _c_int, _c_int, _c_vp, _c_vp]),
    "bz_mean_rows": (_c_int, [_c_vp, _c_int, _c_i64, _c_i64, _c_vp, _c_int, _c_vp, _c_vp]),
    "bz_multikrum": (_c_int, [_c_vp, _c_int, _c_i64, _c_i64, _c_int, _c_int, _c_vp, _c_vp, _c_vp, _c_vp, _c_sz, _c_vp]),
    "bz_bulyan_select": (_c_int, [_c_vp, _c_int, _c_int, _c_vp, _c_vp]),
    "bz_trimmed_mean": (_c_int, [_c_vp, _c_int, _c_i64, _c_i64, _c_vp, _c_int, _c_int, _c_vp, _c_vp]),
    "bz_bulyan": (_c_int, [_c_vp, _c_int, _c_i64, _c_i64, _c_int, _c_vp, _c_vp, _c_vp, _c_sz, _c_vp]),
    "bz_worst_case": (_c_int, [_c_vp, _c_int, _c_int, _c_int, _c_int, _c_u64, _c_vp, _c_vp, _c_vp, _c_vp, _c_sz, _c_vp]),
    "bz_worst_case_part": (_c_int, [_c_vp, _c_int, _c_int, _c_int, _c_int, _c_int, _c_int, _c_u64, _c_vp, _c_vp, _c_vp, _c_vp, _c_sz,
                                    _c_vp]),
    "bz_vote_pairdist": (_c_int, [_c_vp, _c_int, _c_int, _c_i64, _c_i64, _c_i64, _c_vp, _c_i64, _c_vp, _c_vp, _c_sz, _c_vp]),
    "bz_vote_multikrum": (_c_int, [_c_vp, _c_int, _c_int, _c_i64, _c_i64, _c_i64, _c_int, _c_int, _c_vp, _c_i64, _c_vp, _c_vp,
                                   _c_vp, _c_vp, _c_sz, _c_vp]),
    "bz_vote_bulyan": (_c_int, [_c_vp, _c_int, _c_int, _c_i64, _c_i64, _c_i64, _c_int, _c_vp, _c_i64, _c_vp, _c_vp, _c_vp,
                                _c_sz, _c_vp]),
    "bz_worst_case_mols": (_c_int, [_c_int, _c_int, _c_int, _c_u64, _c_vp, _c_vp, _c_vp, _c_vp, _c_sz, _c_vp]),
    "bz_worst_case_mols_part": (_c_int, [_c_int, _c_int, _c_int, _c_int, _c_int, _c_u64, _c_vp, _c_vp, _c_vp, _c_vp, _c_sz, _c_vp]),
    "bz_mols_orbit_count": (_c_int, [_c_int, _c_int, _c_int, _c_vp]),
    "bz_workspace_bytes": (_c_sz, [_c_int, _c_int, _c_int, _c_i64, _c_int, _c_int]),
    "bz_status_string": (ctypes.c_char_p, [_c_int]),
    "bz_last_cuda_error": (ctypes.c_char_p, []),
    "bz_kernel_launch_count": (_c_u64, []),
    "bz_pipeline_timeouts": (_c_int, [_c_vp]),
    "bz_pairdist_status": (_c_int, [_c_vp, _c_int, _c_vp, _c_vp]),
    "bz_debug_stall_pipeline": (_c_int, [_c_int]),
    "bz_last_path": (_c_int, []),
    "bz_stream_probe": (_c_int, [_c_vp, _c_sz, _c_int, _c_vp, _c_vp]),
}

EXPORTS = sorted(_SIGNATURES)


def lib() -> ctypes.CDLL:
    """Load libbz.so (built in-tree by ``python -m paper_2010_04902_b200.build``)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError("libbz.so is missing at %s: run `python -m paper_2010_04902_b200.build` "
                              "(there is no CPU fallback)" % LIB_PATH)
        L = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(L, name)
            fn.restype = res
            fn.argtypes = args
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().bz_status_string(status).decode()


def last_cuda_error() -> str:
    return lib().bz_last_cuda_error().decode()


def kernel_launch_count() -> int:
    return int(lib().bz_kernel_launch_count())


def pipeline_timeouts() -> int:
    """Barrier waits that ran out inside the TMA-staged kernels since the library was loaded (0 when healthy)."""
    n = ctypes.c_uint(0)
    _check(lib().bz_pipeline_timeouts(ctypes.addressof(n)), "bz_pipeline_timeouts")
    return int(n.value)


def stream_probe(buf: torch.Tensor, checksum: torch.Tensor | None = None, staged: bool = False) -> torch.Tensor:
    """bz_stream_probe: XOR of the 64-bit words of `buf` (any dtype, contiguous), read once from device memory
    (staged: through the bulk-copy engine and shared memory instead of plain loads)."""
    if not buf.is_cuda or not buf.is_contiguous():
        raise TypeError("buf must be a contiguous CUDA tensor")
    if checksum is None:
        checksum = torch.zeros(1, dtype=torch.int64, device=buf.device)
    _check(lib().bz_stream_probe(buf.data_ptr(), buf.numel() * buf.element_size(), 1 if staged else 0,
                                 _dev(checksum, torch.int64, "checksum"), _stream()), "bz_stream_probe")
    return checksum


def last_path() -> int:
    """PATH_* of the kernel family this thread's last call dispatched to."""
    return int(lib().bz_last_path())


def pairdist_status(workspace: torch.Tensor, f: int) -> int:
    """STATUS_* bits of the distance stage of the last call that used `workspace` (synchronises the stream)."""
    st = ctypes.c_int32(0)
    _check(lib().bz_pairdist_status(_dev(workspace, torch.uint8, "workspace"), f, ctypes.addressof(st), _stream()),
           "bz_pairdist_status")
    return int(st.value)


def debug_stall_pipeline(on: bool) -> None:
    """Testing aid: make the tensor-core distance kernels' bounded waits run out (see bz.h)."""
    _check(lib().bz_debug_stall_pipeline(1 if on else 0), "bz_debug_stall_pipeline")


def _check(status: int, what: str):
    if status != OK:
        raise BzError(status, what)


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _dev(t: torch.Tensor, dtype, name: str) -> int:
    if not t.is_cuda or t.dtype != dtype:
        raise TypeError("%s must be a CUDA tensor of dtype %s" % (name, dtype))
    return t.data_ptr()


def _rows(t: torch.Tensor, name: str):
    """(f, d, ld) of a [f][d] tensor whose last dimension is contiguous."""
    if t.dim() != 2 or (t.shape[1] > 1 and t.stride(1) != 1):
        raise ValueError("%s must be [f][d] with unit stride along d" % name)
    f, d = t.shape
    return f, d, (max(d, t.stride(0)) if f > 1 else d)


def _replicas(t: torch.Tensor):
    """(r, f, d, ld_file, ld_replica) of a [r][f][d] tensor whose last dimension is contiguous."""
    if t.dim() != 3 or (t.shape[2] > 1 and t.stride(2) != 1):
        raise ValueError("replicas must be [r][f][d] with unit stride along d")
    r, f, d = t.shape
    ld_file = max(d, t.stride(1)) if f > 1 else d
    ld_rep = max(d, t.stride(0)) if r > 1 else f * ld_file
    return r, f, d, ld_file, ld_rep


def workspace_bytes(op: int, r: int = 0, f: int = 0, d: int = 0, c: int = 0, m: int = 0) -> int:
    return int(lib().bz_workspace_bytes(op, r, f, d, c, m))


def alloc_workspace(op: int, r: int = 0, f: int = 0, d: int = 0, c: int = 0, m: int = 0, device="cuda") -> torch.Tensor:
    n = workspace_bytes(op, r, f, d, c, m)
    return torch.empty(max(n, 256), dtype=torch.uint8, device=device)


# --------------------------------------------------------------------------------------------- host

def assign_mols(l: int, r: int):
    """Algorithm 2.  Returns numpy (worker_files[K][l], file_workers[f][r], worker_mask[K] or None)."""
    K, f = max(r * l, 1), max(l * l, 1)
    wf = np.zeros((K, max(l, 1)), np.int32)
    fw = np.zeros((f, max(r, 1)), np.int32)
    mask = np.zeros(K, np.uint64) if l * l <= 64 else None
    st = lib().bz_assign_mols(l, r, wf.ctypes.data, fw.ctypes.data, mask.ctypes.data if mask is not None else None)
    _check(st, "bz_assign_mols(l=%d, r=%d)" % (l, r))
    return wf, fw, mask


def ramanujan_dims(m: int, s: int):
    """(K, f, l, r) of Eq. (7) for the Ramanujan construction with parameters (m, s)."""
    return (m * s, s * s, s, m) if m < s else (s * s, m * s, m, s)


def assign_ramanujan(m: int, s: int):
    """Sec. 4.2.1.  Returns numpy (worker_files[K][l], file_workers[f][r], worker_mask[K] or None)."""
    K, f, l, r = ramanujan_dims(max(m, 1), max(s, 1))
    wf = np.zeros((K, l), np.int32)
    fw = np.zeros((f, r), np.int32)
    mask = np.zeros(K, np.uint64) if f <= 64 else None
    st = lib().bz_assign_ramanujan(m, s, wf.ctypes.data, fw.ctypes.data, mask.ctypes.data if mask is not None else None)
    _check(st, "bz_assign_ramanujan(m=%d, s=%d)" % (m, s))
    return wf, fw, mask


def worst_case(worker_mask, f: int, r: int, q: int, max_subsets: int = 0, workspace: torch.Tensor | None = None):
    """Exhaustive c_max^(q).  Returns (c_max, argmax[q] numpy, n_subsets)."""
    mask = np.ascontiguousarray(worker_mask, np.uint64)
    K = int(mask.shape[0])
    ws = workspace if workspace is not None else alloc_workspace(OP_WORST_CASE, r, f)
    cmax = ctypes.c_int32(0)
    n = ctypes.c_uint64(0)
    arg = np.zeros(max(q, 1), np.int32)
    st = lib().bz_worst_case(mask.ctypes.data, K, f, r, q, max_subsets, ctypes.addressof(cmax), arg.ctypes.data,
                             ctypes.addressof(n), ws.data_ptr(), ws.numel(), _stream())
    _check(st, "bz_worst_case(K=%d, q=%d)" % (K, q))
    return int(cmax.value), arg[:q].copy(), int(n.value)


def worst_case_part(worker_mask, f: int, r: int, q: int, part: int, parts: int, max_subsets: int = 0,
                    workspace: torch.Tensor | None = None):
    """bz_worst_case_part: share `part` of `parts` of the exhaustive search.  Returns (c_max, argmax[q] numpy,
    n_subsets); c_max is -1 for a share that received nothing."""
    mask = np.ascontiguousarray(worker_mask, np.uint64)
    K = int(mask.shape[0])
    ws = workspace if workspace is not None else alloc_workspace(OP_WORST_CASE, r, f)
    cmax = ctypes.c_int32(0)
    n = ctypes.c_uint64(0)
    arg = np.zeros(max(q, 1), np.int32)
    st = lib().bz_worst_case_part(mask.ctypes.data, K, f, r, q, part, parts, max_subsets, ctypes.addressof(cmax),
                                  arg.ctypes.data, ctypes.addressof(n), ws.data_ptr(), ws.numel(), _stream())
    _check(st, "bz_worst_case_part(K=%d, q=%d, part %d of %d)" % (K, q, part, parts))
    return int(cmax.value), arg[:q].copy(), int(n.value)


def worst_case_mols(l: int, r: int, q: int, max_subsets: int = 0, workspace: torch.Tensor | None = None):
    """bz_worst_case_mols: c_max^(q) of the placement assign_mols(l, r), one set per translation orbit.
    Returns (c_max, argmax[q] numpy, n_orbits)."""
    ws = workspace if workspace is not None else alloc_workspace(OP_WORST_CASE_MOLS, r, l * l)
    cmax = ctypes.c_int32(0)
    n = ctypes.c_uint64(0)
    arg = np.zeros(max(q, 1), np.int32)
    st = lib().bz_worst_case_mols(l, r, q, max_subsets, ctypes.addressof(cmax), arg.ctypes.data, ctypes.addressof(n),
                                  ws.data_ptr(), ws.numel(), _stream())
    _check(st, "bz_worst_case_mols(l=%d, r=%d, q=%d)" % (l, r, q))
    return int(cmax.value), arg[:q].copy(), int(n.value)


def worst_case_mols_part(l: int, r: int, q: int, part: int, parts: int, max_subsets: int = 0,
                         workspace: torch.Tensor | None = None):
    """bz_worst_case_mols_part: share `part` of `parts` of the orbit search.  Returns (c_max, argmax[q] numpy, n_orbits);
    c_max is -1 for a share that received nothing."""
    ws = workspace if workspace is not None else alloc_workspace(OP_WORST_CASE_MOLS, r, l * l)
    cmax = ctypes.c_int32(0)
    n = ctypes.c_uint64(0)
    arg = np.zeros(max(q, 1), np.int32)
    st = lib().bz_worst_case_mols_part(l, r, q, part, parts, max_subsets, ctypes.addressof(cmax), arg.ctypes.data,
                                       ctypes.addressof(n), ws.data_ptr(), ws.numel(), _stream())
    _check(st, "bz_worst_case_mols_part(l=%d, r=%d, q=%d, part %d of %d)" % (l, r, q, part, parts))
    return int(cmax.value), arg[:q].copy(), int(n.value)


def mols_orbit_count(l: int, r: int, q: int) -> int:
    n = ctypes.c_uint64(0)
    _check(lib().bz_mols_orbit_count(l, r, q, ctypes.addressof(n)), "bz_mols_orbit_count")
    return int(n.value)


# --------------------------------------------------------------------------------------------- device

def vote(replicas: torch.Tensor, voted: torch.Tensor | None = None) -> torch.Tensor:
    r, f, d, ld_file, ld_rep = _replicas(replicas)
    if voted is None:
        voted = torch.empty((f, d), dtype=torch.float32, device=replicas.device)
    vf, vd, ld_v = _rows(voted, "voted")
    if (vf, vd) != (f, d):
        raise ValueError("voted must be [%d][%d]" % (f, d))
    st = lib().bz_vote(_dev(replicas, torch.float32, "replicas"), r, f, d, ld_file, ld_rep,
                       _dev(voted, torch.float32, "voted"), ld_v, _stream())
    _check(st, "bz_vote")
    return voted


def row_table(worker_buffers, file_workers, worker_files) -> torch.Tensor:
    """Device table of r*f row pointers for bz_vote_median_rows / bz_vote_rows from what the workers sent:
    worker_buffers[u] is a CUDA float32 tensor [l][d] holding worker u's gradients in the order of
    worker_files[u]; entry k*f + i of the table points at the gradient worker file_workers[i][k] returned
    for file i.  The buffers must stay alive while the table is in use."""
    f, r = len(file_workers), len(file_workers[0])
    ptrs = []
    for k in range(r):
        for i in range(f):
            u = int(file_workers[i][k])
            slot = [int(x) for x in worker_files[u]].index(i)
            row = worker_buffers[u][slot]
            if row.dtype != torch.float32 or not row.is_cuda or row.stride(0) != 1:
                raise ValueError("worker buffers must be CUDA float32 tensors with contiguous rows")
            ptrs.append(row.data_ptr())
    return torch.tensor(ptrs, dtype=torch.int64, device=worker_buffers[0].device)


def vote_median_rows(table: torch.Tensor, r: int, f: int, d: int, out: torch.Tensor | None = None) -> torch.Tensor:
    """bz_vote_median_rows on a table made by row_table()."""
    if table.dtype != torch.int64 or not table.is_cuda or table.numel() != r * f:
        raise ValueError("table must be a CUDA int64 tensor of r*f pointers")
    if out is None:
        out = torch.empty(d, dtype=torch.float32, device=table.device)
    st = lib().bz_vote_median_rows(table.data_ptr(), r, f, d, _dev(out, torch.float32, "out"), _stream())
    _check(st, "bz_vote_median_rows")
    return out


def vote_rows(table: torch.Tensor, r: int, f: int, d: int, voted: torch.Tensor | None = None) -> torch.Tensor:
    """bz_vote_rows on a table made by row_table()."""
    if table.dtype != torch.int64 or not table.is_cuda or table.numel() != r * f:
        raise ValueError("table must be a CUDA int64 tensor of r*f pointers")
    if voted is None:
        voted = torch.empty((f, d), dtype=torch.float32, device=table.device)
    _, _, ld_v = _rows(voted, "voted")
    st = lib().bz_vote_rows(table.data_ptr(), r, f, d, _dev(voted, torch.float32, "voted"), ld_v, _stream())
    _check(st, "bz_vote_rows")
    return voted


def vote_vectorwise(replicas: torch.Tensor, voted: torch.Tensor | None = None, workspace: torch.Tensor | None = None):
    """bz_vote_vectorwise: the vote of Eq. (3) on whole gradients.  Returns (voted[f][d], winner[f])."""
    r, f, d, ld_file, ld_rep = _replicas(replicas)
    if voted is None:
        voted = torch.empty((f, d), dtype=torch.float32, device=replicas.device)
    vf, vd, ld_v = _rows(voted, "voted")
    if (vf, vd) != (f, d):
        raise ValueError("voted must be [%d][%d]" % (f, d))
    ws = workspace if workspace is not None else alloc_workspace(OP_VOTE_VECTORWISE, r, f, d, device=replicas.device)
    winner = torch.empty(f, dtype=torch.int32, device=replicas.device)
    st = lib().bz_vote_vectorwise(_dev(replicas, torch.float32, "replicas"), r, f, d, ld_file, ld_rep,
                                  _dev(voted, torch.float32, "voted"), ld_v, winner.data_ptr(), ws.data_ptr(), ws.numel(),
                                  _stream())
    _check(st, "bz_vote_vectorwise")
    return voted, winner


def vote_clusters(replicas: torch.Tensor, abs_tol: float, rel_tol: float, voted: torch.Tensor | None = None,
                  workspace: torch.Tensor | None = None):
    """bz_vote_clusters: the whole-vector vote with agreement up to a tolerance.  Returns (voted[f][d], winner[f])."""
    r, f, d, ld_file, ld_rep = _replicas(replicas)
    if voted is None:
        voted = torch.empty((f, d), dtype=torch.float32, device=replicas.device)
    vf, vd, ld_v = _rows(voted, "voted")
    if (vf, vd) != (f, d):
        raise ValueError("voted must be [%d][%d]" % (f, d))
    ws = workspace if workspace is not None else alloc_workspace(OP_VOTE_VECTORWISE, r, f, d, device=replicas.device)
    winner = torch.empty(f, dtype=torch.int32, device=replicas.device)
    st = lib().bz_vote_clusters(_dev(replicas, torch.float32, "replicas"), r, f, d, ld_file, ld_rep, float(abs_tol),
                                float(rel_tol), _dev(voted, torch.float32, "voted"), ld_v, winner.data_ptr(), ws.data_ptr(),
                                ws.numel(), _stream())
    _check(st, "bz_vote_clusters")
    return voted, winner


def median(voted: torch.Tensor, out: torch.Tensor | None = None) -> torch.Tensor:
    f, d, ld = _rows(voted, "voted")
    if out is None:
        out = torch.empty(d, dtype=torch.float32, device=voted.device)
    st = lib().bz_median(_dev(voted, torch.float32, "voted"), f, d, ld, _dev(out, torch.float32, "out"), _stream())
    _check(st, "bz_median")
    return out


def vote_median(replicas: torch.Tensor, out: torch.Tensor | None = None) -> torch.Tensor:
    r, f, d, ld_file, ld_rep = _replicas(replicas)
    if out is None:
        out = torch.empty(d, dtype=torch.float32, device=replicas.device)
    st = lib().bz_vote_median(_dev(replicas, torch.float32, "replicas"), r, f, d, ld_file, ld_rep,
                              _dev(out, torch.float32, "out"), _stream())
    _check(st, "bz_vote_median")
    return out


def _state(t, d: int, name: str):
    if t is None:
        return None
    if t.dim() != 1 or t.numel() != d or not t.is_contiguous():
        raise TypeError("%s must be a contiguous [d] tensor" % name)
    return _dev(t, torch.float32, name)


def vote_median_update(replicas: torch.Tensor, w: torch.Tensor, eta: float, velocity: torch.Tensor | None = None,
                       mu: float = 0.0, out: torch.Tensor | None = None) -> None:
    """bz_vote_median_update: aggregate and apply Eq. (1) to w (and velocity) in place; `out`, when given,
    also receives the aggregate."""
    r, f, d, ld_file, ld_rep = _replicas(replicas)
    st = lib().bz_vote_median_update(_dev(replicas, torch.float32, "replicas"), r, f, d, ld_file, ld_rep,
                                     _state(w, d, "w"), _state(velocity, d, "velocity"), eta, mu,
                                     _state(out, d, "out"), _stream())
    _check(st, "bz_vote_median_update")


def model_update(g: torch.Tensor, w: torch.Tensor, eta: float, velocity: torch.Tensor | None = None,
                 mu: float = 0.0) -> None:
    d = g.numel()
    st = lib().bz_model_update(_state(g, d, "g"), d, _state(w, d, "w"), _state(velocity, d, "velocity"), eta, mu,
                               _stream())
    _check(st, "bz_model_update")


def vote_median_host(replicas_host: torch.Tensor, out_host: torch.Tensor, workspace: torch.Tensor) -> torch.Tensor:
    """replicas_host: contiguous CPU [r][f][d] (pin it for full copy speed); out_host: CPU [d]."""
    if replicas_host.is_cuda or out_host.is_cuda or not replicas_host.is_contiguous() or not out_host.is_contiguous():
        raise TypeError("replicas_host / out_host must be contiguous CPU tensors")
    if replicas_host.dtype != torch.float32 or out_host.dtype != torch.float32:
        raise TypeError("float32 expected")
    r, f, d = replicas_host.shape
    st = lib().bz_vote_median_host(replicas_host.data_ptr(), r, f, d, out_host.data_ptr(), workspace.data_ptr(),
                                   workspace.numel(), _stream())
    _check(st, "bz_vote_median_host")
    return out_host


def pairdist(voted: torch.Tensor, workspace: torch.Tensor | None = None, dist: torch.Tensor | None = None) -> torch.Tensor:
    f, d, ld = _rows(voted, "voted")
    ws = workspace if workspace is not None else alloc_workspace(OP_PAIRDIST, 0, f, d, device=voted.device)
    if dist is None:
        dist = torch.empty((f, f), dtype=torch.float64, device=voted.device)
    st = lib().bz_pairdist(_dev(voted, torch.float32, "voted"), f, d, ld, _dev(dist, torch.float64, "dist"),
                           ws.data_ptr(), ws.numel(), _stream())
    _check(st, "bz_pairdist")
    return dist


STATIC_SCRATCH_BYTES = 4 << 20
ERR_STATIC_LIMIT = -7


def pairdist_static(voted: torch.Tensor, dist: torch.Tensor) -> torch.Tensor:
    """bz_pairdist_static: the distance matrix for a caller that cannot supply (or allocate) a device
    workspace - for example code running under a frozen memory plan or a fixed memory budget.  The
    scratch is a 4 MiB array inside the library; `dist` ([f][f] float64) must already exist.  Shapes
    that need more scratch (f > 84) raise with status ERR_STATIC_LIMIT.  Calls share that
    array: do not let two of them run on the GPU at the same time."""
    f, d, ld = _rows(voted, "voted")
    st = lib().bz_pairdist_static(_dev(voted, torch.float32, "voted"), f, d, ld, _dev(dist, torch.float64, "dist"),
                                  _stream())
    _check(st, "bz_pairdist_static")
    return dist


def krum_select(dist: torch.Tensor, c: int, m: int) -> torch.Tensor:
    f = dist.shape[0]
    sel = torch.empty(max(m, 1), dtype=torch.int32, device=dist.device)
    st = lib().bz_krum_select(_dev(dist, torch.float64, "dist"), f, c, m, sel.data_ptr(), _stream())
    _check(st, "bz_krum_select")
    return sel[:m]


def mean_rows(voted: torch.Tensor, selected: torch.Tensor, out: torch.Tensor | None = None) -> torch.Tensor:
    f, d, ld = _rows(voted, "voted")
    if out is None:
        out = torch.empty(d, dtype=torch.float32, device=voted.device)
    st = lib().bz_mean_rows(_dev(voted, torch.float32, "voted"), f, d, ld, _dev(selected, torch.int32, "selected"),
                            selected.numel(), _dev(out, torch.float32, "out"), _stream())
    _check(st, "bz_mean_rows")
    return out


def multikrum(voted: torch.Tensor, c: int, m: int, workspace: torch.Tensor | None = None,
              out: torch.Tensor | None = None, want_dist: bool = False):
    """Returns (out[d], selected[m]) or (out, selected, dist) with want_dist."""
    f, d, ld = _rows(voted, "voted")
    ws = workspace if workspace is not None else alloc_workspace(OP_MULTIKRUM, 0, f, d, c, m, device=voted.device)
    if out is None:
        out = torch.empty(d, dtype=torch.float32, device=voted.device)
    sel = torch.empty(max(m, 1), dtype=torch.int32, device=voted.device)
    dist = torch.empty((f, f), dtype=torch.float64, device=voted.device) if want_dist else None
    st = lib().bz_multikrum(_dev(voted, torch.float32, "voted"), f, d, ld, c, m, _dev(out, torch.float32, "out"),
                            sel.data_ptr(), dist.data_ptr() if dist is not None else None, ws.data_ptr(), ws.numel(),
                            _stream())
    _check(st, "bz_multikrum")
    return (out, sel[:m], dist) if want_dist else (out, sel[:m])


def bulyan_select(dist: torch.Tensor, c: int) -> torch.Tensor:
    f = dist.shape[0]
    theta = f - 2 * c
    sel = torch.empty(max(theta, 1), dtype=torch.int32, device=dist.device)
    st = lib().bz_bulyan_select(_dev(dist, torch.float64, "dist"), f, c, sel.data_ptr(), _stream())
    _check(st, "bz_bulyan_select")
    return sel[:theta]


def trimmed_mean(voted: torch.Tensor, selected: torch.Tensor, beta: int, out: torch.Tensor | None = None) -> torch.Tensor:
    f, d, ld = _rows(voted, "voted")
    if out is None:
        out = torch.empty(d, dtype=torch.float32, device=voted.device)
    st = lib().bz_trimmed_mean(_dev(voted, torch.float32, "voted"), f, d, ld, _dev(selected, torch.int32, "selected"),
                               selected.numel(), beta, _dev(out, torch.float32, "out"), _stream())
    _check(st, "bz_trimmed_mean")
    return out


def bulyan(voted: torch.Tensor, c: int, workspace: torch.Tensor | None = None, out: torch.Tensor | None = None):
    """Returns (out[d], selected[f - 2c])."""
    f, d, ld = _rows(voted, "voted")
    ws = workspace if workspace is not None else alloc_workspace(OP_BULYAN, 0, f, d, c, device=voted.device)
    if out is None:
        out = torch.empty(d, dtype=torch.float32, device=voted.device)
    theta = f - 2 * c
    sel = torch.empty(max(theta, 1), dtype=torch.int32, device=voted.device)
    st = lib().bz_bulyan(_dev(voted, torch.float32, "voted"), f, d, ld, c, _dev(out, torch.float32, "out"),
                         sel.data_ptr(), ws.data_ptr(), ws.numel(), _stream())
    _check(st, "bz_bulyan")
    return out, sel[:max(theta, 0)]


# ------------------------------------------------------------------------- from the replicas in one pass

def _voted_for(replicas: torch.Tensor, voted: torch.Tensor | None):
    r, f, d, ld_file, ld_rep = _replicas(replicas)
    if voted is None:
        voted = torch.empty((f, d), dtype=torch.float32, device=replicas.device)
    vf, vd, ld_v = _rows(voted, "voted")
    if (vf, vd) != (f, d):
        raise ValueError("voted must be [%d][%d]" % (f, d))
    return r, f, d, ld_file, ld_rep, voted, ld_v


def vote_pairdist(replicas: torch.Tensor, voted: torch.Tensor | None = None, workspace: torch.Tensor | None = None,
                  dist: torch.Tensor | None = None):
    """bz_vote_pairdist: returns (voted[f][d], dist[f][f])."""
    r, f, d, ld_file, ld_rep, voted, ld_v = _voted_for(replicas, voted)
    ws = workspace if workspace is not None else alloc_workspace(OP_PAIRDIST, 0, f, d, device=replicas.device)
    if dist is None:
        dist = torch.empty((f, f), dtype=torch.float64, device=replicas.device)
    st = lib().bz_vote_pairdist(_dev(replicas, torch.float32, "replicas"), r, f, d, ld_file, ld_rep,
                                _dev(voted, torch.float32, "voted"), ld_v, _dev(dist, torch.float64, "dist"),
                                ws.data_ptr(), ws.numel(), _stream())
    _check(st, "bz_vote_pairdist")
    return voted, dist


def vote_multikrum(replicas: torch.Tensor, c: int, m: int, voted: torch.Tensor | None = None,
                   workspace: torch.Tensor | None = None, out: torch.Tensor | None = None,
                   dist: torch.Tensor | None = None):
    """bz_vote_multikrum: returns (out[d], selected[m], voted[f][d]); the distance matrix goes to `dist` if given."""
    r, f, d, ld_file, ld_rep, voted, ld_v = _voted_for(replicas, voted)
    ws = workspace if workspace is not None else alloc_workspace(OP_MULTIKRUM, 0, f, d, c, m, device=replicas.device)
    if out is None:
        out = torch.empty(d, dtype=torch.float32, device=replicas.device)
    sel = torch.empty(max(m, 1), dtype=torch.int32, device=replicas.device)
    st = lib().bz_vote_multikrum(_dev(replicas, torch.float32, "replicas"), r, f, d, ld_file, ld_rep, c, m,
                                 _dev(voted, torch.float32, "voted"), ld_v, _dev(out, torch.float32, "out"),
                                 sel.data_ptr(), None if dist is None else _dev(dist, torch.float64, "dist"),
                                 ws.data_ptr(), ws.numel(), _stream())
    _check(st, "bz_vote_multikrum")
    return out, sel[:m], voted


def vote_bulyan(replicas: torch.Tensor, c: int, voted: torch.Tensor | None = None,
                workspace: torch.Tensor | None = None, out: torch.Tensor | None = None):
    """bz_vote_bulyan: returns (out[d], selected[f - 2c], voted[f][d])."""
    r, f, d, ld_file, ld_rep, voted, ld_v = _voted_for(replicas, voted)
    ws = workspace if workspace is not None else alloc_workspace(OP_BULYAN, 0, f, d, c, device=replicas.device)
    if out is None:
        out = torch.empty(d, dtype=torch.float32, device=replicas.device)
    theta = f - 2 * c
    sel = torch.empty(max(theta, 1), dtype=torch.int32, device=replicas.device)
    st = lib().bz_vote_bulyan(_dev(replicas, torch.float32, "replicas"), r, f, d, ld_file, ld_rep, c,
                              _dev(voted, torch.float32, "voted"), ld_v, _dev(out, torch.float32, "out"),
                              sel.data_ptr(), ws.data_ptr(), ws.numel(), _stream())
    _check(st, "bz_vote_bulyan")
    return out, sel[:max(theta, 0)], voted
