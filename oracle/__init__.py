"""numpy front-end of the CPU oracle (oracle/bz_oracle.cpp).

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the benchmark's CPU
baseline.  Nothing on the product path may import this package, and this package imports
nothing from the CUDA library or its binding.

Every function takes and returns numpy arrays; the arithmetic lives in the C++ file, each
function there cites the passage of the paper it follows.
"""
import ctypes
import os

import numpy as np

from . import build as _build

_lib = None

_i32p = ctypes.POINTER(ctypes.c_int32)
_u64p = ctypes.POINTER(ctypes.c_uint64)
_f32p = ctypes.POINTER(ctypes.c_float)
_f64p = ctypes.POINTER(ctypes.c_double)


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(_build.build())
        _lib.orc_num_threads.restype = ctypes.c_int
    return _lib


def _p(a, typ):
    return a.ctypes.data_as(typ)


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def num_threads() -> int:
    return int(_load().orc_num_threads())


def assign(l: int, r: int):
    """Algorithm 2 / Ramanujan Case 2 (r == l).  Returns (worker_files[K][l], file_workers[f][r],
    worker_mask[K] uint64 or None when f > 64)."""
    lib = _load()
    K, f = r * l, l * l
    wf = np.zeros((max(K, 1), max(l, 1)), np.int32)
    fw = np.zeros((max(f, 1), max(r, 1)), np.int32)
    mask = np.zeros(max(K, 1), np.uint64)
    rc = lib.orc_assign(ctypes.c_int(l), ctypes.c_int(r), _p(wf, _i32p), _p(fw, _i32p), _p(mask, _u64p))
    if rc != 0:
        raise ValueError("orc_assign(l=%d, r=%d) rejected: %d" % (l, r, rc))
    return wf, fw, (mask if f <= 64 else None)


def field_tables(l: int):
    """Addition and multiplication tables [l][l] of the finite field with l = p^k elements."""
    lib = _load()
    add = np.zeros((l, l), np.int32)
    mul = np.zeros((l, l), np.int32)
    if lib.orc_field_tables(ctypes.c_int(l), _p(add, _i32p), _p(mul, _i32p)) != 0:
        raise ValueError("no field with %d elements" % l)
    return add, mul


def ramanujan_dims(m: int, s: int):
    """(K, f, l, r) of Eq. (7)."""
    return (m * s, s * s, s, m) if m < s else (s * s, m * s, m, s)


def assign_ramanujan(m: int, s: int):
    """Sec. 4.2.1 array-code bigraph.  Returns (worker_files[K][l], file_workers[f][r], worker_mask or None)."""
    lib = _load()
    if m < 2 or s < 2:
        raise ValueError("orc_assign_ramanujan(m=%d, s=%d) rejected" % (m, s))
    K, f, l, r = ramanujan_dims(m, s)
    wf = np.zeros((K, l), np.int32)
    fw = np.zeros((f, r), np.int32)
    mask = np.zeros(K, np.uint64)
    rc = lib.orc_assign_ramanujan(ctypes.c_int(m), ctypes.c_int(s), _p(wf, _i32p), _p(fw, _i32p), _p(mask, _u64p))
    if rc != 0:
        raise ValueError("orc_assign_ramanujan(m=%d, s=%d) rejected: %d" % (m, s, rc))
    return wf, fw, (mask if f <= 64 else None)


def vote(replicas):
    """replicas [r][f][d] float32 -> voted [f][d] (Eq. 3, element by element)."""
    lib = _load()
    rep = _f32(replicas)
    r, f, d = rep.shape
    out = np.empty((f, d), np.float32)
    lib.orc_vote(_p(rep, _f32p), ctypes.c_int(r), ctypes.c_int(f), ctypes.c_int64(d), _p(out, _f32p))
    return out


def vote_vectorwise(replicas):
    """replicas [r][f][d] -> winner[f]: index k of the whole-vector majority copy of each file."""
    lib = _load()
    rep = _f32(replicas)
    r, f, d = rep.shape
    win = np.empty(f, np.int32)
    lib.orc_vote_vectorwise(_p(rep, _f32p), ctypes.c_int(r), ctypes.c_int(f), ctypes.c_int64(d), _p(win, _i32p))
    return win


def vote_clusters(replicas, abs_tol: float, rel_tol: float):
    """replicas [r][f][d] -> winner[f]: the copy that agrees with the most copies of its file, where two copies
    agree iff |a - b| <= abs_tol + rel_tol * max(|a|, |b|) at every coordinate (or the bits are equal)."""
    lib = _load()
    rep = _f32(replicas)
    r, f, d = rep.shape
    win = np.empty(f, np.int32)
    lib.orc_vote_clusters(_p(rep, _f32p), ctypes.c_int(r), ctypes.c_int(f), ctypes.c_int64(d), ctypes.c_float(abs_tol),
                          ctypes.c_float(rel_tol), _p(win, _i32p))
    return win


def median(voted):
    """voted [f][d] -> out[d], coordinate-wise median by IEEE total order."""
    lib = _load()
    v = _f32(voted)
    f, d = v.shape
    out = np.empty(d, np.float32)
    lib.orc_median(_p(v, _f32p), ctypes.c_int(f), ctypes.c_int64(d), _p(out, _f32p))
    return out


def vote_median(replicas):
    return median(vote(replicas))


def pairdist(voted):
    """voted [f][d] -> D[f][f] float64 squared distances."""
    lib = _load()
    v = _f32(voted)
    f, d = v.shape
    D = np.empty((f, f), np.float64)
    lib.orc_pairdist(_p(v, _f32p), ctypes.c_int(f), ctypes.c_int64(d), _p(D, _f64p))
    return D


def krum_scores(D, c: int):
    lib = _load()
    D = np.ascontiguousarray(D, np.float64)
    f = D.shape[0]
    s = np.empty(f, np.float64)
    lib.orc_krum_scores(_p(D, _f64p), ctypes.c_int(f), ctypes.c_int(c), _p(s, _f64p))
    return s


def multikrum_select(D, c: int, m: int):
    lib = _load()
    D = np.ascontiguousarray(D, np.float64)
    f = D.shape[0]
    sel = np.empty(max(m, 1), np.int32)
    rc = lib.orc_multikrum_select(_p(D, _f64p), ctypes.c_int(f), ctypes.c_int(c), ctypes.c_int(m), _p(sel, _i32p))
    if rc != 0:
        raise ValueError("multi-Krum precondition f >= 2c+3, 1 <= m <= f violated (f=%d c=%d m=%d)" % (f, c, m))
    return sel[:m]


def mean_rows(voted, selected):
    lib = _load()
    v = _f32(voted)
    f, d = v.shape
    sel = np.ascontiguousarray(selected, np.int32)
    out = np.empty(d, np.float32)
    lib.orc_mean_rows(_p(v, _f32p), ctypes.c_int(f), ctypes.c_int64(d), _p(sel, _i32p), ctypes.c_int(len(sel)),
                      _p(out, _f32p))
    return out


def multikrum(voted, c: int, m: int):
    """Returns (out[d], selected[m], D[f][f])."""
    D = pairdist(voted)
    sel = multikrum_select(D, c, m)
    return mean_rows(voted, sel), sel, D


def bulyan_select(D, c: int):
    lib = _load()
    D = np.ascontiguousarray(D, np.float64)
    f = D.shape[0]
    theta = f - 2 * c
    sel = np.empty(max(theta, 1), np.int32)
    rc = lib.orc_bulyan_select(_p(D, _f64p), ctypes.c_int(f), ctypes.c_int(c), _p(sel, _i32p))
    if rc != 0:
        raise ValueError("Bulyan precondition f >= 4c+3 violated (f=%d c=%d)" % (f, c))
    return sel[:theta]


def trimmed_mean(voted, selected, beta: int):
    lib = _load()
    v = _f32(voted)
    f, d = v.shape
    sel = np.ascontiguousarray(selected, np.int32)
    out = np.empty(d, np.float32)
    lib.orc_trimmed_mean(_p(v, _f32p), ctypes.c_int(f), ctypes.c_int64(d), _p(sel, _i32p), ctypes.c_int(len(sel)),
                         ctypes.c_int(beta), _p(out, _f32p))
    return out


def bulyan(voted, c: int):
    """Returns (out[d], selected[theta], D)."""
    D = pairdist(voted)
    sel = bulyan_select(D, c)
    beta = len(sel) - 2 * c
    return trimmed_mean(voted, sel, beta), sel, D


def worst_case(worker_files, f: int, r: int, q: int):
    """Exhaustive c_max^(q).  Returns (c_max, argmax[q], n_subsets)."""
    lib = _load()
    wf = np.ascontiguousarray(worker_files, np.int32)
    K, l = wf.shape
    cmax = ctypes.c_int32(0)
    n = ctypes.c_uint64(0)
    arg = np.zeros(max(q, 1), np.int32)
    rc = lib.orc_worst_case(_p(wf, _i32p), ctypes.c_int(K), ctypes.c_int(l), ctypes.c_int(f), ctypes.c_int(r),
                            ctypes.c_int(q), ctypes.byref(cmax), _p(arg, _i32p), ctypes.byref(n))
    if rc != 0:
        raise ValueError("orc_worst_case rejected q=%d K=%d" % (q, K))
    return int(cmax.value), arg[:q].copy(), int(n.value)


def count_distorted(file_workers, byz) -> int:
    lib = _load()
    fw = np.ascontiguousarray(file_workers, np.int32)
    f, r = fw.shape
    b = np.ascontiguousarray(byz, np.int32)
    return int(lib.orc_count_distorted(_p(fw, _i32p), ctypes.c_int(f), ctypes.c_int(r), _p(b, _i32p),
                                       ctypes.c_int(len(b))))


def model_update(w, g, eta: float, velocity=None, mu: float = 0.0):
    """Eq. (1) step on copies of the state: returns (w_new, velocity_new or None)."""
    lib = _load()
    w = _f32(w).copy()
    g = _f32(g)
    v = None if velocity is None else _f32(velocity).copy()
    lib.orc_model_update(_p(w, _f32p), None if v is None else _p(v, _f32p), _p(g, _f32p), ctypes.c_int64(w.shape[0]),
                         ctypes.c_float(eta), ctypes.c_float(mu))
    return w, v
