"""fp64 CPU oracle for the TT-embedding gather -- TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the benchmark's CPU legs may import this package.  It never imports
the CUDA package and the CUDA package never imports it.  The arithmetic lives in `tt_oracle.c`
(plain C, one lookup at a time) and in `tt_oracle_memo.c` (the same definition with each distinct row built
once, so that the full-size configurations finish in test time; the two files share no code and are compared
with each other by the tests); this file marshals numpy arrays and holds the integer grouping oracle
(Sec. 3.3: sort, unique, mixed radix, run-length encoding), written with numpy's sort as the one
library primitive.

Cores are passed as fp64 arrays of shape (r_{k-1}, n_k, d_k, r_k).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import List, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SO = os.path.join(_HERE, "libtt_oracle.so")
_SRC = os.path.join(_HERE, "tt_oracle.c")
_SO_MEMO = os.path.join(_HERE, "libtt_oracle_memo.so")
_SRC_MEMO = os.path.join(_HERE, "tt_oracle_memo.c")
_lib = None
_lib_memo = None


def build(force: bool = False) -> str:
    """Compile tt_oracle.c and tt_oracle_memo.c with gcc into shared libraries next to the sources."""
    for so, src, opt in ((_SO, _SRC, "-O2"), (_SO_MEMO, _SRC_MEMO, "-O3")):
        if force or not os.path.exists(so) or os.path.getmtime(so) < os.path.getmtime(src):
            cmd = ["gcc", opt, "-fopenmp", "-shared", "-fPIC", "-std=c11", "-o", so, src, "-lm"]
            subprocess.run(cmd, check=True)
    return _SO


def lib():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_SO)
        _lib.tt_oracle_forward.restype = ctypes.c_int64
        _lib.tt_oracle_backward.restype = ctypes.c_int64
    return _lib


def lib_memo():
    global _lib_memo
    if _lib_memo is None:
        build()
        _lib_memo = ctypes.CDLL(_SO_MEMO)
        _lib_memo.tt_memo_forward.restype = ctypes.c_int64
        _lib_memo.tt_memo_backward.restype = ctypes.c_int64
    return _lib_memo


def _i64(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.int64))


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _core_ptrs(cores: Sequence[np.ndarray]):
    keep = [np.ascontiguousarray(np.asarray(c, dtype=np.float64)) for c in cores]
    arr = (ctypes.c_void_p * len(keep))(*[c.ctypes.data for c in keep])
    return keep, arr


def _check(n, d, r, cores):
    K = len(n)
    assert len(d) == K and len(r) == K + 1 and r[0] == 1 and r[K] == 1 and 2 <= K <= 8
    for k, c in enumerate(cores):
        assert tuple(c.shape) == (r[k], n[k], d[k], r[k + 1]), (k, c.shape)


def digits(g: int, n: Sequence[int]) -> tuple:
    """Eq. 1 for one row id."""
    nn = _i64(n)
    out = np.zeros(len(n), dtype=np.int64)
    lib().tt_oracle_digits(ctypes.c_int64(int(g)), ctypes.c_int(len(n)), _p(nn), _p(out))
    return tuple(int(x) for x in out)


def row(n, d, r, cores, g: int) -> np.ndarray:
    _check(n, d, r, cores)
    nn, dd, rr = _i64(n), _i64(d), _i64(r)
    keep, cp = _core_ptrs(cores)
    E = np.zeros(int(np.prod(d)), dtype=np.float64)
    lib().tt_oracle_row(ctypes.c_int(len(n)), _p(nn), _p(dd), _p(rr), cp, ctypes.c_int64(int(g)), _p(E))
    return E


def _weights_arg(weights, L):
    if weights is None:
        return None, ctypes.c_void_p(None)
    w = np.ascontiguousarray(np.asarray(weights, dtype=np.float64))
    assert w.shape == (L,)
    return w, _p(w)


def forward(n, d, r, N, cores, indices, offsets, weights=None, mode: str = "sum", memo: bool = False) -> np.ndarray:
    """Pooled rows of one table: fp64 [B, D].  weights: per-lookup factors [L]; mode "sum" (the paper) or "mean".
    memo=True: the memoised oracle (every distinct row built once) instead of the plain per-lookup one."""
    _check(n, d, r, cores)
    nn, dd, rr = _i64(n), _i64(d), _i64(r)
    idx, off = _i64(indices), _i64(offsets)
    B = off.shape[0] - 1
    D = int(np.prod(d))
    keep, cp = _core_ptrs(cores)
    out = np.zeros((B, D), dtype=np.float64)
    wkeep, wp = _weights_arg(weights, idx.shape[0])
    fn = lib_memo().tt_memo_forward if memo else lib().tt_oracle_forward
    fn(ctypes.c_int(len(n)), _p(nn), _p(dd), _p(rr), ctypes.c_int64(int(N)), cp,
                            _p(idx), _p(off), ctypes.c_int64(B), _p(out), ctypes.c_int64(D), wp,
                            ctypes.c_int(1 if mode == "mean" else 0))
    return out


def backward(n, d, r, N, cores, indices, offsets, grad_out, weights=None, mode: str = "sum",
             memo: bool = False) -> List[np.ndarray]:
    """Core gradients of one table for loss = sum(grad_out * out): list of fp64 arrays shaped like the cores.
    memo=True: the memoised oracle (grad_out summed per distinct row first, one backward chain per distinct row)."""
    _check(n, d, r, cores)
    nn, dd, rr = _i64(n), _i64(d), _i64(r)
    idx, off = _i64(indices), _i64(offsets)
    B = off.shape[0] - 1
    D = int(np.prod(d))
    go = np.ascontiguousarray(np.asarray(grad_out, dtype=np.float64))
    assert go.shape == (B, D)
    keep, cp = _core_ptrs(cores)
    grads = [np.zeros(c.shape, dtype=np.float64) for c in keep]
    gp = (ctypes.c_void_p * len(grads))(*[g.ctypes.data for g in grads])
    wkeep, wp = _weights_arg(weights, idx.shape[0])
    fn = lib_memo().tt_memo_backward if memo else lib().tt_oracle_backward
    fn(ctypes.c_int(len(n)), _p(nn), _p(dd), _p(rr), ctypes.c_int64(int(N)), cp,
                             _p(idx), _p(off), ctypes.c_int64(B), _p(go), ctypes.c_int64(D), gp, wp,
                             ctypes.c_int(1 if mode == "mean" else 0))
    return grads


def dense(n, d, r, cores) -> np.ndarray:
    """Brute-force table W[prod(n), D] straight from the definition (tiny tables only)."""
    _check(n, d, r, cores)
    nn, dd, rr = _i64(n), _i64(d), _i64(r)
    keep, cp = _core_ptrs(cores)
    W = np.zeros((int(np.prod(n)), int(np.prod(d))), dtype=np.float64)
    lib().tt_oracle_dense(ctypes.c_int(len(n)), _p(nn), _p(dd), _p(rr), cp, _p(W))
    return W


def sgd(cores: Sequence[np.ndarray], grads: Sequence[np.ndarray], lr: float) -> List[np.ndarray]:
    out = []
    for c, g in zip(cores, grads):
        c2 = np.ascontiguousarray(np.asarray(c, dtype=np.float64)).copy()
        g2 = np.ascontiguousarray(np.asarray(g, dtype=np.float64))
        lib().tt_oracle_sgd(_p(c2), _p(g2), ctypes.c_int64(c2.size), ctypes.c_double(float(lr)))
        out.append(c2)
    return out


# ----------------------------------------------------------------------------- multi-table wrappers

def _table_weights(wl, t, weights):
    if weights is None:
        return None
    lo, hi = int(wl.offsets[t * wl.B]), int(wl.offsets[(t + 1) * wl.B])
    return np.asarray(weights)[lo:hi]


def forward_workload(wl, tables=None, bags=None, weights=None, mode: str = "sum", memo: bool = False) -> np.ndarray:
    """out fp64 [B, T*D] for a workloads.Workload (optionally only some tables; others stay zero).
    weights: per-lookup factors aligned with wl.indices."""
    D = wl.D
    out = np.zeros((wl.B, wl.T * D), dtype=np.float64)
    for t in (range(wl.T) if tables is None else tables):
        s = wl.tables[t]
        idx, off = wl.table_slice(t)
        out[:, t * D:(t + 1) * D] = forward(s.n, s.d, s.r, s.N, wl.cores[t], idx, off,
                                            _table_weights(wl, t, weights), mode, memo)
    return out


def backward_workload(wl, grad_out=None, tables=None, weights=None, mode: str = "sum",
                      memo: bool = False) -> List[List[np.ndarray]]:
    go = wl.grad_out if grad_out is None else grad_out
    D = wl.D
    res = []
    for t in (range(wl.T) if tables is None else tables):
        s = wl.tables[t]
        idx, off = wl.table_slice(t)
        res.append(backward(s.n, s.d, s.r, s.N, wl.cores[t], idx, off, go[:, t * D:(t + 1) * D],
                            _table_weights(wl, t, weights), mode, memo))
    return res


def forward_bags(wl, pairs) -> np.ndarray:
    """Pooled output of selected (table, bag) pairs only: fp64 [len(pairs), D]."""
    res = np.zeros((len(pairs), wl.D), dtype=np.float64)
    for i, (t, b) in enumerate(pairs):
        s = wl.tables[t]
        lo, hi = wl.offsets[t * wl.B + b], wl.offsets[t * wl.B + b + 1]
        res[i] = forward(s.n, s.d, s.r, s.N, wl.cores[t], wl.indices[lo:hi], np.array([0, hi - lo]))[0]
    return res


# ----------------------------------------------------------------------------- grouping (integers)

def grouping(n: Sequence[int], indices) -> dict:
    """Sec. 3.3 for one table: ascending unique rows, and for each prefix length k = 1..K-1 the
    run-length encoding of floor(row / prod_{j>k} n_j) over them.

    Returns
      uniq            int64 [U]    ascending distinct row ids
      inv             int64 [L]    uniq[inv[l]] == indices[l]
      mult            int64 [U]    number of lookups per unique row
      digits          int64 [U,K]  Eq. 1 digits of each unique row
      levels[k-1]     dict(vals, row_counts, lookup_counts) for prefix length k: ascending prefix
                      values, unique rows under each, lookups under each
    """
    idx = _i64(indices)
    K = len(n)
    uniq, inv, mult = np.unique(idx, return_inverse=True, return_counts=True)
    digs = np.zeros((uniq.shape[0], K), dtype=np.int64)
    suffix = 1
    for k in range(K - 1, -1, -1):
        digs[:, k] = (uniq // suffix) % n[k]
        suffix *= n[k]
    levels = []
    for k in range(1, K):
        s = int(np.prod(n[k:]))
        pref = uniq // s
        vals, start, rc = np.unique(pref, return_index=True, return_counts=True)
        lc = np.add.reduceat(mult, start) if uniq.shape[0] else np.zeros(0, np.int64)
        levels.append(dict(vals=vals.astype(np.int64), row_counts=rc.astype(np.int64),
                           lookup_counts=np.asarray(lc, dtype=np.int64)))
    return dict(uniq=uniq, inv=inv.astype(np.int64), mult=mult.astype(np.int64), digits=digs, levels=levels)
