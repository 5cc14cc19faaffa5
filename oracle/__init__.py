"""Python access to the CPU oracle (oracle/gc_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the benchmark's CPU
baseline.  The CUDA library and its binding never import this package.

The C file is compiled on first use with gcc (-O2, no fast-math, OpenMP over rows) into
oracle/libgc_oracle.so and loaded through ctypes.  Inputs are widened to float64 exactly;
bf16 problems must already hold bf16-representable values (those values are the instance).
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gc_oracle.c")
_LIB = os.path.join(_HERE, "libgc_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle if the shared object is missing or older than its source."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + f".tmp{os.getpid()}"
    cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        dp = ctypes.POINTER(ctypes.c_double)
        ip = ctypes.POINTER(ctypes.c_int32)
        lp = ctypes.POINTER(ctypes.c_int64)
        i64 = ctypes.c_int64
        lib.gco_num_threads.restype = ctypes.c_int
        lib.gco_build_cache.restype = ctypes.c_int
        lib.gco_build_cache.argtypes = [dp, dp, ip, i64, i64, i64, ctypes.c_double, ctypes.c_int,
                                        dp, dp, dp, dp, dp]
        lib.gco_query_rows.restype = ctypes.c_int
        lib.gco_query_rows.argtypes = [dp, dp, ip, i64, i64, i64, ctypes.c_double, ctypes.c_int,
                                       lp, i64, dp, dp, dp]
        lib.gco_passage_rows.restype = ctypes.c_int
        lib.gco_passage_rows.argtypes = [dp, dp, ip, i64, i64, i64, ctypes.c_double, ctypes.c_int,
                                         dp, lp, i64, dp]
        lib.gco_build_variant.restype = ctypes.c_int
        lib.gco_build_variant.argtypes = [dp, dp, lp, ip, i64, i64, i64, ctypes.c_double,
                                          ctypes.c_int, ctypes.c_int, ctypes.c_int, dp, dp, dp, dp]
        lib.gco_dist_loss.restype = ctypes.c_int
        lib.gco_dist_loss.argtypes = [dp, ip, i64, i64, ctypes.c_double, ctypes.c_int, dp, dp]
        lib.gco_dist_w.restype = ctypes.c_int
        lib.gco_dist_w.argtypes = [dp, ip, i64, i64, ctypes.c_double, ctypes.c_int, dp]
        lib.gco_cache_apply.restype = ctypes.c_int
        lib.gco_cache_apply.argtypes = [dp, dp, i64, i64, i64, ctypes.c_int, dp]
        _lib = lib
    return _lib


def num_threads() -> int:
    return int(_load().gco_num_threads())


def _f64(a):
    return np.ascontiguousarray(a, dtype=np.float64)


def _ptr(a, ty):
    return a.ctypes.data_as(ctypes.POINTER(ty)) if a is not None else None


def _prep(Q, P, pos_idx):
    Q = _f64(Q)
    P = _f64(P)
    pos = np.ascontiguousarray(pos_idx, dtype=np.int32)
    if Q.ndim != 2 or P.ndim != 2 or Q.shape[1] != P.shape[1] or pos.shape != (Q.shape[0],):
        raise ValueError("shape mismatch")
    return Q, P, pos


def build_cache(Q, P, pos_idx, tau=1.0, mask_mode=0, grads=True):
    """Loss of Eq. 1 and its representation gradients (Eq. 5-7).
    Returns dict(loss, row_lse, pos_logit, dQ, dP) in float64 (dQ/dP None unless grads)."""
    Q, P, pos = _prep(Q, P, pos_idx)
    B, d = Q.shape
    N = P.shape[0]
    loss = ctypes.c_double(0.0)
    row_lse = np.empty(B, np.float64)
    pos_logit = np.empty(B, np.float64)
    dQ = np.empty((B, d), np.float64) if grads else None
    dP = np.empty((N, d), np.float64) if grads else None
    rc = _load().gco_build_cache(
        _ptr(Q, ctypes.c_double), _ptr(P, ctypes.c_double), _ptr(pos, ctypes.c_int32), B, N, d,
        float(tau), int(mask_mode), ctypes.byref(loss), _ptr(row_lse, ctypes.c_double),
        _ptr(pos_logit, ctypes.c_double), _ptr(dQ, ctypes.c_double), _ptr(dP, ctypes.c_double))
    if rc != 0:
        raise ValueError(f"oracle rejected the problem (code {rc})")
    return dict(loss=float(loss.value), row_lse=row_lse, pos_logit=pos_logit, dQ=dQ, dP=dP)


def loss_only(Q, P, pos_idx, tau=1.0, mask_mode=0) -> float:
    return build_cache(Q, P, pos_idx, tau, mask_mode, grads=False)["loss"]


def query_rows(Q, P, pos_idx, rows, tau=1.0, mask_mode=0, grads=True):
    """lse_i, S_{i,r_i} and row i of dQ for the listed query rows only."""
    Q, P, pos = _prep(Q, P, pos_idx)
    B, d = Q.shape
    N = P.shape[0]
    rows = np.ascontiguousarray(rows, dtype=np.int64)
    n = rows.shape[0]
    row_lse = np.empty(n, np.float64)
    pos_logit = np.empty(n, np.float64)
    dQ = np.empty((n, d), np.float64) if grads else None
    rc = _load().gco_query_rows(
        _ptr(Q, ctypes.c_double), _ptr(P, ctypes.c_double), _ptr(pos, ctypes.c_int32), B, N, d,
        float(tau), int(mask_mode), _ptr(rows, ctypes.c_int64), n,
        _ptr(row_lse, ctypes.c_double), _ptr(pos_logit, ctypes.c_double),
        _ptr(dQ, ctypes.c_double))
    if rc != 0:
        raise ValueError(f"oracle rejected the problem (code {rc})")
    return dict(row_lse=row_lse, pos_logit=pos_logit, dQ=dQ)


def passage_rows(Q, P, pos_idx, row_lse, rows, tau=1.0, mask_mode=0):
    """Rows of dP for the listed passage rows, given lse_i for every query."""
    Q, P, pos = _prep(Q, P, pos_idx)
    B, d = Q.shape
    N = P.shape[0]
    lse = _f64(row_lse)
    if lse.shape != (B,):
        raise ValueError("row_lse must have one entry per query")
    rows = np.ascontiguousarray(rows, dtype=np.int64)
    n = rows.shape[0]
    dP = np.empty((n, d), np.float64)
    rc = _load().gco_passage_rows(
        _ptr(Q, ctypes.c_double), _ptr(P, ctypes.c_double), _ptr(pos, ctypes.c_int32), B, N, d,
        float(tau), int(mask_mode), _ptr(lse, ctypes.c_double), _ptr(rows, ctypes.c_int64), n,
        _ptr(dP, ctypes.c_double))
    if rc != 0:
        raise ValueError(f"oracle rejected the problem (code {rc})")
    return dP


def build_variant(Q, P, positives, tau=1.0, mask_mode=0, cosine=False, two_direction=False):
    """Loss variants of Section 3.3's Step 2 remark: cosine similarity (gradients with respect to
    the un-normalised rows), several positives per query (`positives`: a list of index lists, or a
    1-D array for one positive each), the two-direction loss, and dL/dtau.
    Returns dict(loss, dQ, dP, dtau) in float64."""
    Q = _f64(Q)
    P = _f64(P)
    B, d = Q.shape
    N = P.shape[0]
    if isinstance(positives, np.ndarray) and positives.ndim == 1:
        lists = [[int(v)] for v in positives]
    else:
        lists = [[int(v) for v in row] for row in positives]
    if len(lists) != B or P.shape[1] != d:
        raise ValueError("shape mismatch")
    ptr = np.zeros(B + 1, np.int64)
    ptr[1:] = np.cumsum([len(r) for r in lists])
    flat = np.ascontiguousarray([v for r in lists for v in r], dtype=np.int32)
    loss, dtau = ctypes.c_double(0.0), ctypes.c_double(0.0)
    dQ = np.empty((B, d), np.float64)
    dP = np.empty((N, d), np.float64)
    rc = _load().gco_build_variant(
        _ptr(Q, ctypes.c_double), _ptr(P, ctypes.c_double), _ptr(ptr, ctypes.c_int64),
        _ptr(flat, ctypes.c_int32), B, N, d, float(tau), int(mask_mode), int(bool(cosine)),
        int(bool(two_direction)), ctypes.byref(loss), _ptr(dQ, ctypes.c_double),
        _ptr(dP, ctypes.c_double), ctypes.byref(dtau))
    if rc != 0:
        raise ValueError(f"oracle rejected the problem (code {rc})")
    return dict(loss=float(loss.value), dQ=dQ, dP=dP, dtau=float(dtau.value))


def dist_loss(D, pos_idx, tau=1.0, mask_mode=0):
    """Section 5: the loss of Eq. 1 as a function of the matrix of distances D [B x N] (logit of a
    pair = d_ij / tau).  Returns dict(loss, row_lse)."""
    D = _f64(D)
    B, N = D.shape
    pos = np.ascontiguousarray(pos_idx, dtype=np.int32)
    loss = ctypes.c_double(0.0)
    lse = np.empty(B, np.float64)
    rc = _load().gco_dist_loss(_ptr(D, ctypes.c_double), _ptr(pos, ctypes.c_int32), B, N, float(tau),
                               int(mask_mode), ctypes.byref(loss), _ptr(lse, ctypes.c_double))
    if rc != 0:
        raise ValueError(f"oracle rejected the problem (code {rc})")
    return dict(loss=float(loss.value), row_lse=lse)


def dist_w(D, pos_idx, tau=1.0, mask_mode=0):
    """Section 5: the Distance Gradient Cache w_ij = dL/dd_ij as a B x N float64 matrix."""
    D = _f64(D)
    B, N = D.shape
    pos = np.ascontiguousarray(pos_idx, dtype=np.int32)
    W = np.empty((B, N), np.float64)
    rc = _load().gco_dist_w(_ptr(D, ctypes.c_double), _ptr(pos, ctypes.c_int32), B, N, float(tau),
                            int(mask_mode), _ptr(W, ctypes.c_double))
    if rc != 0:
        raise ValueError(f"oracle rejected the problem (code {rc})")
    return W


def cache_apply(U, X, dW=None):
    """Eq. 8 / Eq. 9 for a linear encoder: returns dW (+)= U^T X in float64, where U [rows x d]
    is a slice of the cache and X [rows x d_in] the encoder inputs of the same sub-batch.  With
    dW given (d x d_in, float64, contiguous) the sum is added to it in place."""
    U = _f64(U)
    X = _f64(X)
    if U.ndim != 2 or X.ndim != 2 or U.shape[0] != X.shape[0]:
        raise ValueError("shape mismatch")
    rows, d = U.shape
    d_in = X.shape[1]
    acc = dW is not None
    if acc:
        if dW.dtype != np.float64 or dW.shape != (d, d_in) or not dW.flags.c_contiguous:
            raise ValueError("dW must be a contiguous float64 array of shape (d, d_in)")
    else:
        dW = np.empty((d, d_in), np.float64)
    rc = _load().gco_cache_apply(_ptr(U, ctypes.c_double), _ptr(X, ctypes.c_double), rows, d, d_in,
                                 int(acc), _ptr(dW, ctypes.c_double))
    if rc != 0:
        raise ValueError(f"oracle rejected the problem (code {rc})")
    return dW
