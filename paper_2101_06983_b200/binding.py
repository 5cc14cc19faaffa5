"""Thin ctypes binding over libgradcache.so (include/gradcache.h).

Argument marshalling only: torch tensors supply device memory and the current CUDA stream;
every numerical step runs inside the library's kernels.  There is no CPU fallback: if the
shared library is missing the import fails, and the calls need a CUDA device.
"""
from __future__ import annotations

import ctypes
import os

import torch

from . import _build

GC_F32, GC_BF16 = 0, 1
GC_MASK_NONE, GC_MASK_SELF = 0, 1
GC_OP_FWD, GC_OP_BWD, GC_OP_BUILD, GC_OP_BUILD_STORED = 0, 1, 2, 3
GC_DEV_POS_RANGE, GC_DEV_POS_MASKED, GC_DEV_WAIT_LIMIT = 1, 2, 4

EXPORTS = ("gc_workspace_bytes", "gc_plan_name", "gc_kernel_launches", "gc_loss_fwd",
           "gc_loss_bwd", "gc_build_cache", "gc_build_cache_stored", "gc_status_string",
           "gc_profile_enable",
           "gc_profile_read", "gc_profile_read_call", "gc_static_scratch_need", "gc_loss_fwd_static",
           "gc_cache_apply_workspace_bytes", "gc_cache_apply", "gc_shard_workspace_bytes",
           "gc_shard_fwd_dq", "gc_shard_dp", "gc_selftest_wait_limit", "gc_row_normalize",
           "gc_cosine_bwd", "gc_dtau_workspace_bytes", "gc_dtau", "gc_dist_begin",
           "gc_dist_accumulate", "gc_dist_finish", "gc_dist_w_block", "gc_dist_dot_block",
           "gc_multi_pos_workspace_bytes", "gc_build_cache_multi_pos",
           "gc_two_direction_workspace_bytes", "gc_build_cache_two_direction")
GC_STATIC_SCRATCH_BYTES = 2 << 20


class GradCacheError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (gc_status {status})")


def _load() -> ctypes.CDLL:
    path = _build.LIB
    if not os.path.exists(path):
        raise ImportError(
            f"{path} is missing: build it with `python -m paper_2101_06983_b200._build` "
            "(there is no fallback implementation)")
    lib = ctypes.CDLL(path)
    vp, i64, i32, f32 = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_float
    common = [vp, i64, vp, i64, vp, i64, i64, i32, f32, i32, i32]
    lib.gc_workspace_bytes.restype = ctypes.c_size_t
    lib.gc_workspace_bytes.argtypes = [i32, i64, i64, i32, i32]
    lib.gc_plan_name.restype = ctypes.c_char_p
    lib.gc_plan_name.argtypes = [i32, i64, i64, i32, i32]
    lib.gc_kernel_launches.restype = i32
    lib.gc_kernel_launches.argtypes = [i32, i64, i64, i32, i32]
    lib.gc_status_string.restype = ctypes.c_char_p
    lib.gc_status_string.argtypes = [i32]
    lib.gc_loss_fwd.restype = i32
    lib.gc_loss_fwd.argtypes = common + [vp, vp, vp, vp, ctypes.c_size_t, vp, vp]
    lib.gc_loss_bwd.restype = i32
    lib.gc_loss_bwd.argtypes = common + [vp, vp, i64, vp, i64, vp, ctypes.c_size_t, vp, vp]
    lib.gc_build_cache.restype = i32
    lib.gc_build_cache.argtypes = common + [vp, vp, vp, vp, i64, vp, i64, vp, ctypes.c_size_t,
                                            vp, vp]
    lib.gc_build_cache_stored.restype = i32
    lib.gc_build_cache_stored.argtypes = lib.gc_build_cache.argtypes
    lib.gc_static_scratch_need.restype = ctypes.c_size_t
    lib.gc_static_scratch_need.argtypes = [i64, i64, i32, i32]
    lib.gc_loss_fwd_static.restype = i32
    lib.gc_loss_fwd_static.argtypes = common + [vp, vp, vp, vp, vp]
    lib.gc_cache_apply_workspace_bytes.restype = ctypes.c_size_t
    lib.gc_cache_apply_workspace_bytes.argtypes = [i64, i32, i32]
    lib.gc_cache_apply.restype = i32
    lib.gc_cache_apply.argtypes = [vp, i64, vp, i64, i64, i32, i32, i32, vp, i64, i32, vp,
                                   ctypes.c_size_t, vp, vp]
    lib.gc_shard_workspace_bytes.restype = ctypes.c_size_t
    lib.gc_shard_workspace_bytes.argtypes = [i64, i64, i32, i32, i64, i64]
    lib.gc_shard_fwd_dq.restype = i32
    lib.gc_shard_fwd_dq.argtypes = common + [i64, i64, vp, vp, vp, vp, i64, vp, ctypes.c_size_t,
                                             vp, vp]
    lib.gc_shard_dp.restype = i32
    lib.gc_shard_dp.argtypes = common + [vp, i64, i64, vp, i64, vp, ctypes.c_size_t, vp, vp]
    lib.gc_row_normalize.restype = i32
    lib.gc_row_normalize.argtypes = [vp, i64, i64, i32, i32, vp, i64, vp, vp]
    lib.gc_cosine_bwd.restype = i32
    lib.gc_cosine_bwd.argtypes = [vp, i64, i64, i32, i32, vp, vp, i64, vp, i64, vp]
    lib.gc_dtau_workspace_bytes.restype = ctypes.c_size_t
    lib.gc_dtau_workspace_bytes.argtypes = [i64]
    lib.gc_dtau.restype = i32
    lib.gc_dtau.argtypes = [vp, i64, vp, i64, i64, i32, f32, i32, vp, vp, ctypes.c_size_t, vp]
    lib.gc_multi_pos_workspace_bytes.restype = ctypes.c_size_t
    lib.gc_multi_pos_workspace_bytes.argtypes = [i64, i64, i32, i32, i64]
    lib.gc_build_cache_multi_pos.restype = i32
    lib.gc_build_cache_multi_pos.argtypes = [vp, i64, vp, i64, vp, vp, i64, i64, i64, i32, f32, i32,
                                             i32, vp, vp, vp, i64, vp, i64, vp, ctypes.c_size_t,
                                             vp, vp]
    lib.gc_two_direction_workspace_bytes.restype = ctypes.c_size_t
    lib.gc_two_direction_workspace_bytes.argtypes = [i64, i64, i32, i32]
    lib.gc_build_cache_two_direction.restype = i32
    lib.gc_build_cache_two_direction.argtypes = [vp, i64, vp, i64, vp, i64, i64, i32, f32, i32, vp,
                                                 vp, vp, i64, vp, i64, vp, ctypes.c_size_t, vp, vp]
    lib.gc_dist_begin.restype = i32
    lib.gc_dist_begin.argtypes = [vp, vp, vp, i64, vp]
    lib.gc_dist_accumulate.restype = i32
    lib.gc_dist_accumulate.argtypes = [vp, i64, i64, i64, i64, i64, vp, i64, i64, f32, i32, vp, vp, vp, vp]
    lib.gc_dist_finish.restype = i32
    lib.gc_dist_finish.argtypes = [vp, vp, vp, vp, i64, i64, i32, vp, vp, vp, vp]
    lib.gc_dist_w_block.restype = i32
    lib.gc_dist_w_block.argtypes = [vp, i64, i64, i64, i64, i64, vp, vp, i64, i64, f32, i32, vp, i64, vp]
    lib.gc_dist_dot_block.restype = i32
    lib.gc_dist_dot_block.argtypes = [vp, i64, vp, i64, i64, i64, i32, i32, i64, i64, i64, i64, vp, i64, vp]
    lib.gc_selftest_wait_limit.restype = i32
    lib.gc_selftest_wait_limit.argtypes = [ctypes.c_uint64, vp, vp, vp]
    lib.gc_profile_enable.restype = i32
    lib.gc_profile_enable.argtypes = [i32]
    lib.gc_profile_read.restype = i32
    lib.gc_profile_read.argtypes = [ctypes.POINTER(f32)] * 3
    lib.gc_profile_read_call.restype = i32
    lib.gc_profile_read_call.argtypes = [i64] + [ctypes.POINTER(f32)] * 3
    return lib


_lib = _load()


def status_string(status: int) -> str:
    return _lib.gc_status_string(int(status)).decode()


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return GC_F32
    if t.dtype == torch.bfloat16:
        return GC_BF16
    raise TypeError(f"Q/P must be float32 or bfloat16, got {t.dtype}")


def gc_workspace_bytes(op: int, B: int, N: int, d: int, dtype: int) -> int:
    return int(_lib.gc_workspace_bytes(op, B, N, d, dtype))


def gc_plan_name(op: int, B: int, N: int, d: int, dtype: int) -> str:
    return _lib.gc_plan_name(op, B, N, d, dtype).decode()


def gc_kernel_launches(op: int, B: int, N: int, d: int, dtype: int) -> int:
    return int(_lib.gc_kernel_launches(op, B, N, d, dtype))


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _common(Q, P, pos_idx, tau, mask_mode):
    if Q.dim() != 2 or P.dim() != 2 or Q.stride(1) != 1 or P.stride(1) != 1:
        raise ValueError("Q and P must be 2-D with unit stride along d")
    if pos_idx.dtype != torch.int32 or not pos_idx.is_contiguous():
        raise TypeError("pos_idx must be a contiguous int32 tensor")
    if P.dtype != Q.dtype or P.shape[1] != Q.shape[1]:
        raise ValueError("Q and P must share dtype and width")
    B, d = Q.shape
    N = P.shape[0]
    code = _dtype_code(Q)
    args = [_ptr(Q), Q.stride(0), _ptr(P), P.stride(0), _ptr(pos_idx), B, N, d, float(tau),
            int(mask_mode), code]
    return args, B, N, d, code


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def alloc_workspace(op: int, B: int, N: int, d: int, dtype: int, device) -> torch.Tensor:
    """A workspace tensor of the size gc_workspace_bytes reports (torch memory is 512-byte
    aligned, which covers the 256-byte requirement)."""
    n = max(gc_workspace_bytes(op, B, N, d, dtype), 256)
    return torch.empty(n, dtype=torch.uint8, device=device)


def gc_loss_fwd(Q, P, pos_idx, tau, mask_mode, loss, row_lse, pos_logit=None, ws=None,
                dev_status=None):
    """Eq. 1: writes loss[1], row_lse[B] and optionally pos_logit[B] (all float32 on device)."""
    args, B, N, d, code = _common(Q, P, pos_idx, tau, mask_mode)
    if ws is None:
        ws = alloc_workspace(GC_OP_FWD, B, N, d, code, Q.device)
    rc = _lib.gc_loss_fwd(*args, _ptr(loss), _ptr(row_lse), _ptr(pos_logit), _ptr(ws),
                          ws.numel(), _ptr(dev_status), _stream())
    if rc != 0:
        raise GradCacheError(rc, "gc_loss_fwd")


def gc_static_scratch_need(B: int, N: int, d: int, dtype: int) -> int:
    return int(_lib.gc_static_scratch_need(B, N, d, dtype))


def gc_loss_fwd_static(Q, P, pos_idx, tau, mask_mode, loss, row_lse, pos_logit=None,
                       dev_status=None):
    """gc_loss_fwd without a caller workspace: the scratch is a fixed array inside the library
    (GC_STATIC_SCRATCH_BYTES).  Nothing is allocated by the call; all outputs are the caller's.
    Raises GradCacheError with GC_ERR_LIMIT (9) when the problem needs more scratch than that.
    Calls on one device share the array, so they must not overlap on the GPU."""
    args, B, N, d, code = _common(Q, P, pos_idx, tau, mask_mode)
    rc = _lib.gc_loss_fwd_static(*args, _ptr(loss), _ptr(row_lse), _ptr(pos_logit),
                                 _ptr(dev_status), _stream())
    if rc != 0:
        raise GradCacheError(rc, "gc_loss_fwd_static")


def gc_loss_bwd(Q, P, pos_idx, tau, mask_mode, row_lse, dQ, dP, ws=None, dev_status=None):
    """Eq. 5-7 given row_lse: overwrites dQ[B x d] and dP[N x d] (either may be None)."""
    args, B, N, d, code = _common(Q, P, pos_idx, tau, mask_mode)
    if ws is None:
        ws = alloc_workspace(GC_OP_BWD, B, N, d, code, Q.device)
    rc = _lib.gc_loss_bwd(*args, _ptr(row_lse), _ptr(dQ), 0 if dQ is None else dQ.stride(0),
                          _ptr(dP), 0 if dP is None else dP.stride(0), _ptr(ws), ws.numel(),
                          _ptr(dev_status), _stream())
    if rc != 0:
        raise GradCacheError(rc, "gc_loss_bwd")


def gc_build_cache(Q, P, pos_idx, tau, mask_mode, loss, row_lse, dQ, dP, pos_logit=None,
                   ws=None, dev_status=None):
    """Step 2 of Section 3.3: loss, row_lse and the representation gradient cache dQ, dP."""
    args, B, N, d, code = _common(Q, P, pos_idx, tau, mask_mode)
    if ws is None:
        ws = alloc_workspace(GC_OP_BUILD, B, N, d, code, Q.device)
    rc = _lib.gc_build_cache(*args, _ptr(loss), _ptr(row_lse), _ptr(pos_logit), _ptr(dQ),
                             dQ.stride(0), _ptr(dP), dP.stride(0), _ptr(ws), ws.numel(),
                             _ptr(dev_status), _stream())
    if rc != 0:
        raise GradCacheError(rc, "gc_build_cache")


def gc_build_cache_stored(Q, P, pos_idx, tau, mask_mode, loss, row_lse, dQ, dP, pos_logit=None,
                          ws=None, dev_status=None):
    """gc_build_cache by way of a stored B x N bf16 weight matrix and two GEMMs (comparison plan)."""
    args, B, N, d, code = _common(Q, P, pos_idx, tau, mask_mode)
    if ws is None:
        ws = alloc_workspace(GC_OP_BUILD_STORED, B, N, d, code, Q.device)
    rc = _lib.gc_build_cache_stored(*args, _ptr(loss), _ptr(row_lse), _ptr(pos_logit), _ptr(dQ),
                                    dQ.stride(0), _ptr(dP), dP.stride(0), _ptr(ws), ws.numel(),
                                    _ptr(dev_status), _stream())
    if rc != 0:
        raise GradCacheError(rc, "gc_build_cache_stored")


def gc_cache_apply_workspace_bytes(rows: int, d: int, d_in: int) -> int:
    return int(_lib.gc_cache_apply_workspace_bytes(rows, d, d_in))


def gc_cache_apply(U, X, dW, accumulate: bool, ws=None, dev_status=None):
    """Step 3 for a linear encoder (Eq. 8-9): dW[d x d_in] (+)= U^T X with U [rows x d] float32
    (rows of the cache) and X [rows x d_in] bfloat16 (the same rows' encoder inputs)."""
    if U.dim() != 2 or X.dim() != 2 or dW.dim() != 2 or U.stride(1) != 1 or X.stride(1) != 1 \
            or dW.stride(1) != 1:
        raise ValueError("U, X and dW must be 2-D with unit stride along their rows")
    if U.dtype != torch.float32 or dW.dtype != torch.float32:
        raise TypeError("U and dW must be float32")
    rows, d = U.shape
    d_in = X.shape[1]
    if X.shape[0] != rows or tuple(dW.shape) != (d, d_in):
        raise ValueError("shape mismatch")
    if ws is None:
        ws = torch.empty(max(gc_cache_apply_workspace_bytes(rows, d, d_in), 256),
                         dtype=torch.uint8, device=U.device)
    rc = _lib.gc_cache_apply(_ptr(U), U.stride(0), _ptr(X), X.stride(0), rows, d, d_in,
                             _dtype_code(X), _ptr(dW), dW.stride(0), 1 if accumulate else 0,
                             _ptr(ws), ws.numel(), _ptr(dev_status), _stream())
    if rc != 0:
        raise GradCacheError(rc, "gc_cache_apply")


def gc_shard_workspace_bytes(B: int, N: int, d: int, dtype: int, q_count: int, p_count: int) -> int:
    return int(_lib.gc_shard_workspace_bytes(B, N, d, dtype, q_count, p_count))


def gc_shard_fwd_dq(Q, P, pos_idx, tau, q0, q_count, loss_part, row_lse, dQ, pos_logit=None,
                    ws=None, dev_status=None, mask_mode=GC_MASK_NONE):
    """Section 3.4, local queries [q0, q0 + q_count) of the gathered batch: writes their entries
    of row_lse[B], dQ[q_count x d] and loss_part[1] (this rank's share of the loss of Eq. 1)."""
    args, B, N, d, code = _common(Q, P, pos_idx, tau, mask_mode)
    if ws is None:
        ws = torch.empty(max(gc_shard_workspace_bytes(B, N, d, code, q_count, N), 256),
                         dtype=torch.uint8, device=Q.device)
    rc = _lib.gc_shard_fwd_dq(*args, q0, q_count, _ptr(loss_part), _ptr(row_lse), _ptr(pos_logit),
                              _ptr(dQ), dQ.stride(0), _ptr(ws), ws.numel(), _ptr(dev_status),
                              _stream())
    if rc != 0:
        raise GradCacheError(rc, "gc_shard_fwd_dq")


def gc_shard_dp(Q, P, pos_idx, tau, row_lse, p0, p_count, dP, ws=None, dev_status=None,
                mask_mode=GC_MASK_NONE):
    """Section 3.4, local passages [p0, p0 + p_count) of the gathered batch, given row_lse of all
    B queries: writes dP[p_count x d]."""
    args, B, N, d, code = _common(Q, P, pos_idx, tau, mask_mode)
    if ws is None:
        ws = torch.empty(max(gc_shard_workspace_bytes(B, N, d, code, B, p_count), 256),
                         dtype=torch.uint8, device=Q.device)
    rc = _lib.gc_shard_dp(*args, _ptr(row_lse), p0, p_count, _ptr(dP), dP.stride(0), _ptr(ws),
                          ws.numel(), _ptr(dev_status), _stream())
    if rc != 0:
        raise GradCacheError(rc, "gc_shard_dp")


def gc_row_normalize(X, Xn, inv_norm) -> None:
    """Xn[i] = X[i]/|X[i]| (dtype of X) and inv_norm[i] = 1/|X[i]| (float32): the unit rows of the
    cosine-similarity loss."""
    rows, d = X.shape
    rc = _lib.gc_row_normalize(_ptr(X), X.stride(0), rows, d, _dtype_code(X), _ptr(Xn),
                               Xn.stride(0), _ptr(inv_norm), _stream())
    if rc != 0:
        raise GradCacheError(rc, "gc_row_normalize")


def gc_cosine_bwd(X, inv_norm, dXn, dX) -> None:
    """dX[i] = inv_norm[i] (dXn[i] - n_i <n_i, dXn[i]>): cache rows of the unit rows taken back
    through the normalisation (dX may be dXn)."""
    rows, d = X.shape
    rc = _lib.gc_cosine_bwd(_ptr(X), X.stride(0), rows, d, _dtype_code(X), _ptr(inv_norm),
                            _ptr(dXn), dXn.stride(0), _ptr(dX), dX.stride(0), _stream())
    if rc != 0:
        raise GradCacheError(rc, "gc_cosine_bwd")


def gc_dtau(Q, dQ, tau, dtau, ws=None) -> None:
    """dtau[0] = dL/dtau = -(1/tau) sum_i <Q_i, dQ_i> (Q: the rows the sweeps saw)."""
    B, d = Q.shape
    if ws is None:
        ws = torch.empty(max(int(_lib.gc_dtau_workspace_bytes(B)), 256), dtype=torch.uint8,
                         device=Q.device)
    rc = _lib.gc_dtau(_ptr(Q), Q.stride(0), _ptr(dQ), dQ.stride(0), B, d, float(tau),
                      _dtype_code(Q), _ptr(dtau), _ptr(ws), ws.numel(), _stream())
    if rc != 0:
        raise GradCacheError(rc, "gc_dtau")


def gc_build_cache_multi_pos(Q, P, pos_ptr, pos_list, tau, mask_mode, loss, row_lse, dQ, dP,
                             ws=None, dev_status=None) -> None:
    """Several positives per query (CSR lists pos_ptr [B + 1], pos_list, int32): loss and cache
    rows of the mean-over-positives loss (Section 3.3, Step 2)."""
    B, d = Q.shape
    N = P.shape[0]
    n_pos = pos_list.numel()
    code = _dtype_code(Q)
    if ws is None:
        ws = torch.empty(max(int(_lib.gc_multi_pos_workspace_bytes(B, N, d, code, n_pos)), 256),
                         dtype=torch.uint8, device=Q.device)
    rc = _lib.gc_build_cache_multi_pos(_ptr(Q), Q.stride(0), _ptr(P), P.stride(0), _ptr(pos_ptr),
                                       _ptr(pos_list), n_pos, B, N, d, float(tau), int(mask_mode),
                                       code, _ptr(loss), _ptr(row_lse), _ptr(dQ), dQ.stride(0),
                                       _ptr(dP), dP.stride(0), _ptr(ws), ws.numel(),
                                       _ptr(dev_status), _stream())
    if rc != 0:
        raise GradCacheError(rc, "gc_build_cache_multi_pos")


def gc_build_cache_two_direction(Q, P, pos_idx, tau, loss, row_lse, dQ, dP, ws=None,
                                 dev_status=None) -> None:
    """L = (L_row + L_col) / 2 over the B positive pairs (Section 3.3, Step 2), no mask."""
    B, d = Q.shape
    N = P.shape[0]
    code = _dtype_code(Q)
    if ws is None:
        ws = torch.empty(max(int(_lib.gc_two_direction_workspace_bytes(B, N, d, code)), 256),
                         dtype=torch.uint8, device=Q.device)
    rc = _lib.gc_build_cache_two_direction(_ptr(Q), Q.stride(0), _ptr(P), P.stride(0),
                                           _ptr(pos_idx), B, N, d, float(tau), code, _ptr(loss),
                                           _ptr(row_lse), _ptr(dQ), dQ.stride(0), _ptr(dP),
                                           dP.stride(0), _ptr(ws), ws.numel(), _ptr(dev_status),
                                           _stream())
    if rc != 0:
        raise GradCacheError(rc, "gc_build_cache_two_direction")


class DistanceCache:
    """Section 5 in tiled form: per-row state of the first pass over the distance blocks, then
    row_lse / loss, then blocks of the Distance Gradient Cache w = dL/dd.  Marshalling only."""

    def __init__(self, pos_idx, B, N, tau, mask_mode=GC_MASK_NONE):
        dev = pos_idx.device
        self.pos, self.B, self.N, self.tau, self.mask = pos_idx, B, N, float(tau), int(mask_mode)
        self.run_m = torch.empty(B, device=dev)
        self.run_l = torch.empty(B, device=dev)
        self.pos_d = torch.empty(B, device=dev)
        self.row_lse = torch.empty(B, device=dev)
        self.loss = torch.zeros(1, device=dev)
        self.dev_status = torch.zeros(1, dtype=torch.int32, device=dev)
        rc = _lib.gc_dist_begin(_ptr(self.run_m), _ptr(self.run_l), _ptr(self.pos_d), B, _stream())
        if rc != 0:
            raise GradCacheError(rc, "gc_dist_begin")

    def accumulate(self, D_block, i0, j0):
        bq, bn = D_block.shape
        rc = _lib.gc_dist_accumulate(_ptr(D_block), D_block.stride(0), i0, bq, j0, bn, _ptr(self.pos),
                                     self.B, self.N, self.tau, self.mask, _ptr(self.run_m),
                                     _ptr(self.run_l), _ptr(self.pos_d), _stream())
        if rc != 0:
            raise GradCacheError(rc, "gc_dist_accumulate")

    def finish(self):
        rc = _lib.gc_dist_finish(_ptr(self.run_m), _ptr(self.run_l), _ptr(self.pos_d), _ptr(self.pos),
                                 self.B, self.N, self.mask, _ptr(self.row_lse), _ptr(self.loss),
                                 _ptr(self.dev_status), _stream())
        if rc != 0:
            raise GradCacheError(rc, "gc_dist_finish")

    def w_block(self, D_block, i0, j0, W_block):
        bq, bn = D_block.shape
        rc = _lib.gc_dist_w_block(_ptr(D_block), D_block.stride(0), i0, bq, j0, bn, _ptr(self.pos),
                                  _ptr(self.row_lse), self.B, self.N, self.tau, self.mask,
                                  _ptr(W_block), W_block.stride(0), _stream())
        if rc != 0:
            raise GradCacheError(rc, "gc_dist_w_block")


def gc_dist_dot_block(Q, P, i0, bq, j0, bn, D_block) -> None:
    """D_block[r][c] = <Q[i0 + r], P[j0 + c]>: a block of dot-product distances (float32)."""
    B, d = Q.shape
    N = P.shape[0]
    rc = _lib.gc_dist_dot_block(_ptr(Q), Q.stride(0), _ptr(P), P.stride(0), B, N, d, _dtype_code(Q),
                                i0, bq, j0, bn, _ptr(D_block), D_block.stride(0), _stream())
    if rc != 0:
        raise GradCacheError(rc, "gc_dist_dot_block")


def gc_selftest_wait_limit(limit_ns: int, dev_status, waited_ns=None) -> None:
    """Runs the library's bounded on-chip wait with a limit of `limit_ns` on a barrier nothing
    arrives on: ORs GC_DEV_WAIT_LIMIT into dev_status[0] (int32) and writes the time waited to
    waited_ns[0] (int64 tensor, optional)."""
    rc = _lib.gc_selftest_wait_limit(int(limit_ns), _ptr(dev_status), _ptr(waited_ns), _stream())
    if rc != 0:
        raise GradCacheError(rc, "gc_selftest_wait_limit")


def gc_profile_enable(sets) -> None:
    """Per-kernel timing on (sets >= 1 event sets, True = 1) or off (0 / False)."""
    rc = _lib.gc_profile_enable(int(sets))
    if rc != 0:
        raise GradCacheError(rc, "gc_profile_enable")


def gc_profile_read(call: int | None = None) -> tuple[float, float, float]:
    """Milliseconds of the forward sweep, dQ sweep and dP sweep kernels of call number `call`
    since the enable (default: the most recent call)."""
    a, b, c = ctypes.c_float(), ctypes.c_float(), ctypes.c_float()
    if call is None:
        rc = _lib.gc_profile_read(ctypes.byref(a), ctypes.byref(b), ctypes.byref(c))
    else:
        rc = _lib.gc_profile_read_call(int(call), ctypes.byref(a), ctypes.byref(b), ctypes.byref(c))
    if rc != 0:
        raise GradCacheError(rc, "gc_profile_read")
    return a.value, b.value, c.value


def problem_tensors(prob, device="cuda"):
    """(Q, P, pos_idx) device tensors for an inputs.Problem, in its dtype.  Shared rows stay one
    buffer (Q is P)."""
    import numpy as np
    if prob.dtype == "bf16":
        Q = torch.from_numpy(prob.Q_bits.view(np.int16)).view(torch.bfloat16).to(device)
        P = Q if prob.shared else torch.from_numpy(prob.P_bits.view(np.int16)).view(
            torch.bfloat16).to(device)
    else:
        Q = torch.from_numpy(prob.Q).to(device)
        P = Q if prob.shared else torch.from_numpy(prob.P).to(device)
    return Q, P, torch.from_numpy(prob.pos_idx).to(device)


class Outputs:
    """Device buffers for one problem size, allocated once and reused across calls."""

    def __init__(self, B: int, N: int, d: int, dtype: int, device="cuda", op: int = GC_OP_BUILD):
        f = dict(dtype=torch.float32, device=device)
        self.loss = torch.zeros(1, **f)
        self.row_lse = torch.empty(B, **f)
        self.pos_logit = torch.empty(B, **f)
        self.dQ = torch.empty(B, d, **f)
        self.dP = torch.empty(N, d, **f)
        self.dev_status = torch.zeros(1, dtype=torch.int32, device=device)
        self.ws = alloc_workspace(op, B, N, d, dtype, device)


def build_cache(Q, P, pos_idx, tau=1.0, mask_mode=GC_MASK_NONE, out: Outputs | None = None):
    """Convenience wrapper: allocates outputs (or reuses `out`) and calls gc_build_cache."""
    B, d = Q.shape
    N = P.shape[0]
    if out is None:
        out = Outputs(B, N, d, _dtype_code(Q), Q.device)
    out.dev_status.zero_()
    gc_build_cache(Q, P, pos_idx, tau, mask_mode, out.loss, out.row_lse, out.dQ, out.dP,
                   out.pos_logit, out.ws, out.dev_status)
    return out
