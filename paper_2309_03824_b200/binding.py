"""Thin ctypes binding of liblrd_b200.so: same names as include/lrd.h, argument marshalling only.

Tensors are torch CUDA tensors (or None); the binding passes their device pointers and the
current CUDA stream.  There is no fallback: if the library is not built or cannot be loaded,
importing this module raises.
"""
from __future__ import annotations

import ctypes as C
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "liblrd_b200.so")
if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2309_03824_b200.build`")
_lib = C.CDLL(LIB_PATH)

# enums -------------------------------------------------------------------------------------------
(LRD_OK, LRD_ERR_INVALID_ARG, LRD_ERR_BAD_RANK, LRD_ERR_ALIGNMENT, LRD_ERR_WORKSPACE, LRD_ERR_UNSUPPORTED,
 LRD_ERR_ARCH, LRD_ERR_CUDA, LRD_ERR_TIMEOUT, LRD_ERR_TOO_LARGE) = range(10)
LRD_F32, LRD_BF16 = 0, 1
LRD_FREEZE_NONE, LRD_FREEZE_U, LRD_FREEZE_V = 0, 1, 2
LRD_TK_FREEZE_NONE, LRD_TK_FREEZE_FACTORS, LRD_TK_FREEZE_CORE = 0, 1, 2
LRD_ROUND_UP, LRD_ROUND_DOWN, LRD_ROUND_NEAREST = 0, 1, 2
LRD_PLAN_DZ, LRD_PLAN_DX, LRD_PLAN_DU, LRD_PLAN_DB, LRD_PLAN_DV, LRD_PLAN_NEEDS_Z, LRD_PLAN_NEEDS_X = 1, 2, 4, 8, 16, 32, 64
LRD_PATH_AUTO, LRD_PATH_GENERAL, LRD_PATH_UNFUSED, LRD_PATH_FUSED = 0, 1, 2, 3

EXPORTS = [
    "lrd_rank_quantize", "lrd_freeze_for_epoch", "lrd_tucker_freeze_for_epoch", "lrd_linear_bwd_plan",
    "lrd_status_string", "lrd_launch_count", "lrd_set_path", "lrd_check_device_status", "lrd_linear_workspace_bytes",
    "lrd_tucker2_workspace_bytes", "lrd_dense_workspace_bytes", "lrd_linear_fwd", "lrd_linear_bwd",
    "lrd_dense_fwd", "lrd_dense_bwd", "lrd_tucker2_fwd", "lrd_tucker2_bwd", "lrd_bias_grad_noalloc", "lrd_chain_tuning", "lrd_chain_pair_tuning", "lrd_selftest_wait_timeout", "lrd_gemm_tuning", "lrd_tucker2_overlap", "lrd_rank_search", "lrd_rank_multiple", "lrd_svd_rank", "lrd_tucker_rank", "lrd_tucker_rank_min", "lrd_conv3x3_workspace_bytes", "lrd_conv3x3_fwd", "lrd_conv3x3_bwd", "lrd_linear_group_fwd", "lrd_linear_group_bwd", "lrd_linear_bwd_accumulate", "lrd_linear_bwd_data", "lrd_linear_bwd_weights",
]


class lrd_linear_desc_t(C.Structure):
    _fields_ = [(n, C.c_int64) for n in ("M", "K", "N", "r", "ldx", "ldv", "ldu", "ldy", "ldz")] + [("dtype", C.c_int32)]


class lrd_tucker2_desc_t(C.Structure):
    _fields_ = [(n, C.c_int64) for n in ("B", "H", "W", "C", "S", "r1", "r2", "k", "stride", "pad")] + [("dtype", C.c_int32)]


_vp, _sz, _i64, _int = C.c_void_p, C.c_size_t, C.c_int64, C.c_int
_lib.lrd_rank_quantize.restype = _i64
_lib.lrd_rank_quantize.argtypes = [_i64, _i64, _int, _i64, _i64]
_lib.lrd_freeze_for_epoch.restype = _int
_lib.lrd_freeze_for_epoch.argtypes = [_i64]
_lib.lrd_tucker_freeze_for_epoch.restype = _int
_lib.lrd_tucker_freeze_for_epoch.argtypes = [_i64]
_lib.lrd_linear_bwd_plan.restype = C.c_uint32
_lib.lrd_linear_bwd_plan.argtypes = [_int]
_lib.lrd_status_string.restype = C.c_char_p
_lib.lrd_status_string.argtypes = [_int]
_lib.lrd_launch_count.restype = C.c_uint64
_lib.lrd_launch_count.argtypes = []
_lib.lrd_set_path.restype = _int
_lib.lrd_set_path.argtypes = [_int]
_lib.lrd_rank_search.restype = _i64
_lib.lrd_rank_search.argtypes = [C.POINTER(C.c_double), _i64, _i64, C.c_double, C.c_double, C.POINTER(C.c_int)]
_lib.lrd_rank_multiple.restype = _i64
_lib.lrd_rank_multiple.argtypes = [C.POINTER(C.c_double), _i64, _i64, C.c_double]
_lib.lrd_svd_rank.restype = _i64
_lib.lrd_svd_rank.argtypes = [_i64, _i64, C.c_double]
_lib.lrd_tucker_rank.restype = _i64
_lib.lrd_tucker_rank.argtypes = [_i64, _i64, _i64, C.c_double, C.c_double, C.POINTER(C.c_int64)]
_lib.lrd_tucker_rank_min.restype = _i64
_lib.lrd_tucker_rank_min.argtypes = [_i64, _i64, _i64, C.c_double, C.c_double]
_lib.lrd_conv3x3_workspace_bytes.restype = C.c_size_t
_lib.lrd_conv3x3_workspace_bytes.argtypes = [_i64, _i64, _i64, _i64, _i64, _int]
_lib.lrd_conv3x3_fwd.restype = _int
_lib.lrd_conv3x3_fwd.argtypes = [_i64, _i64, _i64, _i64, _i64, _int] + [C.c_void_p] * 4
_lib.lrd_conv3x3_bwd.restype = _int
_lib.lrd_conv3x3_bwd.argtypes = [_i64, _i64, _i64, _i64, _i64, _int] + [C.c_void_p] * 6 + [C.c_size_t, C.c_void_p]
_lib.lrd_chain_tuning.restype = _int
_lib.lrd_chain_tuning.argtypes = [_int, _int, _int]
_lib.lrd_selftest_wait_timeout.restype = _int
_lib.lrd_selftest_wait_timeout.argtypes = [C.c_void_p]
_lib.lrd_chain_pair_tuning.restype = _int
_lib.lrd_chain_pair_tuning.argtypes = [_int, _int, _int, _int]
_pp = C.POINTER(C.c_void_p)
_lib.lrd_linear_group_fwd.restype = _int
_lib.lrd_linear_group_fwd.argtypes = [_int, C.POINTER(lrd_linear_desc_t), _pp, _pp, _pp, _pp, _pp, _pp, _int, _pp,
                                      C.POINTER(C.c_size_t), C.c_void_p]
_lib.lrd_linear_group_bwd.restype = _int
_lib.lrd_linear_group_bwd.argtypes = [_int, C.POINTER(lrd_linear_desc_t)] + [_pp] * 9 + [_int, _pp, C.POINTER(C.c_size_t), C.c_void_p]
_lib.lrd_gemm_tuning.restype = _int
_lib.lrd_gemm_tuning.argtypes = [_int]
_lib.lrd_tucker2_overlap.restype = _int
_lib.lrd_tucker2_overlap.argtypes = [_int]
_lib.lrd_check_device_status.restype = _int
_lib.lrd_check_device_status.argtypes = []
_lib.lrd_linear_workspace_bytes.restype = _sz
_lib.lrd_linear_workspace_bytes.argtypes = [C.POINTER(lrd_linear_desc_t), _int, _int]
_lib.lrd_dense_workspace_bytes.restype = _sz
_lib.lrd_dense_workspace_bytes.argtypes = [C.POINTER(lrd_linear_desc_t), _int]
_lib.lrd_tucker2_workspace_bytes.restype = _sz
_lib.lrd_tucker2_workspace_bytes.argtypes = [C.POINTER(lrd_tucker2_desc_t), _int, _int]
_lib.lrd_linear_fwd.restype = _int
_lib.lrd_linear_fwd.argtypes = [C.POINTER(lrd_linear_desc_t)] + [_vp] * 6 + [_int, _vp, _sz, _vp]
_lib.lrd_linear_bwd.restype = _int
_lib.lrd_linear_bwd.argtypes = [C.POINTER(lrd_linear_desc_t)] + [_vp] * 9 + [_int, _vp, _sz, _vp]
_lib.lrd_linear_bwd_data.restype = _int
_lib.lrd_linear_bwd_data.argtypes = [C.POINTER(lrd_linear_desc_t)] + [_vp] * 4 + [_int, _vp, _sz, _vp]
_lib.lrd_linear_bwd_weights.restype = _int
_lib.lrd_linear_bwd_weights.argtypes = [C.POINTER(lrd_linear_desc_t)] + [_vp] * 6 + [_int, _vp, _sz, _vp]
_lib.lrd_linear_bwd_accumulate.restype = _int
_lib.lrd_linear_bwd_accumulate.argtypes = [C.POINTER(lrd_linear_desc_t)] + [_vp] * 9 + [_int, _vp, _sz, _vp]
_lib.lrd_dense_fwd.restype = _int
_lib.lrd_dense_fwd.argtypes = [C.POINTER(lrd_linear_desc_t)] + [_vp] * 4 + [_vp, _sz, _vp]
_lib.lrd_dense_bwd.restype = _int
_lib.lrd_dense_bwd.argtypes = [C.POINTER(lrd_linear_desc_t)] + [_vp] * 6 + [_vp, _sz, _vp]
_lib.lrd_bias_grad_noalloc.restype = _int
_lib.lrd_bias_grad_noalloc.argtypes = [_vp, _i64, _i64, _i64, _vp, _int, _vp]
_lib.lrd_tucker2_fwd.restype = _int
_lib.lrd_tucker2_fwd.argtypes = [C.POINTER(lrd_tucker2_desc_t)] + [_vp] * 8 + [_int, _vp, _sz, _vp]
_lib.lrd_tucker2_bwd.restype = _int
_lib.lrd_tucker2_bwd.argtypes = [C.POINTER(lrd_tucker2_desc_t)] + [_vp] * 12 + [_int, _vp, _sz, _vp]


class LrdError(RuntimeError):
    def __init__(self, status):
        self.status = int(status)
        super().__init__(f"lrd status {self.status}: {lrd_status_string(self.status)}")


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream):
    if stream is not None:
        return C.c_void_p(int(stream))
    import torch
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _ws(workspace):
    if workspace is None:
        return None, 0
    return C.c_void_p(workspace.data_ptr()), workspace.numel() * workspace.element_size()


def _check(status):
    if status != LRD_OK:
        raise LrdError(status)


def linear_desc(M, K, N, r, dtype, ldx=0, ldv=0, ldu=0, ldy=0, ldz=0):
    return lrd_linear_desc_t(M, K, N, r, ldx, ldv, ldu, ldy, ldz, dtype)


def tucker2_desc(B, H, W, Cin, S, r1, r2, dtype, k=3, stride=1, pad=1):
    return lrd_tucker2_desc_t(B, H, W, Cin, S, r1, r2, k, stride, pad, dtype)


# host-only helpers ---------------------------------------------------------------------------------
def lrd_rank_quantize(r, multiple, mode, K, N):
    return int(_lib.lrd_rank_quantize(r, multiple, mode, K, N))


def lrd_freeze_for_epoch(e):
    return int(_lib.lrd_freeze_for_epoch(e))


def lrd_tucker_freeze_for_epoch(e):
    return int(_lib.lrd_tucker_freeze_for_epoch(e))


def lrd_rank_search(t, R_min, T_orig, min_rel_drop=0.0):
    """Algorithm 1 on a measured curve: t[i] = step time at rank R_min + i.  Returns (R_opt, use_decomposed)."""
    arr = (C.c_double * len(t))(*[float(x) for x in t])
    use = C.c_int(0)
    r = int(_lib.lrd_rank_search(arr, len(t), int(R_min), float(T_orig), float(min_rel_drop), C.byref(use)))
    if r < 0:
        raise LrdError(-r)
    return r, bool(use.value)


def lrd_rank_multiple(t, R_min, min_rel_drop):
    arr = (C.c_double * len(t))(*[float(x) for x in t])
    r = int(_lib.lrd_rank_multiple(arr, len(t), int(R_min), float(min_rel_drop)))
    if r < 0:
        raise LrdError(-r)
    return r


def lrd_svd_rank(Cin, S, alpha):
    return int(_lib.lrd_svd_rank(int(Cin), int(S), float(alpha)))


def lrd_tucker_rank(Cin, S, k, alpha, beta=1.0):
    r2 = C.c_int64(0)
    r1 = int(_lib.lrd_tucker_rank(int(Cin), int(S), int(k), float(alpha), float(beta), C.byref(r2)))
    return r1, int(r2.value)


def lrd_tucker_rank_min(Cin, S, k, alpha, beta=1.0):
    return int(_lib.lrd_tucker_rank_min(int(Cin), int(S), int(k), float(alpha), float(beta)))


def lrd_conv3x3_workspace_bytes(B, H, W, Cin, S, dtype):
    return int(_lib.lrd_conv3x3_workspace_bytes(B, H, W, Cin, S, dtype))


def lrd_conv3x3_fwd(B, H, W, Cin, S, dtype, X, Wk, Y, stream=None, check=True):
    st = _lib.lrd_conv3x3_fwd(B, H, W, Cin, S, dtype, _ptr(X), _ptr(Wk), _ptr(Y), _stream(stream))
    if check:
        _check(st)
    return st


def lrd_conv3x3_bwd(B, H, W, Cin, S, dtype, dY, X, Wk, dX, dW, workspace, stream=None, check=True):
    w, n = _ws(workspace)
    st = _lib.lrd_conv3x3_bwd(B, H, W, Cin, S, dtype, _ptr(dY), _ptr(X), _ptr(Wk), _ptr(dX), _ptr(dW), w, n, _stream(stream))
    if check:
        _check(st)
    return st


def lrd_linear_bwd_plan(freeze):
    return int(_lib.lrd_linear_bwd_plan(freeze))


def lrd_status_string(status):
    return _lib.lrd_status_string(int(status)).decode()


def lrd_launch_count():
    return int(_lib.lrd_launch_count())


def lrd_selftest_wait_timeout(stream=None):
    _check(_lib.lrd_selftest_wait_timeout(_stream(stream)))


def lrd_set_path(path):
    _check(_lib.lrd_set_path(path))


def lrd_chain_tuning(cluster_blocks=0, kblocks_per_stage=0, chunk_columns=0):
    _check(_lib.lrd_chain_tuning(cluster_blocks, kblocks_per_stage, chunk_columns))


def lrd_chain_pair_tuning(blocks_per_mma=0, pairs_per_cluster=0, kblocks_per_stage=0, chunk_columns=0):
    _check(_lib.lrd_chain_pair_tuning(blocks_per_mma, pairs_per_cluster, kblocks_per_stage, chunk_columns))


def lrd_gemm_tuning(blocks_per_mma=0):
    _check(_lib.lrd_gemm_tuning(blocks_per_mma))


def lrd_tucker2_overlap(on=True):
    _check(_lib.lrd_tucker2_overlap(int(bool(on))))


def lrd_check_device_status():
    return int(_lib.lrd_check_device_status())


def lrd_linear_workspace_bytes(desc, freeze, is_bwd):
    return int(_lib.lrd_linear_workspace_bytes(C.byref(desc), freeze, int(is_bwd)))


def lrd_dense_workspace_bytes(desc, is_bwd):
    return int(_lib.lrd_dense_workspace_bytes(C.byref(desc), int(is_bwd)))


def lrd_tucker2_workspace_bytes(desc, freeze, is_bwd):
    return int(_lib.lrd_tucker2_workspace_bytes(C.byref(desc), freeze, int(is_bwd)))


# device entry points ---------------------------------------------------------------------------------
def lrd_linear_fwd(desc, X, V, U, bias, Y, Z_save, freeze, workspace, stream=None, check=True):
    w, n = _ws(workspace)
    st = _lib.lrd_linear_fwd(C.byref(desc), _ptr(X), _ptr(V), _ptr(U), _ptr(bias), _ptr(Y), _ptr(Z_save), freeze, w, n,
                             _stream(stream))
    if check:
        _check(st)
    return st


def lrd_linear_bwd(desc, dY, X, V, U, Z_save, dX, dU, dV, dbias, freeze, workspace, stream=None, check=True):
    w, n = _ws(workspace)
    st = _lib.lrd_linear_bwd(C.byref(desc), _ptr(dY), _ptr(X), _ptr(V), _ptr(U), _ptr(Z_save), _ptr(dX), _ptr(dU),
                             _ptr(dV), _ptr(dbias), freeze, w, n, _stream(stream))
    if check:
        _check(st)
    return st


def lrd_linear_bwd_data(desc, dY, V, U, dX, freeze, workspace, stream=None, check=True):
    w, n = _ws(workspace)
    st = _lib.lrd_linear_bwd_data(C.byref(desc), _ptr(dY), _ptr(V), _ptr(U), _ptr(dX), freeze, w, n, _stream(stream))
    if check:
        _check(st)
    return st


def lrd_linear_bwd_weights(desc, dY, X, Z_save, dU, dV, dbias, freeze, workspace, stream=None, check=True):
    w, n = _ws(workspace)
    st = _lib.lrd_linear_bwd_weights(C.byref(desc), _ptr(dY), _ptr(X), _ptr(Z_save), _ptr(dU), _ptr(dV), _ptr(dbias), freeze, w, n,
                                     _stream(stream))
    if check:
        _check(st)
    return st


def _ptr_array(ts, n):
    """Host array of n device pointers (NULL entries for None); None for a list that is None as a whole."""
    if ts is None:
        return None
    if len(ts) != n:
        raise ValueError("every per-layer list of a group has one entry per layer")
    return (C.c_void_p * n)(*[None if t is None else t.data_ptr() for t in ts])


def _group_common(descs, workspaces):
    n = len(descs)
    darr = (lrd_linear_desc_t * n)(*descs)
    ws = [_ws(w) for w in workspaces]
    warr = (C.c_void_p * n)(*[w[0] for w in ws])
    wbytes = (C.c_size_t * n)(*[w[1] for w in ws])
    return n, darr, warr, wbytes


def lrd_linear_group_fwd(descs, X, V, U, bias, Y, Z_save, freeze, workspaces, stream=None, check=True):
    """n independent layers side by side: every argument but freeze/stream is a list with one entry per layer."""
    n, darr, warr, wbytes = _group_common(descs, workspaces)
    st = _lib.lrd_linear_group_fwd(n, darr, _ptr_array(X, n), _ptr_array(V, n), _ptr_array(U, n), _ptr_array(bias, n),
                                   _ptr_array(Y, n), _ptr_array(Z_save, n), freeze, warr, wbytes, _stream(stream))
    if check:
        _check(st)
    return st


def lrd_linear_group_bwd(descs, dY, X, V, U, Z_save, dX, dU, dV, dbias, freeze, workspaces, stream=None, check=True):
    n, darr, warr, wbytes = _group_common(descs, workspaces)
    st = _lib.lrd_linear_group_bwd(n, darr, _ptr_array(dY, n), _ptr_array(X, n), _ptr_array(V, n), _ptr_array(U, n),
                                   _ptr_array(Z_save, n), _ptr_array(dX, n), _ptr_array(dU, n), _ptr_array(dV, n),
                                   _ptr_array(dbias, n), freeze, warr, wbytes, _stream(stream))
    if check:
        _check(st)
    return st


def lrd_linear_bwd_accumulate(desc, dY, X, V, U, Z_save, dX, dU, dV, dbias, freeze, workspace, stream=None, check=True):
    w, n = _ws(workspace)
    st = _lib.lrd_linear_bwd_accumulate(C.byref(desc), _ptr(dY), _ptr(X), _ptr(V), _ptr(U), _ptr(Z_save), _ptr(dX), _ptr(dU),
                                        _ptr(dV), _ptr(dbias), freeze, w, n, _stream(stream))
    if check:
        _check(st)
    return st


def lrd_dense_fwd(desc, X, W, bias, Y, workspace, stream=None, check=True):
    w, n = _ws(workspace)
    st = _lib.lrd_dense_fwd(C.byref(desc), _ptr(X), _ptr(W), _ptr(bias), _ptr(Y), w, n, _stream(stream))
    if check:
        _check(st)
    return st


def lrd_dense_bwd(desc, dY, X, W, dX, dW, dbias, workspace, stream=None, check=True):
    w, n = _ws(workspace)
    st = _lib.lrd_dense_bwd(C.byref(desc), _ptr(dY), _ptr(X), _ptr(W), _ptr(dX), _ptr(dW), _ptr(dbias), w, n,
                            _stream(stream))
    if check:
        _check(st)
    return st


def lrd_tucker2_fwd(desc, X, A, G, Bm, bias, Y, Z1_save, Z2_save, freeze, workspace, stream=None, check=True):
    w, n = _ws(workspace)
    st = _lib.lrd_tucker2_fwd(C.byref(desc), _ptr(X), _ptr(A), _ptr(G), _ptr(Bm), _ptr(bias), _ptr(Y), _ptr(Z1_save),
                              _ptr(Z2_save), freeze, w, n, _stream(stream))
    if check:
        _check(st)
    return st


def lrd_tucker2_bwd(desc, dY, X, A, G, Bm, Z1_save, Z2_save, dX, dA, dG, dB, dbias, freeze, workspace, stream=None,
                    check=True):
    w, n = _ws(workspace)
    st = _lib.lrd_tucker2_bwd(C.byref(desc), _ptr(dY), _ptr(X), _ptr(A), _ptr(G), _ptr(Bm), _ptr(Z1_save),
                              _ptr(Z2_save), _ptr(dX), _ptr(dA), _ptr(dG), _ptr(dB), _ptr(dbias), freeze, w, n,
                              _stream(stream))
    if check:
        _check(st)
    return st


def lrd_bias_grad_noalloc(dY, ldy, M, N, dbias, dtype, stream=None, check=True):
    """Column sums of dY into dbias with the library's built-in scratch (no workspace, no allocation)."""
    st = _lib.lrd_bias_grad_noalloc(_ptr(dY), ldy, M, N, _ptr(dbias), dtype, _stream(stream))
    if check:
        _check(st)
    return st
