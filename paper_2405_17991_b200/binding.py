"""ctypes binding of libvelora.so: argument marshalling only.

Each function has the name and meaning of the C entry point it wraps
(``include/velora.h``); tensors are torch CUDA tensors whose device memory,
row pitch and current stream are handed to the library as plain pointers and
integers.  Every step of the path runs inside the library's kernels; there is
no fallback: a missing library or a non-zero status raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libvelora.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_ALIGNMENT, ERR_WORKSPACE, ERR_DEGENERATE_V, ERR_TIMEOUT, ERR_CUDA = range(8)
F32, BF16, FP8_E4M3 = 0, 1, 2
WG_FACTORED, WG_EXPLICIT = 0, 1
PRODUCT_A_BT, PRODUCT_A_B, PRODUCT_AT_B = 0, 1, 2
(OP_INIT_V, OP_WEIGHT_GRAD_FACTORED, OP_WEIGHT_GRAD_EXPLICIT, OP_LINEAR_FORWARD,
 OP_LINEAR_BACKWARD_FACTORED, OP_LINEAR_BACKWARD_EXPLICIT, OP_UPDATE_V, OP_Z8_CALIBRATE) = range(8)

_p, _i64, _int, _sz = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_size_t

SIGNATURES = {
    "velora_version": (_int, []),
    "velora_status_string": (ctypes.c_char_p, [_int]),
    "velora_workspace_bytes": (_sz, [_int, _i64, _i64, _i64, _int]),
    "velora_launch_count": (ctypes.c_ulonglong, []),
    "velora_host_step_staging_bytes": (_sz, [_i64, _i64, _i64, _int]),
    "velora_linear_step_host": (_int, [_p, _p, _p, _p, _p, _p, _p, _p, _sz, _i64, _i64, _i64, _int, _p, _sz, _p]),
    "velora_workspace_init": (_int, [_p, _sz, _p]),
    "velora_workspace_status": (_int, [_p, _p]),
    "velora_device_error": (_int, [_p]),
    "velora_selftest_wait_timeout": (_int, [_p, _sz, ctypes.c_ulonglong, _p, _p]),
    "velora_init_v": (_int, [_p, _int, _i64, _i64, _i64, _int, _p, _p, _sz, _p]),
    "velora_init_v_static": (_int, [_p, _int, _i64, _i64, _i64, _int, _p, _p]),
    "velora_subtoken_sum": (_int, [_p, _int, _i64, _i64, _i64, _int, _p, _p, _sz, _p]),
    "velora_normalize_v": (_int, [_p, _int, _p, _p, _sz, _p]),
    "velora_update_v": (_int, [_p, _int, _i64, _i64, _i64, _int, ctypes.c_float, _p, _p, _p, _sz, _p]),
    "velora_weight_grad_p": (_int, [_p, _int, _i64, _i64, _i64, _p, _int, _i64, _i64, _int, _p, _i64, _int, _p, _sz, _p]),
    "velora_expand_p": (_int, [_p, _i64, _p, _i64, _i64, _int, _p, _int, _i64, _int, _p]),
    "velora_z8_calibrate": (_int, [_p, _int, _i64, _i64, _i64, _int, _p, ctypes.c_float, _p, _p, _p, _p, _sz, _p]),
    "velora_dense_product": (_int, [_int, _p, _i64, _p, _i64, _p, _int, _i64, _int, _i64, _i64, _i64, _int, _p, _sz, _p]),
    "velora_compress": (_int, [_p, _int, _i64, _i64, _i64, _int, _p, _p, _int, _i64, _p]),
    "velora_reconstruct": (_int, [_p, _int, _i64, _i64, _i64, _int, _p, _p, _int, _i64, _p]),
    "velora_weight_grad": (_int, [_p, _int, _i64, _i64, _i64, _p, _int, _i64, _p, _i64, _int,
                                  _p, _int, _i64, _int, _int, _p, _sz, _p]),
    "velora_linear_forward": (_int, [_p, _i64, _p, _i64, _p, _p, _i64, _p, _int, _i64,
                                     _int, _i64, _i64, _i64, _int, _p, _sz, _p]),
    "velora_linear_backward": (_int, [_p, _i64, _p, _i64, _p, _int, _i64, _p, _p, _i64, _p, _int, _i64, _int, _int,
                                      _int, _i64, _i64, _i64, _int, _p, _sz, _p]),
}


class VeloraError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib().velora_status_string(status).decode()
        super().__init__("%s: status %d (%s)" % (where, status, msg))


_lib = None


def lib() -> ctypes.CDLL:
    """The loaded C-ABI library.  Raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                "libvelora.so is missing at %s: build it with `python -m paper_2405_17991_b200.build` "
                "(nvcc, sm_100a). There is no CPU or PyTorch fallback." % LIB_PATH)
        handle = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(handle, name)
            fn.restype = res
            fn.argtypes = args
        _lib = handle
    return _lib


Z8_TORCH = getattr(torch, "float8_e4m3fn", None)      # torch's name for the E4M3 byte; torch.uint8 is accepted as well


def _dt(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    if t.dtype == torch.uint8 or (Z8_TORCH is not None and t.dtype == Z8_TORCH):
        return FP8_E4M3                                 # only Z may have this type; the library checks
    raise TypeError("unsupported dtype %s (float32, bfloat16, or uint8 / float8_e4m3fn for Z)" % t.dtype)


def _mat(t: torch.Tensor, name: str):
    if t.ndim != 2 or not t.is_cuda:
        raise ValueError("%s must be a 2-d CUDA tensor" % name)
    if t.shape[1] > 1 and t.stride(1) != 1:
        raise ValueError("%s must have contiguous rows" % name)
    ld = t.stride(0) if t.shape[0] > 1 else max(t.stride(0), t.shape[1])
    return ctypes.c_void_p(t.data_ptr()), int(ld)


def _vec(v: torch.Tensor):
    if v.ndim != 1 or v.dtype != torch.float32 or not v.is_cuda or not v.is_contiguous():
        raise ValueError("v must be a contiguous 1-d float32 CUDA tensor")
    return ctypes.c_void_p(v.data_ptr())


def _stream(stream) -> ctypes.c_void_p:
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _ws(ws: Optional[torch.Tensor], need: int, device) -> torch.Tensor:
    if ws is None:
        ws = velora_workspace_alloc(need, device)
    return ws


def velora_workspace_alloc(nbytes: int, device) -> torch.Tensor:
    """Device workspace of at least ``nbytes`` with its status header zeroed."""
    ws = torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)
    velora_workspace_init(ws)
    return ws


def velora_workspace_init(ws: torch.Tensor, stream=None) -> None:
    _check(lib().velora_workspace_init(ctypes.c_void_p(ws.data_ptr()), ws.numel(), _stream(stream)),
           "velora_workspace_init")


def velora_workspace_status(ws: torch.Tensor, stream=None) -> int:
    """Synchronises the stream; 0, ERR_TIMEOUT if a kernel's bounded wait expired, or ERR_DEGENERATE_V
    left by velora_update_v."""
    return int(lib().velora_workspace_status(ctypes.c_void_p(ws.data_ptr()), _stream(stream)))


def velora_device_error(stream=None) -> int:
    """Synchronises the stream; 0, or ERR_TIMEOUT if a streaming kernel's bounded wait expired (then cleared)."""
    return int(lib().velora_device_error(_stream(stream)))


def velora_selftest_wait_timeout(ws: torch.Tensor, limit_ns: int, observed: torch.Tensor, stream=None) -> None:
    """Runs the one-CTA kernel whose bounded waits expire; ``observed`` is a 4-element int32 CUDA tensor."""
    if observed.dtype != torch.int32 or observed.numel() < 4 or not observed.is_cuda or not observed.is_contiguous():
        raise ValueError("observed must be a contiguous int32 CUDA tensor with 4 elements")
    _check(lib().velora_selftest_wait_timeout(ctypes.c_void_p(ws.data_ptr()), ws.numel(), int(limit_ns),
                                              ctypes.c_void_p(observed.data_ptr()), _stream(stream)),
           "velora_selftest_wait_timeout")


def _check(status: int, where: str):
    if status != OK:
        raise VeloraError(status, where)


def num_subtokens(D: int, Dsub: int) -> int:
    return -(-D // Dsub)


def velora_version() -> int:
    return lib().velora_version()


def velora_status_string(status: int) -> str:
    return lib().velora_status_string(status).decode()


def velora_workspace_bytes(op: int, N: int, D: int, O: int, Dsub: int) -> int:
    return int(lib().velora_workspace_bytes(op, N, D, O, Dsub))


def velora_init_v(X: torch.Tensor, Dsub: int, v: Optional[torch.Tensor] = None,
                  ws: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    xp, ldx = _mat(X, "X")
    N, D = X.shape
    if v is None:
        v = torch.empty(Dsub, dtype=torch.float32, device=X.device)
    ws = _ws(ws, velora_workspace_bytes(OP_INIT_V, N, D, 1, Dsub), X.device)
    rc = lib().velora_init_v(xp, _dt(X), N, D, ldx, Dsub, _vec(v), ctypes.c_void_p(ws.data_ptr()), ws.numel(),
                             _stream(stream))
    _check(rc, "velora_init_v")
    return v


def velora_init_v_static(X: torch.Tensor, Dsub: int, v: torch.Tensor, stream=None) -> torch.Tensor:
    """velora_init_v through the library's built-in scratch: no workspace, nothing allocated by the call.

    ``v`` must be supplied by the caller (this wrapper allocates nothing either).  Dsub is limited to
    256; calls on one device must not overlap on the GPU, since they share the scratch array.
    """
    xp, ldx = _mat(X, "X")
    N, D = X.shape
    rc = lib().velora_init_v_static(xp, _dt(X), N, D, ldx, Dsub, _vec(v), _stream(stream))
    _check(rc, "velora_init_v_static")
    return v


def velora_compress(X: torch.Tensor, v: torch.Tensor, Z: Optional[torch.Tensor] = None,
                    z_dtype=torch.float32, stream=None) -> torch.Tensor:
    xp, ldx = _mat(X, "X")
    N, D = X.shape
    Dsub = v.shape[0]
    if Z is None:
        Z = torch.empty((N, num_subtokens(D, Dsub)), dtype=z_dtype, device=X.device)
    zp, ldz = _mat(Z, "Z")
    rc = lib().velora_compress(xp, _dt(X), N, D, ldx, Dsub, _vec(v), zp, _dt(Z), ldz, _stream(stream))
    _check(rc, "velora_compress")
    return Z


def velora_reconstruct(Z: torch.Tensor, v: torch.Tensor, D: int, Xhat: Optional[torch.Tensor] = None,
                       x_dtype=torch.bfloat16, stream=None) -> torch.Tensor:
    zp, ldz = _mat(Z, "Z")
    N = Z.shape[0]
    Dsub = v.shape[0]
    if Xhat is None:
        Xhat = torch.empty((N, D), dtype=x_dtype, device=Z.device)
    xp, ldx = _mat(Xhat, "Xhat")
    rc = lib().velora_reconstruct(zp, _dt(Z), ldz, N, D, Dsub, _vec(v), xp, _dt(Xhat), ldx, _stream(stream))
    _check(rc, "velora_reconstruct")
    return Xhat


def velora_weight_grad(dY: torch.Tensor, Z: torch.Tensor, v: torch.Tensor, D: int,
                       dW: Optional[torch.Tensor] = None, dw_dtype=None, beta: int = 0, mode: int = WG_FACTORED,
                       ws: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    yp, lddy = _mat(dY, "dY")
    zp, ldz = _mat(Z, "Z")
    N, O = dY.shape
    Dsub = v.shape[0]
    if dW is None:
        dW = torch.empty((O, D), dtype=dw_dtype or dY.dtype, device=dY.device)
    wp, lddw = _mat(dW, "dW")
    op = OP_WEIGHT_GRAD_FACTORED if mode == WG_FACTORED else OP_WEIGHT_GRAD_EXPLICIT
    ws = _ws(ws, velora_workspace_bytes(op, N, D, O, Dsub), dY.device)
    rc = lib().velora_weight_grad(yp, _dt(dY), N, O, lddy, zp, _dt(Z), ldz, _vec(v), D, Dsub,
                                  wp, _dt(dW), lddw, beta, mode, ctypes.c_void_p(ws.data_ptr()), ws.numel(),
                                  _stream(stream))
    _check(rc, "velora_weight_grad")
    return dW


def velora_linear_forward(X: torch.Tensor, W: torch.Tensor, v: torch.Tensor,
                          Y: Optional[torch.Tensor] = None, Z: Optional[torch.Tensor] = None,
                          z_dtype=torch.float32, ws: Optional[torch.Tensor] = None, stream=None):
    xp, ldx = _mat(X, "X")
    wp, ldw = _mat(W, "W")
    N, D = X.shape
    O = W.shape[0]
    Dsub = v.shape[0]
    if W.shape[1] != D or W.dtype != X.dtype:
        raise ValueError("W must be [O, D] with X's dtype")
    if Y is None:
        Y = torch.empty((N, O), dtype=X.dtype, device=X.device)
    if Z is None:
        Z = torch.empty((N, num_subtokens(D, Dsub)), dtype=z_dtype, device=X.device)
    yp, ldy = _mat(Y, "Y")
    zp, ldz = _mat(Z, "Z")
    ws = _ws(ws, velora_workspace_bytes(OP_LINEAR_FORWARD, N, D, O, Dsub), X.device)
    rc = lib().velora_linear_forward(xp, ldx, wp, ldw, _vec(v), yp, ldy, zp, _dt(Z), ldz,
                                     _dt(X), N, D, O, Dsub, ctypes.c_void_p(ws.data_ptr()), ws.numel(),
                                     _stream(stream))
    _check(rc, "velora_linear_forward")
    return Y, Z


def velora_linear_backward(dY: torch.Tensor, W: torch.Tensor, Z: torch.Tensor, v: torch.Tensor,
                           dX: Optional[torch.Tensor] = None, dW: Optional[torch.Tensor] = None,
                           need_dX: bool = True, need_dW: bool = True, dw_dtype=None, beta: int = 0,
                           mode: int = WG_FACTORED, ws: Optional[torch.Tensor] = None, stream=None):
    yp, lddy = _mat(dY, "dY")
    wp, ldw = _mat(W, "W")
    zp, ldz = _mat(Z, "Z")
    N, O = dY.shape
    D = W.shape[1]
    Dsub = v.shape[0]
    if need_dX and dX is None:
        dX = torch.empty((N, D), dtype=dY.dtype, device=dY.device)
    if need_dW and dW is None:
        dW = torch.empty((O, D), dtype=dw_dtype or dY.dtype, device=dY.device)
    xp, lddx = _mat(dX, "dX") if need_dX else (ctypes.c_void_p(0), D)
    gp, lddw = _mat(dW, "dW") if need_dW else (ctypes.c_void_p(0), D)
    op = OP_LINEAR_BACKWARD_FACTORED if mode == WG_FACTORED else OP_LINEAR_BACKWARD_EXPLICIT
    ws = _ws(ws, velora_workspace_bytes(op, N, D, O, Dsub), dY.device)
    rc = lib().velora_linear_backward(yp, lddy, wp, ldw, zp, _dt(Z), ldz, _vec(v), xp, lddx,
                                      gp, _dt(dW) if need_dW else _dt(dY), lddw, beta, mode,
                                      _dt(dY), N, D, O, Dsub, ctypes.c_void_p(ws.data_ptr()), ws.numel(),
                                      _stream(stream))
    _check(rc, "velora_linear_backward")
    return dX, dW


def velora_dense_product(kind: int, A: torch.Tensor, B: torch.Tensor, C: Optional[torch.Tensor] = None,
                         c_dtype=None, beta: int = 0, ws: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """C = beta * C + op(A) op(B): the plain products of the layer (PRODUCT_A_BT, PRODUCT_A_B, PRODUCT_AT_B)."""
    ap, lda = _mat(A, "A")
    bp, ldb = _mat(B, "B")
    Mdim, Kdim = (A.shape[1], A.shape[0]) if kind == PRODUCT_AT_B else (A.shape[0], A.shape[1])
    Ndim = B.shape[0] if kind == PRODUCT_A_BT else B.shape[1]
    if (B.shape[1] if kind == PRODUCT_A_BT else B.shape[0]) != Kdim or A.dtype != B.dtype:
        raise ValueError("operand shapes or dtypes do not match")
    if C is None:
        C = torch.empty((Mdim, Ndim), dtype=c_dtype or A.dtype, device=A.device)
    cp, ldc = _mat(C, "C")
    ws = _ws(ws, 256, A.device)
    rc = lib().velora_dense_product(kind, ap, lda, bp, ldb, cp, _dt(C), ldc, beta, Mdim, Ndim, Kdim, _dt(A),
                                    ctypes.c_void_p(ws.data_ptr()), ws.numel(), _stream(stream))
    _check(rc, "velora_dense_product")
    return C


def velora_z8_calibrate(X: torch.Tensor, v: torch.Tensor, headroom: float = 2.0, ws: Optional[torch.Tensor] = None,
                        stream=None):
    """Scale of the 8-bit Z store from a batch: returns (zscale[1], v_store = v / zscale, v_load = v * zscale)."""
    xp, ldx = _mat(X, "X")
    N, D = X.shape
    Dsub = v.shape[0]
    zscale = torch.empty(1, dtype=torch.float32, device=X.device)
    v_store, v_load = torch.empty_like(v), torch.empty_like(v)
    ws = _ws(ws, velora_workspace_bytes(OP_Z8_CALIBRATE, N, D, 0, Dsub), X.device)
    rc = lib().velora_z8_calibrate(xp, _dt(X), N, D, ldx, Dsub, _vec(v), float(headroom), _vec(zscale), _vec(v_store),
                                   _vec(v_load), ctypes.c_void_p(ws.data_ptr()), ws.numel(), _stream(stream))
    _check(rc, "velora_z8_calibrate")
    return zscale, v_store, v_load


def velora_launch_count() -> int:
    return int(lib().velora_launch_count())


def velora_host_step_staging_bytes(N: int, D: int, O: int, Dsub: int) -> int:
    return int(lib().velora_host_step_staging_bytes(N, D, O, Dsub))


def _host_ptr(t: Optional[torch.Tensor], shape, name: str) -> ctypes.c_void_p:
    if t is None:
        return ctypes.c_void_p(0)
    if t.is_cuda or t.dtype != torch.bfloat16 or tuple(t.shape) != tuple(shape) or not t.is_contiguous():
        raise ValueError("%s must be a contiguous CPU bfloat16 tensor of shape %r" % (name, tuple(shape)))
    return ctypes.c_void_p(t.data_ptr())


def velora_linear_step_host(hX: torch.Tensor, hdY: torch.Tensor, W: torch.Tensor, v: torch.Tensor,
                            staging: torch.Tensor, ws: torch.Tensor, hY: Optional[torch.Tensor] = None,
                            hdX: Optional[torch.Tensor] = None, hdW: Optional[torch.Tensor] = None,
                            stream=None) -> None:
    """Forward + backward on host-resident (pinned) X and dY; results copied back to the given host tensors."""
    N, D = hX.shape
    O = W.shape[0]
    Dsub = v.shape[0]
    wp, ldw = _mat(W, "W")
    if ldw != D:
        raise ValueError("W must be dense")
    rc = lib().velora_linear_step_host(
        _host_ptr(hX, (N, D), "hX"), _host_ptr(hdY, (N, O), "hdY"), _host_ptr(hY, (N, O), "hY"),
        _host_ptr(hdX, (N, D), "hdX"), _host_ptr(hdW, (O, D), "hdW"), wp, _vec(v),
        ctypes.c_void_p(staging.data_ptr()), staging.numel(), N, D, O, Dsub,
        ctypes.c_void_p(ws.data_ptr()), ws.numel(), _stream(stream))
    _check(rc, "velora_linear_step_host")


def velora_subtoken_sum(X: torch.Tensor, Dsub: int, s: Optional[torch.Tensor] = None,
                        ws: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """Un-normalised sub-token sum of this rank's shard (add the ranks' sums, then velora_normalize_v)."""
    N, D = X.shape
    xp, ldx = (_mat(X, "X") if N > 0 else (ctypes.c_void_p(0), D))
    if s is None:
        s = torch.empty(Dsub, dtype=torch.float32, device=X.device)
    ws = _ws(ws, velora_workspace_bytes(OP_INIT_V, max(N, 1), D, 1, Dsub), X.device)
    rc = lib().velora_subtoken_sum(xp, _dt(X), N, D, ldx, Dsub, _vec(s), ctypes.c_void_p(ws.data_ptr()), ws.numel(),
                                   _stream(stream))
    _check(rc, "velora_subtoken_sum")
    return s


def velora_update_v(X: torch.Tensor, Dsub: int, rho: float, a: torch.Tensor, v: torch.Tensor,
                    ws: Optional[torch.Tensor] = None, stream=None) -> None:
    """Running-average variant: a <- (1 - rho) a + rho * (mean sub-token of X), v <- a / ||a||, in place, no sync."""
    xp, ldx = _mat(X, "X")
    N, D = X.shape
    if ws is None:
        ws = velora_workspace_alloc(velora_workspace_bytes(OP_UPDATE_V, N, D, 1, Dsub), X.device)
    rc = lib().velora_update_v(xp, _dt(X), N, D, ldx, Dsub, float(rho), _vec(a), _vec(v),
                               ctypes.c_void_p(ws.data_ptr()), ws.numel(), _stream(stream))
    _check(rc, "velora_update_v")


def velora_normalize_v(s: torch.Tensor, v: Optional[torch.Tensor] = None, ws: Optional[torch.Tensor] = None,
                       stream=None) -> torch.Tensor:
    Dsub = s.shape[0]
    if v is None:
        v = torch.empty_like(s)
    ws = _ws(ws, 256, s.device)
    rc = lib().velora_normalize_v(_vec(s), Dsub, _vec(v), ctypes.c_void_p(ws.data_ptr()), ws.numel(), _stream(stream))
    _check(rc, "velora_normalize_v")
    return v


def velora_weight_grad_p(dY: torch.Tensor, Z: torch.Tensor, D: int, Dsub: int, P: Optional[torch.Tensor] = None,
                         beta: int = 0, ws: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """P[O, M] = beta * P + dY^T Z in fp32: the weight gradient before its expansion by v."""
    N, O = dY.shape
    M = num_subtokens(D, Dsub)
    yp, lddy = (_mat(dY, "dY") if N > 0 else (ctypes.c_void_p(0), O))
    zp, ldz = (_mat(Z, "Z") if N > 0 else (ctypes.c_void_p(0), M))
    if P is None:
        P = torch.zeros((O, M), dtype=torch.float32, device=dY.device)
    pp, ldp = _mat(P, "P")
    ws = _ws(ws, velora_workspace_bytes(OP_WEIGHT_GRAD_FACTORED, N, D, O, Dsub), dY.device)
    rc = lib().velora_weight_grad_p(yp, _dt(dY), N, O, lddy, zp, _dt(Z), ldz, D, Dsub, pp, ldp, beta,
                                    ctypes.c_void_p(ws.data_ptr()), ws.numel(), _stream(stream))
    _check(rc, "velora_weight_grad_p")
    return P


def velora_expand_p(P: torch.Tensor, v: torch.Tensor, D: int, dW: Optional[torch.Tensor] = None,
                    dw_dtype=torch.bfloat16, beta: int = 0, stream=None) -> torch.Tensor:
    """dW[o, m*Dsub + j] = beta * dW + P[o, m] v[j]."""
    O = P.shape[0]
    Dsub = v.shape[0]
    pp, ldp = _mat(P, "P")
    if dW is None:
        dW = torch.empty((O, D), dtype=dw_dtype, device=P.device)
    wp, lddw = _mat(dW, "dW")
    rc = lib().velora_expand_p(pp, ldp, _vec(v), O, D, Dsub, wp, _dt(dW), lddw, beta, _stream(stream))
    _check(rc, "velora_expand_p")
    return dW
