"""VeLoRA fp64 CPU oracle -- TEST INFRASTRUCTURE, NOT A PRODUCT PATH.

Thin numpy/ctypes front of ``velora_oracle.c`` (same directory), the plain
double-precision restatement of the paper's operators (arxiv 2405.17991,
Section 3.1 and Algorithm 1).  Only the tests, the smoke check and the
benchmark's CPU-baseline leg may import this module; the CUDA library and its
Python binding never do, and this module imports nothing of theirs.

All arrays are float64, C-contiguous, row-major.  Shapes use
``N`` tokens, ``D`` input width, ``Dsub`` sub-token length (the paper's M),
``M = ceil(D / Dsub)`` sub-tokens per token, ``O`` output width.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "velora_oracle.c")
_LIB = os.path.join(_HERE, "libvelora_oracle.so")

OK = 0
BAD_ARG = 1
DEGENERATE_V = 5


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (-O2, OpenMP) into this directory."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.run(
            ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"],
            check=True,
        )
        os.replace(tmp, _LIB)
    return _LIB


_lib = None
_p = ctypes.c_void_p
_i64 = ctypes.c_int64


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.velora_oracle_threads.restype = ctypes.c_int
        lib.velora_oracle_threads.argtypes = []
        lib.velora_oracle_init_v.argtypes = [_p, _i64, _i64, _i64, _i64, _p, _p, _p]
        lib.velora_oracle_update_v.argtypes = [_p, _i64, _i64, _i64, _i64, ctypes.c_double, _p, _p, _p]
        lib.velora_oracle_update_v.restype = ctypes.c_int
        lib.velora_oracle_compress.argtypes = [_p, _i64, _i64, _i64, _i64, _p, _p, _i64]
        lib.velora_oracle_reconstruct.argtypes = [_p, _i64, _i64, _i64, _i64, _p, _p, _i64]
        lib.velora_oracle_weight_grad_bruteforce.argtypes = [
            _p, _i64, _i64, _i64, _p, _i64, _p, _i64, _i64, _p, _i64, ctypes.c_int]
        lib.velora_oracle_weight_grad_factored.argtypes = [
            _p, _i64, _i64, _i64, _p, _i64, _p, _i64, _i64, _p, _i64, ctypes.c_int, _p]
        lib.velora_oracle_linear_forward.argtypes = [_p, _i64, _i64, _i64, _p, _i64, _i64, _p, _i64]
        lib.velora_oracle_input_grad.argtypes = [_p, _i64, _i64, _i64, _p, _i64, _i64, _p, _i64]
        for name in ("init_v", "compress", "reconstruct", "weight_grad_bruteforce",
                     "weight_grad_factored", "linear_forward", "input_grad"):
            getattr(lib, "velora_oracle_" + name).restype = ctypes.c_int
        _lib = lib
    return _lib


def _f64(a, ndim):
    a = np.ascontiguousarray(a, dtype=np.float64)
    if a.ndim != ndim:
        raise ValueError("expected a %d-d array, got shape %r" % (ndim, a.shape))
    return a


def _ptr(a):
    return ctypes.c_void_p(a.ctypes.data)


def _check(rc, what):
    if rc != OK:
        raise OracleError(rc, what)


class OracleError(RuntimeError):
    def __init__(self, code, what):
        super().__init__("%s failed with oracle status %d" % (what, code))
        self.code = code


def threads() -> int:
    """Number of OpenMP threads the C oracle will use."""
    return int(_load().velora_oracle_threads())


def num_subtokens(D: int, Dsub: int) -> int:
    return -(-D // Dsub)


def init_v(X, Dsub, return_sum=False):
    """v = s/||s||, s = sum of all sub-tokens of X (Section 3.2, cheap initialisation)."""
    X = _f64(X, 2)
    N, D = X.shape
    v = np.zeros(Dsub, dtype=np.float64)
    s = np.zeros(Dsub, dtype=np.float64)
    norm = ctypes.c_double(0.0)
    rc = _load().velora_oracle_init_v(_ptr(X), N, D, D, Dsub, _ptr(v), _ptr(s), ctypes.byref(norm))
    _check(rc, "init_v")
    if return_sum:
        return v, s, norm.value
    return v


def update_v(X, Dsub, rho, a=None):
    """Running-average variant (Section 5, initialisation ablation): a' = (1-rho) a + rho mean, v = a'/||a'||.

    Returns (a', v)."""
    X = _f64(X, 2)
    N, D = X.shape
    a_in = None if a is None else _f64(a, 1)
    a_out = np.zeros(Dsub, dtype=np.float64)
    v = np.zeros(Dsub, dtype=np.float64)
    rc = _load().velora_oracle_update_v(_ptr(X), N, D, D, Dsub, float(rho),
                                        _ptr(a_in) if a_in is not None else None, _ptr(a_out), _ptr(v))
    _check(rc, "update_v")
    return a_out, v


def compress(X, v):
    """Z[n,m] = <sub-token m of token n, v> (Section 3.1, Eq. 1)."""
    X = _f64(X, 2)
    v = _f64(v, 1)
    N, D = X.shape
    Dsub = v.shape[0]
    M = num_subtokens(D, Dsub)
    Z = np.zeros((N, M), dtype=np.float64)
    _check(_load().velora_oracle_compress(_ptr(X), N, D, D, Dsub, _ptr(v), _ptr(Z), M), "compress")
    return Z


def reconstruct(Z, v, D):
    """Xhat[n, m*Dsub+j] = Z[n,m] v[j] (Section 3.1, Eq. 2)."""
    Z = _f64(Z, 2)
    v = _f64(v, 1)
    N, M = Z.shape
    Dsub = v.shape[0]
    if M != num_subtokens(D, Dsub):
        raise ValueError("Z has %d columns, expected %d" % (M, num_subtokens(D, Dsub)))
    Xhat = np.zeros((N, D), dtype=np.float64)
    _check(_load().velora_oracle_reconstruct(_ptr(Z), M, N, D, Dsub, _ptr(v), _ptr(Xhat), D), "reconstruct")
    return Xhat


def weight_grad(dY, Z, v, D, dW0=None, factored=False, return_P=False):
    """dW = beta*dW0 + dY^T reconstruct(Z, v) (Algorithm 1, backward).

    ``factored=False`` is the plain definition; ``factored=True`` the rank-1 form
    ``(dY^T Z)[o,m] v[j]``.  ``dW0`` given means beta = 1.
    """
    dY = _f64(dY, 2)
    Z = _f64(Z, 2)
    v = _f64(v, 1)
    N, O = dY.shape
    Dsub = v.shape[0]
    M = num_subtokens(D, Dsub)
    if Z.shape != (N, M):
        raise ValueError("Z shape %r, expected %r" % (Z.shape, (N, M)))
    beta = 0 if dW0 is None else 1
    dW = np.zeros((O, D), dtype=np.float64) if dW0 is None else _f64(dW0, 2).copy()
    if dW.shape != (O, D):
        raise ValueError("dW0 shape %r, expected %r" % (dW.shape, (O, D)))
    lib = _load()
    if factored:
        P = np.zeros((O, M), dtype=np.float64)
        rc = lib.velora_oracle_weight_grad_factored(_ptr(dY), N, O, O, _ptr(Z), M, _ptr(v), D, Dsub,
                                                    _ptr(dW), D, beta, _ptr(P))
        _check(rc, "weight_grad_factored")
        return (dW, P) if return_P else dW
    rc = lib.velora_oracle_weight_grad_bruteforce(_ptr(dY), N, O, O, _ptr(Z), M, _ptr(v), D, Dsub,
                                                  _ptr(dW), D, beta)
    _check(rc, "weight_grad_bruteforce")
    return dW


def linear_forward(X, W):
    """Y = X W^T with W[O, D] (Algorithm 1, forward)."""
    X = _f64(X, 2)
    W = _f64(W, 2)
    N, D = X.shape
    O = W.shape[0]
    if W.shape[1] != D:
        raise ValueError("W shape %r does not match D=%d" % (W.shape, D))
    Y = np.zeros((N, O), dtype=np.float64)
    _check(_load().velora_oracle_linear_forward(_ptr(X), N, D, D, _ptr(W), O, D, _ptr(Y), O), "linear_forward")
    return Y


def input_grad(dY, W):
    """dX = dY W with W[O, D] (Algorithm 1, backward)."""
    dY = _f64(dY, 2)
    W = _f64(W, 2)
    N, O = dY.shape
    D = W.shape[1]
    if W.shape[0] != O:
        raise ValueError("W shape %r does not match O=%d" % (W.shape, O))
    dX = np.zeros((N, D), dtype=np.float64)
    _check(_load().velora_oracle_input_grad(_ptr(dY), N, O, O, _ptr(W), D, D, _ptr(dX), D), "input_grad")
    return dX


# ---- value-format helpers used when an oracle result is compared with a stored dtype ----

def round_to_bf16(a):
    """Round float64 values to the nearest bfloat16 value (ties to even), returned as float64.

    bfloat16 has an 8-bit significand: scale each value so its significand is an
    integer below 256, round to the nearest even integer, scale back.  Zeros,
    infinities and NaNs pass through; subnormal and overflow ranges are not needed here.
    """
    a = np.asarray(a, dtype=np.float64)
    mant, expo = np.frexp(a)                       # a = mant * 2**expo, 0.5 <= |mant| < 1
    return np.ldexp(np.rint(mant * 256.0), expo - 8)


def round_to_f32(a):
    """Round float64 values to the nearest float32 value, returned as float64."""
    return np.asarray(a, dtype=np.float64).astype(np.float32).astype(np.float64)


FP8_E4M3_MAX = 448.0


def round_to_fp8_e4m3(a):
    """Round float64 values to the nearest value of the 8-bit format E4M3 (1 sign, 4 exponent bits with
    bias 7, 3 mantissa bits; no infinities, largest finite value 448), ties to even, SATURATING: anything
    beyond +-448 (infinities included) becomes +-448.  Returned as float64; NaN stays NaN.

    Normal values (|x| >= 2^-6) have a 4-bit significand, so in frexp form (x = mant * 2^expo,
    0.5 <= |mant| < 1) neighbours are 2^(expo - 4) apart.  Below 2^-6 the format is subnormal with the
    fixed spacing 2^-9, which is the same formula with expo held at -5.
    """
    a = np.asarray(a, dtype=np.float64)
    _, expo = np.frexp(a)
    step = np.ldexp(1.0, np.maximum(expo, -5) - 4)
    with np.errstate(invalid="ignore"):
        q = np.rint(a / step) * step
    q = np.where(np.isnan(a), a, np.clip(q, -FP8_E4M3_MAX, FP8_E4M3_MAX))
    return np.where(np.isinf(a), np.sign(a) * FP8_E4M3_MAX, q)


def zscale_from_batch(Z, headroom: float = 2.0) -> float:
    """Scale for storing Z in E4M3 (extension of Section 3.1's stored scalars to an 8-bit store; not in
    the paper): the largest magnitude of a calibration batch times ``headroom`` maps to 448.  A batch
    without a finite positive maximum gives 1."""
    amax = float(np.max(np.abs(Z))) if np.size(Z) else 0.0
    if not np.isfinite(amax) or amax <= 0.0:
        return 1.0
    return headroom * amax / FP8_E4M3_MAX


def quantize_z_fp8(Z, zscale: float):
    """The values an E4M3 store of Z holds: round_to_fp8_e4m3(Z / zscale), as float64 (multiply by zscale
    to get the Z that the backward pass sees)."""
    return round_to_fp8_e4m3(np.asarray(Z, dtype=np.float64) / float(zscale))


def round_to(a, dtype: str):
    if dtype == "bf16":
        return round_to_bf16(a)
    if dtype == "f32":
        return round_to_f32(a)
    if dtype == "f64":
        return np.asarray(a, dtype=np.float64)
    raise ValueError(dtype)
