"""Helpers shared by the GPU parity tests (comparison rules only; no method arithmetic)."""
import numpy as np
import torch

import oracle

TOL_Z = 1e-3        # Z and Xhat: relative error, norm-wise
TOL_GEMM = 1e-2     # dW, Y, dX: relative Frobenius error


def to_f64(t: torch.Tensor) -> np.ndarray:
    """Exact widening of a tensor's stored values."""
    return t.detach().to("cpu").to(torch.float64).numpy()


def dtype_name(t: torch.Tensor) -> str:
    return {torch.float32: "f32", torch.bfloat16: "bf16"}[t.dtype]


def rel_err(got: np.ndarray, ref: np.ndarray) -> float:
    den = np.linalg.norm(ref)
    return float(np.linalg.norm(got - ref) / (den if den > 0 else 1.0))


def ulp(ref: np.ndarray, dtype: str) -> np.ndarray:
    bits = {"bf16": 8, "f32": 24}[dtype]
    _, e = np.frexp(ref)
    return np.ldexp(1.0, e - bits)


def assert_matches(got_t: torch.Tensor, ref64: np.ndarray, tol: float, what: str, ulps: float = None):
    """The comparison rule for a stored output.

    The oracle's float64 result is rounded once (nearest even) to the output's storage type, then
    (i) the norm-wise relative error must be below ``tol``; (ii) if ``ulps`` is given every element
    must be within that many units in the last place of the rounded oracle value, or within
    ``1e-3 * rms(ref)`` absolutely (cancellation near zero).
    """
    dt = dtype_name(got_t)
    got = to_f64(got_t)
    assert got.shape == ref64.shape, (what, got.shape, ref64.shape)
    assert np.all(np.isfinite(got)), what + ": non-finite output"
    ref = oracle.round_to(ref64, dt)
    err = rel_err(got, ref)
    assert err <= tol, "%s: relative error %.3e > %.1e" % (what, err, tol)
    if ulps is not None:
        rms = np.sqrt(np.mean(ref64 * ref64)) if ref64.size else 0.0
        bad = np.abs(got - ref) > np.maximum(ulps * ulp(ref, dt), 1e-3 * rms)
        assert not bad.any(), "%s: %d elements beyond %g ulp" % (what, int(bad.sum()), ulps)
    return err
