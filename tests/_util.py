"""Helpers shared by the GPU parity tests: the comparison rule and guard-banded output buffers.

Nothing here computes any step of the method; the oracle is only asked to round its own results to
a storage type.

Comparison rule for a stored output ``got`` against the oracle's float64 result ``ref64``:

1. ``ref64`` is rounded once (nearest even) to the output's storage type -> ``ref``.
2. Norm-wise:  ``||got - ref|| / ||ref|| <= tol``   (TOL_Z for Z and Xhat, TOL_GEMM for Y, dX, dW, P).
3. Element-wise, for EVERY element:
   ``|got - ref| <= ulps * ulp(ref) + c * max(rms of ref's column, rms of all of ref)``.

Where the rule and its constants come from (arithmetic of the kernels, not from what happened to pass):

* The kernel stores ``RN(x + e)`` where ``x`` is the exact value, ``e`` the error of its fp32 arithmetic and
  ``RN`` the rounding to the storage type; the oracle side is ``RN(x)``.  Two roundings of values ``|e|``
  apart differ by at most ``|e|`` plus one unit in the last place, hence the SUM of the two terms with
  ``ulps = 1`` (for an fp32 output the unit is negligible and the rule is the absolute term alone).
* ``C_STREAM = 1e-3`` (Z, Xhat, v): an fp32 sum of K <= 1024 products carries, with probability all
  but 1e-9 per element, an error below ``6 * sqrt(K) * 2^-24 * sum|x_j v_j|`` (random-sign rounding
  model), and ``sum|x_j v_j|`` is about ``0.64 * sqrt(K)`` times the rms of the result: ``3.84 * K *
  2^-24 = 2.3e-4`` of the rms at K = 1024.  1e-3 is that with a factor four in hand.
* ``C_SUM = 4e-3`` (Y, dX, dW and P from operands used as stored): the same bound for contractions
  of up to K = 16384 terms, ``3.84 * 16384 * 2^-24 = 3.75e-3``.
* ``C_ROUNDED = C_SUM + 1.16e-2`` (dW through the explicit route, whose Xhat is stored in bf16; dW and P
  through the factored route when Z arrives in fp32 and is fed to the tensor cores as bf16): every
  term then carries an independent relative rounding error.  bf16 values in [1, 2) are 2^-7 apart, so the
  error is uniform within +-2^-8 of the binade's base: standard deviation ``2^-7 / sqrt(12) / m`` for a
  significand m, ``1.66e-3`` in the root mean square over m.  A sum of terms with independent errors of
  that size is off by 1.66e-3 of its own root-mean-square size (one sigma); 7 sigma = 1.16e-2 leaves a
  chance of 1e-4 that any of 5e7 elements exceeds it.

The root-mean-square size is taken per output column (channel scales differ by column: heavy-tailed
or outlier channels) with the whole output's rms as a floor, which covers elements that are small
by cancellation.
"""
import numpy as np
import torch

import oracle

TOL_Z = 1e-3        # Z and Xhat: relative error, norm-wise
TOL_GEMM = 1e-2     # dW, Y, dX: relative Frobenius error

C_STREAM = 1e-3
C_SUM = 4e-3
C_ROUNDED = C_SUM + 1.16e-2
C_TINY = 1e-4       # configuration 1 (every contraction has K <= 256 terms): 3.84 * 256 * 2^-24 = 5.9e-5


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


def _default_c(tol: float) -> float:
    return C_STREAM if tol <= TOL_Z else C_SUM


def assert_matches(got_t: torch.Tensor, ref64: np.ndarray, tol: float, what: str, ulps: float = 1.0,
                   c: float = None):
    """The comparison rule of this module's docstring.  ``c`` defaults to C_STREAM when ``tol`` is
    TOL_Z or tighter and to C_SUM otherwise; pass C_ROUNDED where an operand was rounded on the way."""
    dt = dtype_name(got_t)
    got = to_f64(got_t)
    assert got.shape == ref64.shape, (what, got.shape, ref64.shape)
    assert np.all(np.isfinite(got)), what + ": non-finite output"
    ref = oracle.round_to(ref64, dt)
    err = rel_err(got, ref)
    assert err <= tol, "%s: relative error %.3e > %.1e" % (what, err, tol)
    if c is None:
        c = _default_c(tol)
    if ref64.size:
        rms_all = float(np.sqrt(np.mean(ref64 * ref64)))
        if ref64.ndim == 2:
            scale = np.maximum(np.sqrt(np.mean(ref64 * ref64, axis=0, keepdims=True)), rms_all)
        else:
            scale = rms_all
        diff = np.abs(got - ref)
        bound = ulps * ulp(ref, dt) + c * scale
        bad = diff > bound
        if bad.any():
            worst = np.unravel_index(np.argmax(diff / bound), diff.shape)
            raise AssertionError("%s: %d of %d elements beyond %g ulp + %.1e rms; worst at %r: got %r, ref %r"
                                 % (what, int(bad.sum()), bad.size, ulps, c, tuple(int(i) for i in worst),
                                    got[worst], ref[worst]))
    return err


# ------------------------------------------------------------------ guard-banded outputs
_SENTINEL = {torch.bfloat16: (torch.int16, 0x7FC1), torch.float32: (torch.int32, 0x7FC00001),
             torch.uint8: (torch.uint8, 0xA5), torch.int32: (torch.int32, 0x7FC00001)}


class Guard:
    """Hands out output tensors that are views into larger buffers filled with a NaN bit pattern, and
    afterwards checks that every byte outside the views still holds it.

    A kernel that stores past the last row, into the padding between a row's width and its pitch, or
    before its first element shows up here even when the values it was meant to write are right -- the
    stand-in for a memory checker.  Matrices get ``rows`` sentinel rows above and below and a pitch wider
    than their width (a multiple of 8 elements, so that the vector kernels still run); vectors and workspaces
    get 256 sentinel elements on either side.
    """

    def __init__(self, device, rows: int = 3):
        self.device, self.rows = device, rows
        self.items = []

    def _filled(self, shape, dtype):
        idt, pat = _SENTINEL[dtype]
        raw = torch.full(shape, pat, dtype=idt, device=self.device)
        return raw, raw.view(dtype)

    def mat(self, n_rows: int, n_cols: int, dtype=torch.bfloat16, ld: int = None, init: torch.Tensor = None):
        if ld is None:
            ld = -(-n_cols // 8) * 8 + 8
        assert ld >= n_cols
        g = self.rows
        raw, buf = self._filled((n_rows + 2 * g, ld), dtype)
        view = buf[g:g + n_rows, :n_cols]
        if init is not None:
            view.copy_(init)
        bands = [("rows above", raw[:g]), ("rows below", raw[g + n_rows:]), ("row padding", raw[g:g + n_rows, n_cols:])]
        self.items.append((bands, _SENTINEL[dtype][1], "matrix %dx%d (pitch %d)" % (n_rows, n_cols, ld)))
        return view

    def vec(self, n: int, dtype=torch.float32):
        raw, buf = self._filled((n + 512,), dtype)
        self.items.append(([("before", raw[:256]), ("after", raw[256 + n:])], _SENTINEL[dtype][1], "vector %d" % n))
        return buf[256:256 + n]

    def workspace(self, vl, nbytes: int):
        """A workspace of exactly ``nbytes`` (at least the status header) between two sentinel bands."""
        ws = self.vec(max(int(nbytes), 256), torch.uint8)
        vl.velora_workspace_init(ws)
        return ws

    def check(self):
        torch.cuda.synchronize(self.device)
        for bands, pat, what in self.items:
            for name, band in bands:
                touched = band != pat
                if band.numel() and bool(touched.any()):
                    where = torch.nonzero(touched)[:4].tolist()
                    raise AssertionError("guard band of %s overwritten: %s, at %r (%d elements)"
                                         % (what, name, where, int(touched.sum())))
        self.items = []
