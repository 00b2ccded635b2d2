"""CPU-only checks: the C-ABI library loads and exports what include/velora.h declares,
host-side validation rejects bad arguments before any launch, and the memory model
reproduces the structure of the paper's Table 5(b)."""
import ctypes
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2405_17991_b200 import build, binding
    build.build()
    return binding.lib()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "velora.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(velora_[a-z_0-9]+)\s*\(", text)))


def test_header_symbols_are_exported_and_bound(lib):
    from paper_2405_17991_b200 import binding
    names = declared_symbols()
    assert {"velora_init_v", "velora_compress", "velora_reconstruct", "velora_weight_grad",
            "velora_linear_forward", "velora_linear_backward"} <= set(names)
    for name in names:
        assert hasattr(lib, name), name
        assert name in binding.SIGNATURES, name
        assert callable(getattr(binding, name, None)), name


def test_version_and_status_strings(lib):
    assert lib.velora_version() >= 100
    seen = {lib.velora_status_string(i) for i in range(8)}
    assert len(seen) == 8 and all(s for s in seen)


def test_workspace_queries_need_no_device(lib):
    from paper_2405_17991_b200 import binding as b
    assert lib.velora_workspace_bytes(b.OP_INIT_V, 8192, 4096, 4096, 64) >= 1184 * 64 * 4
    assert lib.velora_workspace_bytes(b.OP_WEIGHT_GRAD_EXPLICIT, 100, 30, 8, 8) >= 100 * 32 * 2
    assert lib.velora_workspace_bytes(b.OP_WEIGHT_GRAD_FACTORED, 100, 64, 8, 8) >= 8 * 8 * 4
    assert lib.velora_workspace_bytes(b.OP_INIT_V, 10, 4, 4, 8) == 0          # Dsub > D
    assert lib.velora_workspace_bytes(99, 10, 8, 4, 4) == 0


def test_validation_happens_on_the_host_before_any_launch(lib):
    """Bad arguments are rejected from metadata alone: the fake pointers are never dereferenced."""
    from paper_2405_17991_b200 import binding as b
    P = ctypes.c_void_p
    good, odd = P(0x10000), P(0x10001)
    null = P(0)
    # compress
    f = lib.velora_compress
    assert f(null, b.BF16, 4, 64, 64, 16, good, good, b.F32, 4, null) == b.ERR_INVALID_ARG
    assert f(good, b.BF16, -1, 64, 64, 16, good, good, b.F32, 4, null) == b.ERR_INVALID_ARG
    assert f(good, b.BF16, 4, 64, 63, 16, good, good, b.F32, 4, null) == b.ERR_INVALID_ARG     # ldx < D
    assert f(good, b.BF16, 4, 64, 64, 16, good, good, b.F32, 3, null) == b.ERR_INVALID_ARG     # ldz < M
    assert f(good, b.BF16, 4, 64, 64, 0, good, good, b.F32, 4, null) == b.ERR_INVALID_ARG
    assert f(good, b.BF16, 4, 64, 64, 65, good, good, b.F32, 1, null) == b.ERR_INVALID_ARG     # Dsub > D
    assert f(good, b.BF16, 4, 4096, 4096, 2048, good, good, b.F32, 2, null) == b.ERR_UNSUPPORTED
    assert f(good, 7, 4, 64, 64, 16, good, good, b.F32, 4, null) == b.ERR_UNSUPPORTED
    assert f(odd, b.BF16, 4, 64, 64, 16, good, good, b.F32, 4, null) == b.ERR_ALIGNMENT
    assert f(good, b.BF16, 0, 64, 64, 16, good, good, b.F32, 4, null) == b.OK                   # N = 0: no-op
    # init_v
    g = lib.velora_init_v
    assert g(good, b.BF16, 4, 64, 64, 16, good, null, 0, null) == b.ERR_WORKSPACE
    assert g(good, b.BF16, 4, 64, 64, 16, good, good, 16, null) == b.ERR_WORKSPACE
    assert g(good, b.BF16, 0, 64, 64, 16, good, good, 1 << 30, null) == b.ERR_DEGENERATE_V
    # weight_grad
    h = lib.velora_weight_grad
    args = [good, b.BF16, 4, 8, 8, good, b.F32, 4, good, 64, 16, good, b.BF16, 64]
    assert h(*args, 2, b.WG_FACTORED, good, 1 << 30, null) == b.ERR_INVALID_ARG                 # beta
    assert h(*args, 0, 5, good, 1 << 30, null) == b.ERR_INVALID_ARG                             # mode
    assert h(*args, 0, b.WG_FACTORED, null, 0, null) == b.ERR_WORKSPACE
    assert h(*args, 0, b.WG_FACTORED, good, 8, null) == b.ERR_WORKSPACE
    # an empty batch may come with NULL data pointers: dW = beta * dW, nothing to launch when beta = 1
    assert h(null, b.BF16, 0, 8, 8, null, b.F32, 4, null, 64, 16, good, b.BF16, 64, 1, b.WG_FACTORED,
             good, 1 << 30, null) == b.OK
    assert h(null, b.BF16, 0, 8, 8, null, b.F32, 4, null, 64, 16, null, b.BF16, 64, 1, b.WG_FACTORED,
             good, 1 << 30, null) == b.ERR_INVALID_ARG                                          # dW is still needed
    # the wait self-test validates its limit and workspace before launching
    st = lib.velora_selftest_wait_timeout
    assert st(good, 256, 10, good, null) == b.ERR_INVALID_ARG                                   # below 1 us
    assert st(good, 256, 10 ** 9, good, null) == b.ERR_INVALID_ARG                              # above 100 ms
    assert st(null, 256, 10 ** 6, good, null) == b.ERR_WORKSPACE
    assert st(good, 256, 10 ** 6, null, null) == b.ERR_INVALID_ARG
    # the 8-bit type is a storage type for Z only
    assert f(good, b.FP8_E4M3, 4, 64, 64, 16, good, good, b.F32, 4, null) == b.ERR_UNSUPPORTED  # X in E4M3: no
    assert h(good, b.BF16, 4, 8, 8, good, b.FP8_E4M3, 4, good, 64, 16, good, b.FP8_E4M3, 64, 0, b.WG_FACTORED,
             good, 1 << 30, null) == b.ERR_UNSUPPORTED                                           # dW in E4M3: no
    zc = lib.velora_z8_calibrate
    assert zc(good, b.BF16, 4, 64, 64, 16, good, 0.5, good, good, good, good, 1 << 20, null) == b.ERR_INVALID_ARG   # headroom < 1
    assert zc(good, b.BF16, 4, 64, 64, 16, good, 2.0, good, good, good, good, 16, null) == b.ERR_WORKSPACE
    assert lib.velora_workspace_bytes(b.OP_Z8_CALIBRATE, 100, 64, 0, 16) >= 100 * 4 * 4
    # reconstruct / linear
    r = lib.velora_reconstruct
    assert r(good, b.F32, 4, 4, 64, 16, good, good, b.BF16, 60, null) == b.ERR_INVALID_ARG
    lf = lib.velora_linear_forward
    assert lf(good, 64, good, 64, good, good, 7, good, b.F32, 4, b.BF16, 4, 64, 8, 16, null, 0, null) == b.ERR_INVALID_ARG
    lb = lib.velora_linear_backward
    assert lb(null, 8, good, 64, good, b.F32, 4, good, good, 64, good, b.BF16, 64, 0, 0,
              b.BF16, 4, 64, 8, 16, good, 1 << 30, null) == b.ERR_INVALID_ARG


def test_binding_fails_loudly_without_the_library(monkeypatch, tmp_path):
    from paper_2405_17991_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "missing.so"))
    with pytest.raises(RuntimeError, match="no CPU or PyTorch fallback"):
        binding.lib()


def test_memory_model_matches_table_5b_structure():
    """Stored bytes are affine in the number of sub-tokens: the table's differences halve."""
    from paper_2405_17991_b200 import saved_activation_bytes
    rows = [tuple(map(float, l.split())) for l in open(os.path.join(ROOT, "tests", "golden",
            "table5b_activation_memory.txt")) if l.strip() and not l.startswith("#")]
    k = np.array([r[0] for r in rows])
    mb = np.array([r[1] for r in rows])
    # printed values: affine in the group count k within the table's 1 MB rounding
    A = np.stack([k, np.ones_like(k)], axis=1)
    coef, *_ = np.linalg.lstsq(A, mb, rcond=None)
    assert np.max(np.abs(A @ coef - mb)) < 1.0 and coef[0] > 0
    # the model: same affine law, exactly
    D, N = 4096, 512
    model = np.array([saved_activation_bytes(N, D, int(D // kk)) - (D // kk) * 4 for kk in k], dtype=float)
    slope = (model[0] - model[-1]) / (k[0] - k[-1])
    np.testing.assert_allclose(model, model[-1] + slope * (k - k[-1]), rtol=1e-12)
    assert saved_activation_bytes(N, D, 64) * 30 < saved_activation_bytes(N, D, None)
    assert saved_activation_bytes(10, 1376, 64) == 10 * 22 * 4 + 64 * 4      # ragged: ceil(1376/64) = 22
    # storage types of Z: 4, 2 and 1 bytes per scalar; against the bf16 input at Dsub = 64 that is 32x, 64x, 128x
    full = saved_activation_bytes(1 << 20, D, None)
    for zb, ratio in ((4, 32), (2, 64), (1, 128)):
        assert abs(full / saved_activation_bytes(1 << 20, D, 64, z_bytes=zb) / ratio - 1) < 1e-3
