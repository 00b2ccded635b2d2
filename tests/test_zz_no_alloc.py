"""velora_init_v_static: the workspace-free variant of velora_init_v.

Some callers cannot hand the library a workspace because they cannot allocate device memory at the
point of the call (a plugin inside a framework that owns the allocator, a loop that must stay clear
of the driver's allocator).  For them the library keeps a fixed scratch array of its own.  This test
calls that entry point through the C-ABI twice in a row, on different inputs, and checks each result
against what velora_init_v gives with an ordinary workspace and against the CPU oracle; the second call
also shows that whatever the first one left in the shared array does no harm.  The file name keeps it last in collection
order, so a run that stops at the first failure has already been through every other test.
"""
import ctypes

import pytest
import torch

import oracle
import velora_inputs as vi

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


def test_static_scratch_matches_workspace_variant_on_two_calls_in_a_row():
    import paper_2405_17991_b200 as vl
    lib = vl.lib()
    stream = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    cases = [
        vi.small_case(901, 3000, 1024, 8, dtype="bf16", mean_offset=0.2)["X"],   # vector kernels
        vi.small_case(902, 517, 200, 8, dtype="f32", mean_offset=-0.3)["X"],     # element kernels
    ]
    for Xa, Dsub in zip(cases, (256, 40)):
        X = Xa.torch(DEV)
        N, D = X.shape
        ref = vl.velora_init_v(X, Dsub)                       # existing entry point, caller's workspace
        v = torch.zeros(Dsub, dtype=torch.float32, device=DEV)
        rc = lib.velora_init_v_static(ctypes.c_void_p(X.data_ptr()), 1 if X.dtype == torch.bfloat16 else 0,
                                      N, D, X.stride(0), Dsub, ctypes.c_void_p(v.data_ptr()), stream)
        assert rc == 0, vl.velora_status_string(rc)
        err = float(torch.linalg.vector_norm(v.double() - ref.double()) / torch.linalg.vector_norm(ref.double()))
        assert err <= 1e-3, err                               # the tolerance used for v elsewhere
        v_ref = oracle.init_v(Xa.f64(), Dsub)
        got = v.double().cpu().numpy()
        assert float(((got - v_ref) ** 2).sum() ** 0.5) <= 1e-3           # ||v_ref|| = 1: relative = absolute
        assert float(abs(got - v_ref).max()) <= 1e-3 * Dsub ** -0.5       # element-wise, against v's rms
        assert abs(float(torch.linalg.vector_norm(v.double())) - 1.0) < 1e-5


def test_static_scratch_rejects_what_does_not_fit():
    import paper_2405_17991_b200 as vl
    lib = vl.lib()
    X = torch.ones((4, 1024), dtype=torch.bfloat16, device=DEV)
    v = torch.zeros(512, dtype=torch.float32, device=DEV)
    rc = lib.velora_init_v_static(ctypes.c_void_p(X.data_ptr()), 1, 4, 1024, 1024, 512,
                                  ctypes.c_void_p(v.data_ptr()), ctypes.c_void_p(0))
    assert rc == vl.binding.ERR_UNSUPPORTED
    assert torch.all(v == 0)
