"""GPU parity: every C-ABI entry point against the fp64 CPU oracle on the same seeded inputs.

Tolerances (derived from the arithmetic: bf16 inputs, fp32 products and sums): Z and Xhat within
1e-3 norm-wise relative error; dW, Y, dX within 1e-2 relative Frobenius error; on top of that every
single element is held to the element-wise bound of ``_util.assert_matches``.  An output stored in
bf16 or fp32 is compared with the oracle's float64 result rounded once to that type.  Each entry
point is checked on its own inputs: reconstruct and weight_grad oracles take the very Z buffer the
GPU call receives.  Every output a test hands to the library lives inside a sentinel-filled buffer
(``_util.Guard``) whose bands are checked after the test: stores past a row's width, past the last
row or outside a workspace's declared size fail the test even if all values are right.
"""
import numpy as np
import pytest
import torch

import oracle
import velora_inputs as vi
from _util import C_ROUNDED, C_SUM, C_TINY, TOL_GEMM, TOL_Z, Guard, assert_matches, rel_err, to_f64

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


@pytest.fixture(scope="module")
def vl():
    import paper_2405_17991_b200 as pkg
    pkg.lib()                      # raises if the CUDA library is missing: no fallback
    return pkg


@pytest.fixture
def guard():
    g = Guard(DEV)
    yield g
    g.check()


class Outs:
    """The library's entry points with every output placed in a guard-banded buffer."""

    def __init__(self, vl, g):
        self.vl, self.g = vl, g

    def ws(self, op, N, D, O, Dsub):
        return self.g.workspace(self.vl, self.vl.velora_workspace_bytes(op, N, D, O, Dsub))

    def init_v(self, X, Dsub):
        N, D = X.shape
        return self.vl.velora_init_v(X, Dsub, v=self.g.vec(Dsub), ws=self.ws(self.vl.OP_INIT_V, N, D, 1, Dsub))

    def compress(self, X, v, z_dtype=torch.float32):
        N, D = X.shape
        return self.vl.velora_compress(X, v, Z=self.g.mat(N, self.vl.num_subtokens(D, v.shape[0]), z_dtype))

    def reconstruct(self, Z, v, D, x_dtype=torch.bfloat16):
        return self.vl.velora_reconstruct(Z, v, D, Xhat=self.g.mat(Z.shape[0], D, x_dtype))

    def weight_grad(self, dY, Z, v, D, mode=0, dw_dtype=None, beta=0, init=None):
        N, O = dY.shape
        op = self.vl.OP_WEIGHT_GRAD_FACTORED if mode == 0 else self.vl.OP_WEIGHT_GRAD_EXPLICIT
        dW = self.g.mat(O, D, dw_dtype or dY.dtype, init=init)
        return self.vl.velora_weight_grad(dY, Z, v, D, dW=dW, beta=beta, mode=mode, ws=self.ws(op, N, D, O, v.shape[0]))

    def forward(self, X, W, v, z_dtype=torch.float32, ws=None):
        N, D = X.shape
        O, Dsub = W.shape[0], v.shape[0]
        ws = ws if ws is not None else self.ws(self.vl.OP_LINEAR_FORWARD, N, D, O, Dsub)
        return self.vl.velora_linear_forward(X, W, v, Y=self.g.mat(N, O, X.dtype),
                                             Z=self.g.mat(N, self.vl.num_subtokens(D, Dsub), z_dtype), ws=ws)

    def backward(self, dY, W, Z, v, mode=0, ws=None, dw_dtype=None):
        N, O = dY.shape
        D, Dsub = W.shape[1], v.shape[0]
        op = self.vl.OP_LINEAR_BACKWARD_FACTORED if mode == 0 else self.vl.OP_LINEAR_BACKWARD_EXPLICIT
        ws = ws if ws is not None else self.ws(op, N, D, O, Dsub)
        return self.vl.velora_linear_backward(dY, W, Z, v, dX=self.g.mat(N, D, dY.dtype),
                                              dW=self.g.mat(O, D, dw_dtype or dY.dtype), mode=mode, ws=ws)

    def weight_grad_p(self, dY, Z, D, Dsub, P=None, beta=0):
        N, O = dY.shape
        if P is None:
            P = self.g.mat(O, self.vl.num_subtokens(D, Dsub), torch.float32)
        return self.vl.velora_weight_grad_p(dY, Z, D, Dsub, P=P, beta=beta,
                                            ws=self.ws(self.vl.OP_WEIGHT_GRAD_FACTORED, N, D, O, Dsub))

    def expand_p(self, P, v, D, dw_dtype=torch.bfloat16):
        return self.vl.velora_expand_p(P, v, D, dW=self.g.mat(P.shape[0], D, dw_dtype))


@pytest.fixture
def outs(vl, guard):
    return Outs(vl, guard)


def _distinct_D(cfg):
    seen, out = set(), []
    for i, layer in enumerate(cfg.layers):
        if layer.D not in seen:
            seen.add(layer.D)
            out.append(i)
    return out


STREAM_CASES = [(c, li, ds) for c in (2, 3, 4, 5) for li in _distinct_D(vi.CONFIGS[c]) for ds in vi.CONFIGS[c].Dsubs]


# ------------------------------------------------------------------ config 1: everything, brute force
def test_config1_fp32_every_entry_point(vl, outs):
    cfg = vi.CONFIGS[1]
    Dsub = cfg.Dsubs[0]
    Xa, Wa, dYa = vi.make_X(cfg, 0), vi.make_W(cfg, 0), vi.make_dY(cfg, 0)
    X, W, dY = Xa.torch(DEV), Wa.torch(DEV), dYa.torch(DEV)
    N, D = X.shape
    v = outs.init_v(X, Dsub)
    v_ref = oracle.init_v(Xa.f64(), Dsub)
    assert_matches(v, v_ref, 1e-5, "v", c=C_TINY)
    assert abs(float(torch.linalg.vector_norm(v.double())) - 1.0) < 1e-6
    v64 = to_f64(v)                                   # later steps use the fp32 v the GPU holds
    Z = outs.compress(X, v)
    assert_matches(Z, oracle.compress(Xa.f64(), v64), 1e-5, "Z", ulps=16, c=C_TINY)
    Xhat = outs.reconstruct(Z, v, D, x_dtype=torch.float32)
    assert_matches(Xhat, oracle.reconstruct(to_f64(Z), v64, D), 1e-6, "Xhat", ulps=2, c=C_TINY)
    dW_ref = oracle.weight_grad(dYa.f64(), to_f64(Z), v64, D)            # brute force
    for mode in (vl.WG_FACTORED, vl.WG_EXPLICIT):
        dW = outs.weight_grad(dY, Z, v, D, mode=mode)
        assert_matches(dW, dW_ref, 1e-5, "dW mode %d" % mode, c=C_TINY)
    Y, Z2 = outs.forward(X, W, v)
    assert_matches(Y, oracle.linear_forward(Xa.f64(), Wa.f64()), 1e-5, "Y", c=C_TINY)
    assert torch.equal(Z2, Z)
    dX, dW = outs.backward(dY, W, Z, v)
    assert_matches(dX, oracle.input_grad(dYa.f64(), Wa.f64()), 1e-5, "dX", c=C_TINY)
    assert_matches(dW, dW_ref, 1e-5, "dW (linear_backward)", c=C_TINY)


# ------------------------------------------------------------------ streaming kernels, full size
@pytest.mark.parametrize("c,li,Dsub", STREAM_CASES)
def test_init_v_compress_reconstruct_full_size(vl, outs, c, li, Dsub):
    cfg = vi.CONFIGS[c]
    Xa = vi.make_X(cfg, li)
    X64 = Xa.f64()
    N, D = Xa.shape
    ld = -(-D // 8) * 8                               # rows padded to 16 bytes (D = 5461 -> 5464)
    X = Xa.torch(DEV, ld=ld)
    v = outs.init_v(X, Dsub)
    v_ref, s, norm = oracle.init_v(X64, Dsub, return_sum=True)
    assert_matches(v, v_ref, TOL_Z, "v")
    v64 = to_f64(v)
    Z_ref = oracle.compress(X64, v64)
    Z = outs.compress(X, v)
    assert_matches(Z, Z_ref, TOL_Z, "Z f32")
    Zb = outs.compress(X, v, z_dtype=torch.bfloat16)
    assert_matches(Zb, Z_ref, TOL_Z, "Z bf16")
    for Zin in (Z, Zb):
        Xhat = outs.reconstruct(Zin, v, D)
        assert_matches(Xhat, oracle.reconstruct(to_f64(Zin), v64, D), TOL_Z, "Xhat")
    # properties that hold at any size: unit norm; sum of Z equals ||s||
    assert abs(float(torch.linalg.vector_norm(v.double())) - 1.0) < 1e-5
    assert abs(float(Z.double().sum()) - norm) < 1e-3 * norm + 1e-2 * np.sqrt(Z.numel())


def test_unpadded_odd_rows_take_the_elementwise_kernels(vl, guard):
    cfg = vi.CONFIGS[4]
    li = 6                                            # down projection: D = 5461, odd row pitch
    Xa = vi.make_X(cfg, li, N=512)
    X = Xa.torch(DEV)
    assert X.stride(0) == 5461
    v = vl.velora_init_v(X, 128, v=guard.vec(128))
    assert_matches(v, oracle.init_v(Xa.f64(), 128), TOL_Z, "v")
    v64 = to_f64(v)
    Z = vl.velora_compress(X, v, Z=guard.mat(512, 43, torch.float32, ld=43))         # odd pitch on Z too
    assert_matches(Z, oracle.compress(Xa.f64(), v64), TOL_Z, "Z")
    Xhat = vl.velora_reconstruct(Z, v, 5461, Xhat=guard.mat(512, 5461, ld=5461))     # dense odd rows: only row guards
    assert Xhat.stride(0) == 5461
    assert_matches(Xhat, oracle.reconstruct(to_f64(Z), v64, 5461), TOL_Z, "Xhat")
    # padded and unpadded layouts give the same numbers
    Xp = Xa.torch(DEV, ld=5464)
    Zp = vl.velora_compress(Xp, v)
    assert rel_err(to_f64(Zp), to_f64(Z)) < 1e-5


EDGE = [
    # N, D, O, Dsub
    (1, 64, 8, 64),        # one token, Dsub = D
    (3, 8, 5, 1),          # Dsub = 1: exact
    (129, 72, 24, 24),     # Dsub multiple of 8 but not a power of two
    (77, 100, 17, 16),     # ragged tail: M = 7, last sub-token has 4 entries; D not a multiple of 8
    (300, 1024, 40, 512),  # long sub-tokens (two chunks per lane)
    (130, 2048, 16, 1024), # longest supported sub-token
    (1000, 40, 33, 8),     # one chunk per sub-token
    (257, 136, 130, 10),   # Dsub not a multiple of 8
    (1000, 768, 48, 96),   # the sub-token sizes of the paper's ablation on a 768-wide layer: D/8 ...
    (1000, 768, 40, 48),   # ... D/16 ...
    (700, 768, 24, 24),    # ... D/32: none a power of two (segmented reduction, per-chunk expansion)
    (333, 1000, 56, 40),   # sub-tokens straddling the 32-chunk windows of a row, D not a multiple of Dsub
    (200, 4096, 32, 1000), # a sub-token longer than three windows; ragged last one (96 of 1000)
    (1000, 768, 40, 4),    # the paper's shortest sub-tokens: two per 16-byte chunk
    (300, 260, 24, 2),     # four per chunk; D not a multiple of 8 (last chunk half real)
    (257, 104, 16, 1),     # eight per chunk
    (500, 99, 12, 4),      # ragged last sub-token (3 of 4) inside the last chunk
    (700, 640, 300, 16),   # clustered weight gradient: three row blocks, the last one with 44 rows, 40 sub-tokens
    (300, 520, 200, 8),    # ... 65 sub-tokens: the one-CTA-per-SM shape, two Zb slabs, five 64-token blocks to split
    (1000, 1416, 130, 8),  # ... 177 sub-tokens (three slabs), a row block with two rows
]


@pytest.mark.parametrize("N,D,O,Dsub", EDGE)
@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_edge_shapes_all_entry_points(vl, outs, N, D, O, Dsub, dtype):
    case = vi.small_case(7000 + N + D, N, D, O, dtype=dtype, mean_offset=0.25)
    Xa, Wa, dYa = case["X"], case["W"], case["dY"]
    ld = -(-D // 8) * 8
    X, W, dY = Xa.torch(DEV, ld=ld), Wa.torch(DEV, ld=ld), dYa.torch(DEV, ld=-(-O // 8) * 8)
    v = outs.init_v(X, Dsub)
    assert_matches(v, oracle.init_v(Xa.f64(), Dsub), 1e-4, "v")
    v64 = to_f64(v)
    Z = outs.compress(X, v)
    Z_ref = oracle.compress(Xa.f64(), v64)
    assert_matches(Z, Z_ref, TOL_Z, "Z")
    out_dt = torch.bfloat16 if dtype == "bf16" else torch.float32
    Xhat = outs.reconstruct(Z, v, D, x_dtype=out_dt)
    assert_matches(Xhat, oracle.reconstruct(to_f64(Z), v64, D), TOL_Z, "Xhat")
    if Dsub == 1:
        assert_matches(Xhat, Xa.f64(), 1e-6, "Xhat exact for Dsub=1")
    dW_ref = oracle.weight_grad(dYa.f64(), to_f64(Z), v64, D)
    for mode in (vl.WG_FACTORED, vl.WG_EXPLICIT):
        for dw_dt in (out_dt, torch.float32):
            dW = outs.weight_grad(dY, Z, v, D, mode=mode, dw_dtype=dw_dt)
            assert_matches(dW, dW_ref, TOL_GEMM, "dW", c=C_ROUNDED)
    Y, Z2 = outs.forward(X, W, v)
    assert_matches(Y, oracle.linear_forward(Xa.f64(), Wa.f64()), TOL_GEMM, "Y")
    assert_matches(Z2, Z_ref, TOL_Z, "Z from linear_forward")
    dX, dW = outs.backward(dY, W, Z, v)
    assert_matches(dX, oracle.input_grad(dYa.f64(), Wa.f64()), TOL_GEMM, "dX")
    assert_matches(dW, dW_ref, TOL_GEMM, "dW", c=C_ROUNDED)


FUSED_EDGE = [
    # N, D, O, Dsub: outputs wide enough (>= 4 column tiles) for the forward to compute Z inside the GEMM
    (300, 320, 1100, 16),    # four sub-tokens per 64-column block
    (200, 264, 1024, 8),     # eight per block; D not a multiple of 64
    (257, 1376, 1040, 64),   # ragged last sub-token (32 of 64 columns)
    (130, 320, 1025, 256),   # sub-token spans four blocks, the last one has only one block of columns
    (513, 640, 1536, 128),   # sub-token spans two blocks
    (129, 2048, 1030, 1024), # longest sub-token
    (260, 1536, 1100, 512),  # sub-token of 64 chunks: two loads per lane complete it
    (140, 1000, 1026, 32),   # D a multiple of 8 only: the last 64-column block and the last sub-token are ragged
]


@pytest.mark.parametrize("N,D,O,Dsub", FUSED_EDGE)
@pytest.mark.parametrize("z_dtype", [torch.float32, torch.bfloat16])
def test_forward_with_compress_inside_the_gemm(vl, outs, N, D, O, Dsub, z_dtype):
    case = vi.small_case(9000 + D + Dsub, N, D, O, dtype="bf16", mean_offset=0.25)
    Xa, Wa = case["X"], case["W"]
    X, W = Xa.torch(DEV), Wa.torch(DEV)
    v = vl.velora_init_v(X, Dsub)
    v64 = to_f64(v)
    ws = outs.ws(vl.OP_LINEAR_FORWARD, N, D, O, Dsub)
    Y, Z = outs.forward(X, W, v, z_dtype=z_dtype, ws=ws)
    assert vl.velora_workspace_status(ws) == 0
    assert_matches(Y, oracle.linear_forward(Xa.f64(), Wa.f64()), TOL_GEMM, "Y")
    assert_matches(Z, oracle.compress(Xa.f64(), v64), TOL_Z, "Z")
    # the stand-alone kernel and the fused path agree to fp32 rounding
    assert rel_err(to_f64(Z), to_f64(vl.velora_compress(X, v, z_dtype=z_dtype))) < (4e-3 if z_dtype == torch.bfloat16 else 1e-5)
    assert vl.velora_device_error() == 0


ADAPTER = [
    # N, D, O, Dsub: adapter-shaped layers (output width = adapter rank): Y and Z come from one pass over X
    (12608, 768, 8, 32),     # ViT-B/16 adapter down-projection, rank 8
    (2048, 4096, 16, 64),    # LoRA A on a 4096-wide projection
    (1000, 1096, 12, 32),    # D not a multiple of 64: four two-dimensional boxes per stage instead of one
    (777, 520, 40, 8),       # eight sub-tokens per tile, ragged tokens and columns
    (300, 2048, 4, 256),     # a sub-token spans one stage of the ring
    (513, 4096, 33, 1024),   # a sub-token spans four stages; O just over one TMEM lane quarter
    (64, 64, 64, 16),        # one tile, one stage, the widest adapter
    (130, 11008, 1, 64),     # a single output column; 172 tiles of columns = 43 stages
    (500, 1024, 24, 128),    # 17..32 output columns: four-stage ring
    (1, 256, 8, 64),         # a single token
    (65, 128, 20, 32),       # one token beyond a tile
    (8192, 4096, 16, 64),    # the benchmark's adapter row at full size
    (8192, 11008, 64, 256),  # full-size down-projection input, widest adapter, sub-token = one stage
]


@pytest.mark.parametrize("N,D,O,Dsub", ADAPTER)
@pytest.mark.parametrize("z_dtype", [torch.float32, torch.bfloat16])
def test_adapter_shaped_layer_forward_and_backward(vl, outs, N, D, O, Dsub, z_dtype):
    case = vi.small_case(9500 + D + O, N, D, O, dtype="bf16", mean_offset=0.25)
    Xa, Wa, dYa = case["X"], case["W"], case["dY"]
    X, W = Xa.torch(DEV), Wa.torch(DEV)
    dY = dYa.torch(DEV, ld=-(-O // 8) * 8)
    v = vl.velora_init_v(X, Dsub)
    v64 = to_f64(v)
    ws = outs.ws(vl.OP_LINEAR_BACKWARD_FACTORED, N, D, O, Dsub)
    Y_ref, Z_ref = oracle.linear_forward(Xa.f64(), Wa.f64()), oracle.compress(Xa.f64(), v64)
    for trial in range(2):                             # the second call reuses barriers' memory and TMEM
        Y, Z = outs.forward(X, W, v, z_dtype=z_dtype, ws=ws)
        assert vl.velora_workspace_status(ws) == 0
        assert_matches(Y, Y_ref, TOL_GEMM, "Y")
        assert_matches(Z, Z_ref, TOL_Z, "Z")
    dX, dW = outs.backward(dY, W, Z, v, ws=ws)
    assert_matches(dX, oracle.input_grad(dYa.f64(), Wa.f64()), TOL_GEMM, "dX")
    dW_ref = oracle.weight_grad(dYa.f64(), to_f64(Z), v64, D, factored=True)
    assert_matches(dW, dW_ref, TOL_GEMM, "dW", c=C_ROUNDED)
    P = outs.weight_grad_p(dY, Z, D, Dsub)
    assert_matches(outs.expand_p(P, v, D), dW_ref, TOL_GEMM, "dW via P", c=C_ROUNDED)
    assert vl.velora_workspace_status(ws) == 0 and vl.velora_device_error() == 0


def test_adapter_shaped_gradient_accumulation(vl, outs):
    """beta = 1 on the adapter-shaped weight-gradient path: dW += ..., and P accumulated over two micro-batches."""
    N, D, O, Dsub = 900, 768, 24, 32
    case = vi.small_case(9700, N, D, O, dtype="bf16", mean_offset=0.25)
    X, dY = case["X"].torch(DEV), case["dY"].torch(DEV)
    v = vl.velora_init_v(X, Dsub)
    Z = vl.velora_compress(X, v)
    v64, Z64, dY64 = to_f64(v), to_f64(Z), case["dY"].f64()
    base = torch.randn(O, D, device=DEV, generator=torch.Generator(DEV).manual_seed(6))
    for dt in (torch.float32, torch.bfloat16):
        dW = outs.weight_grad(dY, Z, v, D, dw_dtype=dt, beta=1, init=base.to(dt))
        ref = oracle.weight_grad(dY64, Z64, v64, D, dW0=to_f64(base.to(dt)))
        assert_matches(dW, ref, TOL_GEMM, "dW accumulate, adapter-shaped", c=C_ROUNDED)
    cut = 333
    P = outs.weight_grad_p(dY[:cut], Z[:cut], D, Dsub)
    outs.weight_grad_p(dY[cut:], Z[cut:], D, Dsub, P=P, beta=1)
    assert_matches(outs.expand_p(P, v, D, dw_dtype=torch.float32), oracle.weight_grad(dY64, Z64, v64, D, factored=True),
                   TOL_GEMM, "dW from P over two micro-batches", c=C_ROUNDED)


def test_a_layer_replayed_from_a_cuda_graph_gives_the_same_bits(vl):
    """Forward + backward captured once (after a warm-up call) and replayed: identical results, no device error."""
    cfg = vi.CONFIGS[2]
    for li in (0, 4):                                  # q (product then compress) and up (compress inside the product)
        X, W, dY = vi.make_X(cfg, li).torch(DEV), vi.make_W(cfg, li).torch(DEV), vi.make_dY(cfg, li).torch(DEV)
        N, D = X.shape
        O = W.shape[0]
        ws = vl.velora_workspace_alloc(vl.velora_workspace_bytes(vl.OP_LINEAR_BACKWARD_FACTORED, N, D, O, 64), DEV)
        v = vl.velora_init_v(X, 64)
        out = {k: torch.empty(shape, device=DEV, dtype=dt) for k, shape, dt in
               (("Y", (N, O), torch.bfloat16), ("Z", (N, D // 64), torch.float32), ("dX", (N, D), torch.bfloat16),
                ("dW", (O, D), torch.bfloat16))}

        def layer():
            vl.velora_linear_forward(X, W, v, Y=out["Y"], Z=out["Z"], ws=ws)
            vl.velora_linear_backward(dY, W, out["Z"], v, dX=out["dX"], dW=out["dW"], ws=ws)

        layer()
        torch.cuda.synchronize()
        eager = {k: t.clone() for k, t in out.items()}
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            layer()
        torch.cuda.current_stream().wait_stream(side)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            layer()
        for t in out.values():
            t.zero_()
        g.replay()
        g.replay()
        torch.cuda.synchronize()
        for k in out:
            assert torch.equal(out[k], eager[k]), k
        assert vl.velora_workspace_status(ws) == 0 and vl.velora_device_error() == 0


def test_no_device_wait_expired_during_a_full_layer(vl):
    cfg = vi.CONFIGS[3]
    li = 0
    X, W, dY = vi.make_X(cfg, li).torch(DEV), vi.make_W(cfg, li).torch(DEV), vi.make_dY(cfg, li).torch(DEV)
    N, D = X.shape
    O = W.shape[0]
    ws = vl.velora_workspace_alloc(max(vl.velora_workspace_bytes(op, N, D, O, 32) for op in
                                       (vl.OP_INIT_V, vl.OP_LINEAR_BACKWARD_FACTORED, vl.OP_LINEAR_BACKWARD_EXPLICIT)), DEV)
    v = vl.velora_init_v(X, 32, ws=ws)
    Y, Z = vl.velora_linear_forward(X, W, v, ws=ws)
    for mode in (vl.WG_FACTORED, vl.WG_EXPLICIT):
        vl.velora_linear_backward(dY, W, Z, v, mode=mode, ws=ws)
    vl.velora_compress(X, v)
    assert vl.velora_workspace_status(ws) == 0
    assert vl.velora_device_error() == 0


def test_gradient_accumulation_beta_one(vl, outs):
    case = vi.small_case(11, 200, 256, 96, dtype="bf16")
    X, dY = case["X"].torch(DEV), case["dY"].torch(DEV)
    v = vl.velora_init_v(X, 32)
    Z = vl.velora_compress(X, v)
    v64 = to_f64(v)
    base = torch.randn(96, 256, device=DEV, generator=torch.Generator(DEV).manual_seed(5))
    for mode in (vl.WG_FACTORED, vl.WG_EXPLICIT):
        dW = outs.weight_grad(dY, Z, v, 256, mode=mode, dw_dtype=torch.float32, beta=1, init=base)
        ref = oracle.weight_grad(case["dY"].f64(), to_f64(Z), v64, 256, dW0=to_f64(base))
        assert_matches(dW, ref, TOL_GEMM, "dW accumulate", c=C_ROUNDED)


@pytest.mark.parametrize("N,D,O,Dsub,pad", [(1000, 3072, 776, 32, 0), (777, 1376, 520, 64, 0), (777, 1376, 520, 64, 2),
                                            (600, 512, 264, 8, 0)])
def test_weight_grad_takes_bf16_Z_as_stored(vl, outs, N, D, O, Dsub, pad):
    """bf16 Z: rows that TMA can address (pitch a multiple of 8) are read in place, others are repacked
    first; either way the oracle gets the very Z buffer the GPU call receives."""
    case = vi.small_case(23, N, D, O, dtype="bf16")
    X, dY = case["X"].torch(DEV), case["dY"].torch(DEV)
    v = vl.velora_init_v(X, Dsub)
    M = vl.num_subtokens(D, Dsub)
    Zbuf = torch.zeros(N, M + pad, device=DEV, dtype=torch.bfloat16)
    Z = Zbuf[:, :M]
    vl.velora_compress(X, v, Z=Z)
    dW = outs.weight_grad(dY, Z, v, D)
    ref = oracle.weight_grad(case["dY"].f64(), to_f64(Z), to_f64(v), D, factored=True)
    assert_matches(dW, ref, TOL_GEMM, "dW from bf16 Z")         # no operand is rounded on this route: C_SUM


def test_empty_batch_and_degenerate_mean(vl):
    X = torch.zeros((0, 64), dtype=torch.bfloat16, device=DEV)
    v = torch.full((16,), 7.0, device=DEV)
    Z = vl.velora_compress(X, v)
    assert Z.shape == (0, 4)
    with pytest.raises(vl.VeloraError) as e:
        vl.velora_init_v(X, 16, v=v)
    assert e.value.status == 5
    Xz = torch.zeros((10, 64), dtype=torch.bfloat16, device=DEV)
    with pytest.raises(vl.VeloraError) as e:
        vl.velora_init_v(Xz, 16, v=v)
    assert e.value.status == 5
    assert torch.all(v == 7.0)                        # v untouched
    Xc = torch.tensor([[1.0, -2.0, -1.0, 2.0]], dtype=torch.float32, device=DEV)
    with pytest.raises(vl.VeloraError):
        vl.velora_init_v(Xc, 2)
    Xn = torch.full((4, 16), float("nan"), dtype=torch.bfloat16, device=DEV)
    with pytest.raises(vl.VeloraError):
        vl.velora_init_v(Xn, 8)


def test_empty_batch_weight_gradient_is_the_empty_sum(vl, guard):
    """N = 0 on the gradient entry points: dW = beta * dW (zeros for beta = 0), dX has no rows, NULL data accepted."""
    O, D, Dsub = 24, 200, 8
    dY = torch.zeros((0, O), dtype=torch.bfloat16, device=DEV)
    Z = torch.zeros((0, 25), dtype=torch.float32, device=DEV)
    W = torch.ones((O, D), dtype=torch.bfloat16, device=DEV)
    v = torch.full((Dsub,), Dsub ** -0.5, device=DEV)
    base = torch.randn(O, D, device=DEV, generator=torch.Generator(DEV).manual_seed(3))
    for dt in (torch.bfloat16, torch.float32):
        for mode in (vl.WG_FACTORED, vl.WG_EXPLICIT):
            ws = guard.workspace(vl, 1 << 16)
            kept = guard.mat(O, D, dt, init=base.to(dt))
            vl.velora_weight_grad(dY, Z, v, D, dW=kept, beta=1, mode=mode, ws=ws)
            assert torch.equal(kept, base.to(dt))
            zeroed = guard.mat(O, D, dt, init=base.to(dt))
            vl.velora_weight_grad(dY, Z, v, D, dW=zeroed, beta=0, mode=mode, ws=ws)
            assert torch.all(zeroed == 0)
            dX, dW = vl.velora_linear_backward(dY, W, Z, v, dW=guard.mat(O, D, dt, init=base.to(dt)), mode=mode, ws=ws)
            assert dX.shape == (0, D) and torch.all(dW == 0)
    P = vl.velora_weight_grad_p(dY, Z, D, Dsub, P=guard.mat(O, 25, torch.float32, init=base[:, :25]), beta=1)
    assert torch.equal(P, base[:, :25])


def test_a_bounded_wait_that_runs_out_is_reported_and_cleared(vl, guard):
    """A tiny CTA waits, through the library's own wait routine, on barriers nobody signals: the first wait
    gives up after the 2 ms limit passed in, the second (one-second limit) is released by the abort flag.
    The kernel returns; both status readers say TIMEOUT, then OK once cleared; ordinary work is unaffected."""
    case = vi.small_case(77, 300, 512, 264, dtype="bf16", mean_offset=0.1)
    X, W, dY = case["X"].torch(DEV), case["W"].torch(DEV), case["dY"].torch(DEV)
    ws = guard.workspace(vl, vl.velora_workspace_bytes(vl.OP_LINEAR_BACKWARD_FACTORED, 300, 512, 264, 64))
    v = vl.velora_init_v(X, 64)

    def layer():
        Y, Z = vl.velora_linear_forward(X, W, v, ws=ws)
        dX, dW = vl.velora_linear_backward(dY, W, Z, v, ws=ws)
        return Y, Z, dX, dW, vl.velora_compress(X, v)

    before = layer()
    assert vl.velora_workspace_status(ws) == 0 and vl.velora_device_error() == 0
    observed = guard.vec(4, torch.int32)
    vl.velora_selftest_wait_timeout(ws, 2_000_000, observed)
    assert vl.velora_workspace_status(ws) == vl.ERR_TIMEOUT
    assert vl.velora_workspace_status(ws) == vl.ERR_TIMEOUT          # sticky until the header is cleared
    assert vl.velora_device_error() == vl.ERR_TIMEOUT
    assert vl.velora_device_error() == 0                             # that read cleared the device word
    gave_up, waited_us, released, released_us = observed.tolist()
    assert gave_up == 1 and released == 1
    assert 1_900 <= waited_us < 100_000                              # the limit passed in, not the one-second default
    assert released_us < 100_000                                     # left through the abort flag, long before its own limit
    vl.velora_workspace_init(ws)
    assert vl.velora_workspace_status(ws) == 0
    after = layer()
    for a, b in zip(before, after):
        assert torch.equal(a, b)
    assert vl.velora_workspace_status(ws) == 0 and vl.velora_device_error() == 0


def test_results_are_run_to_run_identical(vl):
    cfg = vi.CONFIGS[2]
    X, dY = vi.make_X(cfg, 6).torch(DEV), vi.make_dY(cfg, 6).torch(DEV)
    W = vi.make_W(cfg, 6).torch(DEV)
    outs = []
    for _ in range(2):
        v = vl.velora_init_v(X, 64)
        Y, Z = vl.velora_linear_forward(X, W, v)
        dX, dW = vl.velora_linear_backward(dY, W, Z, v)
        outs.append((v, Y, Z, dX, dW))
    for a, b in zip(*outs):
        assert torch.equal(a, b)
    # a frozen v survives a save / reload: Z is bit-identical
    v2 = outs[0][0].cpu().clone().to(DEV)
    assert torch.equal(vl.velora_compress(X, v2), vl.velora_compress(X, outs[0][0]))
    # the adapter-shaped kernels (sliced partial sums, compress warp sets) and the large clustered and paired ones
    for (N, D, O, Dsub) in ((8192, 4096, 16, 64), (4096, 4096, 4096, 64)):
        case = vi.small_case(41 + O, N, D, O, dtype="bf16", mean_offset=0.1)
        X, W, dY = case["X"].torch(DEV), case["W"].torch(DEV), case["dY"].torch(DEV)
        v = vl.velora_init_v(X, Dsub)
        outs = []
        for _ in range(3):
            Y, Z = vl.velora_linear_forward(X, W, v)
            dX, dW = vl.velora_linear_backward(dY, W, Z, v)
            outs.append((Y, Z, dX, dW))
        for other in outs[1:]:
            for a, b in zip(outs[0], other):
                assert torch.equal(a, b)


# ------------------------------------------------------------------ weight gradient and dense products
GEMM_CASES = [(c, li, ds) for c in (2, 3, 4, 5) for li in range(len(vi.CONFIGS[c].layers))
              for ds in vi.CONFIGS[c].Dsubs
              if vi.CONFIGS[c].layers[li].name in ("q", "up", "down", "qkv", "proj", "fc1", "fc2")]


@pytest.mark.parametrize("c,li,Dsub", GEMM_CASES)
def test_linear_forward_backward_configs(vl, outs, c, li, Dsub):
    """Full-size launches.  The oracle checks Z in full; Y and dX in full on configurations 2 and 3 and on
    a seeded sample of 192 token rows on configurations 4 and 5 (the oracle's plain loops over 8192 x 4096 x
    11008 would take minutes); dW in full where the factored oracle is cheap enough, else on 256 seeded
    output rows, and always on a few rows against the plain definition."""
    cfg = vi.CONFIGS[c]
    layer = cfg.layers[li]
    N, D, O = cfg.N, layer.D, layer.O
    Xa, Wa, dYa = vi.make_X(cfg, li), vi.make_W(cfg, li), vi.make_dY(cfg, li)
    ldD, ldO = -(-D // 8) * 8, -(-O // 8) * 8
    X, W, dY = Xa.torch(DEV, ld=ldD), Wa.torch(DEV, ld=ldD), dYa.torch(DEV, ld=ldO)
    v = outs.init_v(X, Dsub)
    v64 = to_f64(v)
    ws = outs.ws(vl.OP_LINEAR_BACKWARD_FACTORED, N, D, O, Dsub)
    Y, Z = outs.forward(X, W, v, ws=ws)
    assert_matches(Z, oracle.compress(Xa.f64(), v64), TOL_Z, "Z (fused forward)")
    W64 = Wa.f64()
    dX, dW = outs.backward(dY, W, Z, v, ws=ws)
    if c in (2, 3):
        assert_matches(Y, oracle.linear_forward(Xa.f64(), W64), TOL_GEMM, "Y")
        assert_matches(dX, oracle.input_grad(dYa.f64(), W64), TOL_GEMM, "dX")
    else:
        rows = vi.sample_rows(cfg, li, N, 192)
        assert_matches(Y[rows], oracle.linear_forward(Xa.rows(rows).f64(), W64), TOL_GEMM, "Y rows")
        assert_matches(dX[rows], oracle.input_grad(dYa.rows(rows).f64(), W64), TOL_GEMM, "dX rows")
    Z64 = to_f64(Z)
    dY64 = dYa.f64()
    M = Z.shape[1]
    if N * O * M <= 1.5e9:                              # the factored oracle over every output row
        dW_ref = oracle.weight_grad(dY64, Z64, v64, D, factored=True)
        dW_chk, sel = dW, slice(None)
    else:                                               # seeded sample of output rows
        sel = vi.sample_rows(cfg, li, O, 256, salt=2)
        dW_ref = oracle.weight_grad(np.ascontiguousarray(dY64[:, sel]), Z64, v64, D, factored=True)
        dW_chk = dW[sel]
    # Z is fp32 here and reaches the tensor cores rounded to bf16 (factored) or inside a bf16 Xhat (explicit)
    assert_matches(dW_chk, dW_ref, TOL_GEMM, "dW factored", c=C_ROUNDED)
    orows = vi.sample_rows(cfg, li, O, 48 if N * D < 5e7 else 16, salt=1)
    dW_bf = oracle.weight_grad(np.ascontiguousarray(dY64[:, orows]), Z64, v64, D)    # plain definition
    assert_matches(dW[orows], dW_bf, TOL_GEMM, "dW rows vs brute force", c=C_ROUNDED)
    dW_ex = outs.weight_grad(dY, Z, v, D, mode=vl.WG_EXPLICIT)
    assert_matches(dW_ex[sel], dW_ref, TOL_GEMM, "dW explicit", c=C_ROUNDED)
    assert rel_err(to_f64(dW_ex), to_f64(dW)) < TOL_GEMM
    assert vl.velora_workspace_status(ws) == 0 and vl.velora_device_error() == 0


@pytest.mark.parametrize("N,D,O,dtype", [(300, 320, 264, "bf16"), (1000, 1376, 520, "bf16"), (4096, 1024, 2048, "bf16"),
                                          (77, 100, 17, "bf16"), (129, 72, 24, "f32")])
def test_plain_products_of_the_uncompressed_layer(vl, guard, N, D, O, dtype):
    """velora_dense_product: Y = X W^T, dX = dY W, dW = dY^T X.  The oracle's weight gradient with sub-token
    length 1 (v = [1], Z = X) is the exact dY^T X, so all three have an oracle counterpart."""
    case = vi.small_case(31 + N, N, D, O, dtype=dtype)
    Xa, Wa, dYa = case["X"], case["W"], case["dY"]
    ldD, ldO = -(-D // 8) * 8, -(-O // 8) * 8
    X, W, dY = Xa.torch(DEV, ld=ldD), Wa.torch(DEV, ld=ldD), dYa.torch(DEV, ld=ldO)
    dt = X.dtype
    ws = guard.workspace(vl, 256)
    Y = vl.velora_dense_product(vl.PRODUCT_A_BT, X, W, C=guard.mat(N, O, dt), ws=ws)
    assert_matches(Y, oracle.linear_forward(Xa.f64(), Wa.f64()), TOL_GEMM, "Y")
    dX = vl.velora_dense_product(vl.PRODUCT_A_B, dY, W, C=guard.mat(N, D, dt), ws=ws)
    assert_matches(dX, oracle.input_grad(dYa.f64(), Wa.f64()), TOL_GEMM, "dX")
    dW_ref = oracle.weight_grad(dYa.f64(), Xa.f64(), np.ones(1), D)
    for cdt in (dt, torch.float32):
        dW = vl.velora_dense_product(vl.PRODUCT_AT_B, dY, X, C=guard.mat(O, D, cdt), ws=ws)
        assert_matches(dW, dW_ref, TOL_GEMM, "dW = dY^T X")
    base = torch.randn(O, D, device=DEV, generator=torch.Generator(DEV).manual_seed(9))
    acc = vl.velora_dense_product(vl.PRODUCT_AT_B, dY, X, C=guard.mat(O, D, torch.float32, init=base), beta=1, ws=ws)
    assert_matches(acc, oracle.weight_grad(dYa.f64(), Xa.f64(), np.ones(1), D, dW0=to_f64(base)), TOL_GEMM, "dW += dY^T X")
    assert vl.velora_workspace_status(ws) == 0


# ------------------------------------------------------------------ Z stored in 8 bits (E4M3)
def _e4m3_decode_table():
    """Value of every E4M3 byte, from the format's definition (bias 7, 3 mantissa bits, E = 0 subnormal,
    0x7F / 0xFF NaN)."""
    t = np.empty(256)
    for code in range(256):
        s, E, m = code >> 7, (code >> 3) & 15, code & 7
        mag = np.nan if (E == 15 and m == 7) else ((m / 8.0) * 2.0 ** -6 if E == 0 else (1.0 + m / 8.0) * 2.0 ** (E - 7))
        t[code] = -mag if s else mag
    return t


E4M3 = _e4m3_decode_table()


def _check_codes(Z8: torch.Tensor, z_over_scale64: np.ndarray, what: str):
    """Stored bytes against the oracle's rounding of the exact scalars.  The kernel takes the rounding decision
    on its fp32 value (relative error about 1e-6), the oracle on the exact one: they may differ where the exact
    value sits within that error of a rounding boundary, i.e. for about 2 * 1e-6 / 2^-4 = 3e-5 of the
    elements (bound used: 2e-4), and then only by one step of the format."""
    got = E4M3[Z8.cpu().numpy().astype(np.uint8)]
    assert not np.isnan(got).any(), what + ": NaN code stored"
    ref = oracle.round_to_fp8_e4m3(z_over_scale64)
    diff = got != ref
    assert diff.mean() <= 2e-4, "%s: %.2e of the codes differ" % (what, diff.mean())
    _, e = np.frexp(ref[diff])
    step = np.ldexp(1.0, np.maximum(e, -5) - 4)
    assert np.all(np.abs(got[diff] - ref[diff]) <= 2 * step), what + ": a code is off by more than one step"
    return got


@pytest.mark.parametrize("c,li,N", [(2, 6, None), (3, 3, None), (5, 0, None), (4, 6, 1024)])
def test_z_stored_in_8_bits_full_layers(vl, outs, guard, c, li, N):
    """E4M3 storage of Z through every entry point that writes or reads Z, on full-size layers (ragged last
    sub-token, outlier channels, heavy-tailed scales, padded odd rows)."""
    cfg = vi.CONFIGS[c]
    layer = cfg.layers[li]
    Dsub = cfg.Dsubs[0]
    D, O = layer.D, layer.O
    Xa, Wa, dYa = vi.make_X(cfg, li, N=N), vi.make_W(cfg, li), vi.make_dY(cfg, li, N=N)
    N = Xa.shape[0]
    ldD, ldO = -(-D // 8) * 8, -(-O // 8) * 8
    X, W, dY = Xa.torch(DEV, ld=ldD), Wa.torch(DEV, ld=ldD), dYa.torch(DEV, ld=ldO)
    X64, dY64 = Xa.f64(), dYa.f64()
    v = outs.init_v(X, Dsub)
    v64 = to_f64(v)
    # the scale and the two scaled vectors
    zscale, v_store, v_load = vl.velora_z8_calibrate(X, v, headroom=2.0,
                                                     ws=outs.ws(vl.OP_Z8_CALIBRATE, N, D, 0, Dsub))
    Z_exact = oracle.compress(X64, v64)
    scale_ref = oracle.zscale_from_batch(Z_exact, 2.0)
    scale = float(zscale.item())
    assert abs(scale / scale_ref - 1.0) < 1e-5                     # the maximum of fp32 dot products, fp32 arithmetic
    assert rel_err(to_f64(v_store), v64 / scale) < 1e-6 and rel_err(to_f64(v_load), v64 * scale) < 1e-6
    vs64, vl64 = to_f64(v_store), to_f64(v_load)
    # writers: the compress kernel and the forward product with compress inside
    Z8 = outs.compress(X, v_store, z_dtype=torch.uint8)
    q = _check_codes(Z8, oracle.compress(X64, vs64), "compress")
    assert np.abs(q).max() <= 240.0                                 # headroom 2: the batch's maximum sits at 224
    ws = outs.ws(vl.OP_LINEAR_BACKWARD_FACTORED, N, D, O, Dsub)
    Y, Z8f = outs.forward(X, W, v_store, z_dtype=torch.uint8, ws=ws)
    _check_codes(Z8f, oracle.compress(X64, vs64), "linear_forward")
    rows = vi.sample_rows(cfg, li, N, 128)
    assert_matches(Y[rows], oracle.linear_forward(Xa.rows(rows).f64(), Wa.f64()), TOL_GEMM, "Y rows")
    # readers, each on the very bytes it is given
    Xhat = outs.reconstruct(Z8, v_load, D)
    assert_matches(Xhat, oracle.reconstruct(q, vl64, D), TOL_Z, "Xhat from 8-bit Z")
    if N * O * q.shape[1] <= 1.5e9:
        sel = slice(None)
        dW_ref = oracle.weight_grad(dY64, q, vl64, D, factored=True)
    else:
        sel = vi.sample_rows(cfg, li, O, 256, salt=4)
        dW_ref = oracle.weight_grad(np.ascontiguousarray(dY64[:, sel]), q, vl64, D, factored=True)
    dX, dW = outs.backward(dY, W, Z8, v_load, ws=ws)
    assert_matches(dW[sel], dW_ref, TOL_GEMM, "dW factored from 8-bit Z")            # decoded values are exact bf16 operands: C_SUM
    assert_matches(dX[rows], oracle.input_grad(dYa.rows(rows).f64(), Wa.f64()), TOL_GEMM, "dX rows")
    dW_ex = outs.weight_grad(dY, Z8, v_load, D, mode=vl.WG_EXPLICIT)
    assert_matches(dW_ex[sel], dW_ref, TOL_GEMM, "dW explicit from 8-bit Z", c=C_ROUNDED)
    P = outs.weight_grad_p(dY, Z8, D, Dsub)
    assert_matches(outs.expand_p(P, v_load, D)[sel], dW_ref, TOL_GEMM, "dW via P from 8-bit Z")
    # what the 8-bit store costs: every scalar is within 2^-4 of its exact value (relative), so is the gradient
    dW_exact = oracle.weight_grad(np.ascontiguousarray(dY64[:, sel]) if not isinstance(sel, slice) else dY64, Z_exact, v64, D, factored=True)
    assert rel_err(dW_ref, dW_exact) < 2.0 ** -4
    # a later batch four times as large saturates at +-448 and stores no NaN
    Xbig = (X.float() * 4.0).to(torch.bfloat16)
    Zsat = E4M3[vl.velora_compress(Xbig, v_store, z_dtype=torch.uint8).cpu().numpy()]
    assert not np.isnan(Zsat).any() and np.abs(Zsat).max() == 448.0
    assert vl.velora_workspace_status(ws) == 0 and vl.velora_device_error() == 0


@pytest.mark.parametrize("N,D,O,Dsub,dtype", [(77, 100, 17, 16, "bf16"), (257, 136, 130, 10, "f32"), (300, 1024, 40, 512, "bf16"),
                                               (1000, 768, 40, 48, "bf16"), (500, 99, 12, 4, "bf16"), (2048, 4096, 16, 64, "bf16"),
                                               (3, 8, 5, 1, "f32")])
def test_z_stored_in_8_bits_edge_shapes(vl, outs, N, D, O, Dsub, dtype):
    """The shapes that leave the fast kernels (element-wise kernels, adapter-shaped layers, fp32 data)."""
    case = vi.small_case(8100 + N + D, N, D, O, dtype=dtype, mean_offset=0.25)
    Xa, Wa, dYa = case["X"], case["W"], case["dY"]
    ld = -(-D // 8) * 8
    X, W, dY = Xa.torch(DEV, ld=ld), Wa.torch(DEV, ld=ld), dYa.torch(DEV, ld=-(-O // 8) * 8)
    out_dt = torch.bfloat16 if dtype == "bf16" else torch.float32
    v = outs.init_v(X, Dsub)
    zscale, v_store, v_load = vl.velora_z8_calibrate(X, v, headroom=1.5, ws=outs.ws(vl.OP_Z8_CALIBRATE, N, D, 0, Dsub))
    vs64, vl64 = to_f64(v_store), to_f64(v_load)
    Z8 = outs.compress(X, v_store, z_dtype=torch.uint8)
    q = _check_codes(Z8, oracle.compress(Xa.f64(), vs64), "compress")
    Y, Z8f = outs.forward(X, W, v_store, z_dtype=torch.uint8)
    _check_codes(Z8f, oracle.compress(Xa.f64(), vs64), "linear_forward")
    assert_matches(Y, oracle.linear_forward(Xa.f64(), Wa.f64()), TOL_GEMM, "Y")
    Xhat = outs.reconstruct(Z8, v_load, D, x_dtype=out_dt)
    assert_matches(Xhat, oracle.reconstruct(q, vl64, D), TOL_Z, "Xhat")
    dW_ref = oracle.weight_grad(dYa.f64(), q, vl64, D)                               # plain definition
    for mode in (vl.WG_FACTORED, vl.WG_EXPLICIT):
        dW = outs.weight_grad(dY, Z8, v_load, D, mode=mode, dw_dtype=out_dt)
        assert_matches(dW, dW_ref, TOL_GEMM, "dW mode %d" % mode, c=C_ROUNDED if mode == vl.WG_EXPLICIT else C_SUM)
    dX, dW = outs.backward(dY, W, Z8, v_load)
    assert_matches(dW, dW_ref, TOL_GEMM, "dW (linear_backward)")
    assert_matches(dX, oracle.input_grad(dYa.f64(), Wa.f64()), TOL_GEMM, "dX")


def test_z8_calibrate_degenerate_batches(vl, guard):
    v = torch.full((16,), 0.25, device=DEV)
    for X in (torch.zeros((10, 64), dtype=torch.bfloat16, device=DEV), torch.zeros((0, 64), dtype=torch.bfloat16, device=DEV),
              torch.full((4, 64), float("nan"), dtype=torch.bfloat16, device=DEV)):
        zscale, v_store, v_load = vl.velora_z8_calibrate(X, v)
        assert float(zscale.item()) == 1.0 and torch.equal(v_store, v) and torch.equal(v_load, v)


# ------------------------------------------------------------------ factored form kept factored; sharded batches
@pytest.mark.parametrize("c,li,Dsub", [(2, 6, 64), (3, 0, 32), (4, 0, 128), (5, 0, 64)])
def test_factor_p_accumulates_over_micro_batches_and_expands_once(vl, outs, c, li, Dsub):
    cfg = vi.CONFIGS[c]
    Xa, dYa = vi.make_X(cfg, li), vi.make_dY(cfg, li)
    N, D = Xa.shape
    O = dYa.shape[1]
    ldO = -(-O // 8) * 8
    X, dY = Xa.torch(DEV, ld=-(-D // 8) * 8), dYa.torch(DEV, ld=ldO)
    v = vl.velora_init_v(X, Dsub)
    v64 = to_f64(v)
    Z = vl.velora_compress(X, v)
    Z64, dY64 = to_f64(Z), dYa.f64()
    cut = (N // 3 // 64) * 64 + 17                       # two uneven micro-batches
    P = outs.weight_grad_p(dY[:cut], Z[:cut], D, Dsub)
    outs.weight_grad_p(dY[cut:], Z[cut:], D, Dsub, P=P, beta=1)
    sel = vi.sample_rows(cfg, li, O, 256, salt=3)
    dW_ref, P_ref = oracle.weight_grad(np.ascontiguousarray(dY64[:, sel]), Z64, v64, D, factored=True, return_P=True)
    assert_matches(P[sel], P_ref, TOL_GEMM, "P over two micro-batches", c=C_ROUNDED)
    dW = outs.expand_p(P, v, D)
    dW_one = outs.weight_grad(dY, Z, v, D)
    assert rel_err(to_f64(dW), to_f64(dW_one)) < TOL_GEMM
    assert_matches(dW[sel], dW_ref, TOL_GEMM, "dW expanded from P", c=C_ROUNDED)


def test_gradient_step_straight_from_the_factor(vl, outs, guard):
    """W <- W - lr * (P (x) v) through velora_expand_p (beta = 1, v scaled by -lr): no dW buffer."""
    case = vi.small_case(29, 600, 512, 264, dtype="bf16")
    X, dY = case["X"].torch(DEV), case["dY"].torch(DEV)
    W = guard.mat(264, 512, torch.float32, init=case["W"].torch(DEV).float())   # fp32 master weights
    Dsub, lr = 32, 0.125
    v = vl.velora_init_v(X, Dsub)
    Z = vl.velora_compress(X, v)
    P = outs.weight_grad_p(dY, Z, 512, Dsub)
    W_ref = case["W"].f64() - lr * oracle.weight_grad(case["dY"].f64(), to_f64(Z), to_f64(v), 512, factored=True)
    vl.velora_expand_p(P, v * (-lr), 512, dW=W, beta=1)
    assert_matches(W, W_ref, TOL_GEMM, "W after the step", c=C_ROUNDED)     # the update dominates W here
    assert rel_err(to_f64(W) - case["W"].f64(), W_ref - case["W"].f64()) < TOL_GEMM


def test_token_sharded_init_v_gives_every_shard_the_same_v(vl, guard):
    cfg = vi.CONFIGS[2]
    Xa = vi.make_X(cfg, 6)
    X = Xa.torch(DEV)
    N = X.shape[0]
    shards = [X[: N // 3], X[N // 3: N // 3 + 5], X[N // 3 + 5:], X[:0]]      # uneven, one empty
    s = sum(vl.velora_subtoken_sum(x, 64, s=guard.vec(64)) for x in shards)    # what the all-reduce computes
    v = vl.velora_normalize_v(s, v=guard.vec(64))
    v_ref, s_ref, _ = oracle.init_v(Xa.f64(), 64, return_sum=True)
    assert_matches(s, s_ref, 1e-4, "s")
    assert_matches(v, v_ref, 1e-4, "v")
    assert rel_err(to_f64(v), to_f64(vl.velora_init_v(X, 64))) < 1e-5
    with pytest.raises(vl.VeloraError):
        vl.velora_normalize_v(torch.zeros(64, device=DEV))


@pytest.mark.parametrize("N,D,Dsub,dtype", [(8192, 4096, 64, "bf16"), (777, 1376, 64, "bf16"), (300, 200, 24, "f32"),
                                             (1000, 768, 32, "bf16")])
def test_running_average_v_follows_the_oracle_over_several_batches(vl, guard, N, D, Dsub, dtype):
    """velora_update_v (running-average initialisation): three batches with rho = 1, 1/2, 0.3."""
    a = guard.vec(Dsub).zero_()
    v = guard.vec(Dsub).zero_()
    ws = guard.workspace(vl, vl.velora_workspace_bytes(vl.OP_UPDATE_V, N, D, 1, Dsub))
    a_ref = None
    for t, rho in enumerate((1.0, 0.5, 0.3)):
        X = vi.small_case(50 + t, N, D, 8, dtype=dtype, mean_offset=0.05 * (t + 1))["X"]
        vl.velora_update_v(X.torch(DEV), Dsub, rho, a, v, ws=ws)
        a_ref, v_ref = oracle.update_v(X.f64(), Dsub, rho, a_ref)
        assert_matches(a, a_ref, 1e-5, "a")
        assert_matches(v, v_ref, 1e-5, "v")
        a_ref = to_f64(a)                              # the state the next GPU call reads is the stored fp32 one
    assert vl.velora_workspace_status(ws) == 0
    # rho = 1 is init_v of the batch
    X = vi.small_case(60, N, D, 8, dtype=dtype, mean_offset=0.1)["X"].torch(DEV)
    vl.velora_update_v(X, Dsub, 1.0, a, v, ws=ws)
    assert rel_err(to_f64(v), to_f64(vl.velora_init_v(X, Dsub))) < 1e-5
    # a zero batch at rho = 1 has no direction: state kept, sticky status raised, no exception, no sync
    before = v.clone()
    vl.velora_update_v(torch.zeros_like(X), Dsub, 1.0, a, v, ws=ws)
    assert vl.velora_workspace_status(ws) == vl.ERR_DEGENERATE_V
    assert torch.equal(v, before)
    vl.velora_workspace_init(ws)
    assert vl.velora_workspace_status(ws) == 0


def test_chained_path_against_chained_oracle(vl, outs):
    """init_v -> compress -> weight_grad on the GPU against the same chain in fp64 (bf16 Z storage)."""
    cfg = vi.CONFIGS[3]
    li = 3
    Xa, dYa = vi.make_X(cfg, li), vi.make_dY(cfg, li)
    X, dY = Xa.torch(DEV), dYa.torch(DEV)
    D = Xa.shape[1]
    v = outs.init_v(X, 32)
    Z = outs.compress(X, v, z_dtype=torch.bfloat16)
    dW = outs.weight_grad(dY, Z, v, D)
    v_ref = oracle.init_v(Xa.f64(), 32)
    dW_ref = oracle.weight_grad(dYa.f64(), oracle.compress(Xa.f64(), v_ref), v_ref, D, factored=True)
    assert rel_err(to_f64(dW), dW_ref) < TOL_GEMM
