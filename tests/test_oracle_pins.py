"""Pins of the fp64 CPU oracle against what the paper and the mathematics fix.

The paper (arxiv 2405.17991) prints no worked numerical example for the
projection, so the oracle is pinned by closed forms, invariants of an
orthogonal rank-1 projection, special cases that reduce to numpy routines,
and brute force on small inputs.  Each test names the passage it follows.
None of these tests touches the CUDA library.
"""
import numpy as np
import pytest

import oracle
import velora_inputs as vi

RTOL = 1e-12


def _rel(a, b):
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    den = np.linalg.norm(b)
    return np.linalg.norm(a - b) / (den if den > 0 else 1.0)


def _case(seed, N, D, O, offset=0.0):
    rng = np.random.default_rng(seed)
    X = rng.standard_normal((N, D)) * np.exp(0.5 * rng.standard_normal(D))[None, :] + offset
    W = rng.standard_normal((O, D)) / np.sqrt(D)
    dY = rng.standard_normal((N, O))
    return X, W, dY


def _pad(X, Dsub):
    N, D = X.shape
    M = -(-D // Dsub)
    Xp = np.zeros((N, M * Dsub))
    Xp[:, :D] = X
    return Xp, M


SHAPES = [(256, 64, 16), (37, 96, 32), (50, 88, 16), (19, 70, 64), (8, 5, 5), (11, 7, 3)]


# --- S1: initialisation of v (Section 3.2 "Cheap initialisation strategies"; Section 3.1 unit length) ---

@pytest.mark.parametrize("N,D,Dsub", SHAPES)
def test_v_has_unit_norm_and_is_the_normalised_subtoken_mean(N, D, Dsub):
    X, _, _ = _case(1, N, D, 4, offset=0.3)
    v, s, norm = oracle.init_v(X, Dsub, return_sum=True)
    assert abs(np.linalg.norm(v) - 1.0) < RTOL
    Xp, M = _pad(X, Dsub)
    mean = Xp.reshape(N * M, Dsub).mean(axis=0)            # numpy's own reduction
    assert _rel(v, mean / np.linalg.norm(mean)) < 1e-11
    assert _rel(s, mean * N * M) < 1e-11
    assert abs(norm - np.linalg.norm(s)) <= RTOL * norm


def test_constant_input_closed_form():
    # X == c: every sub-token is c*ones, so v = sign(c)/sqrt(Dsub), Z = |c| sqrt(Dsub), Xhat = X.
    for c in (2.5, -0.75):
        N, D, Dsub, O = 12, 48, 16, 5
        X = np.full((N, D), c)
        v = oracle.init_v(X, Dsub)
        np.testing.assert_allclose(v, np.sign(c) / np.sqrt(Dsub) * np.ones(Dsub), rtol=RTOL)
        Z = oracle.compress(X, v)
        np.testing.assert_allclose(Z, abs(c) * np.sqrt(Dsub) * np.ones((N, D // Dsub)), rtol=RTOL)
        np.testing.assert_allclose(oracle.reconstruct(Z, v, D), X, rtol=RTOL)
        dY = np.random.default_rng(3).standard_normal((N, O))
        dW = oracle.weight_grad(dY, Z, v, D)
        np.testing.assert_allclose(dW, c * dY.sum(axis=0)[:, None] * np.ones((O, D)), rtol=1e-11, atol=1e-13)


def test_degenerate_mean_is_reported_not_papered_over():
    X = np.zeros((4, 8))
    with pytest.raises(oracle.OracleError) as e:
        oracle.init_v(X, 4)
    assert e.value.code == oracle.DEGENERATE_V
    X = np.array([[1.0, -2.0, -1.0, 2.0]])                  # sub-tokens cancel exactly
    with pytest.raises(oracle.OracleError):
        oracle.init_v(X, 2)


@pytest.mark.parametrize("N,D,Dsub", SHAPES)
def test_sum_of_stored_scalars_equals_norm_of_subtoken_sum(N, D, Dsub):
    # With the mean initialisation, sum_{n,m} Z = <s, v> = ||s||.
    X, _, _ = _case(2, N, D, 4, offset=0.2)
    v, s, norm = oracle.init_v(X, Dsub, return_sum=True)
    Z = oracle.compress(X, v)
    assert abs(Z.sum() - norm) <= 1e-11 * norm


# --- S3/S4: compress and reconstruct (Section 3.1, Eq. 1, Eq. 2, proj_v) ---

@pytest.mark.parametrize("N,D,Dsub", SHAPES)
def test_compress_is_a_matrix_vector_product_of_the_grouped_input(N, D, Dsub):
    X, _, _ = _case(4, N, D, 4)
    v = oracle.init_v(X + 0.1, Dsub)
    Xp, M = _pad(X, Dsub)
    Z_np = (Xp.reshape(N * M, Dsub) @ v).reshape(N, M)      # group() then z . v by numpy
    assert _rel(oracle.compress(X, v), Z_np) < RTOL


@pytest.mark.parametrize("N,D,Dsub", SHAPES)
def test_reconstruct_is_an_outer_product_per_subtoken(N, D, Dsub):
    rng = np.random.default_rng(5)
    M = -(-D // Dsub)
    Z = rng.standard_normal((N, M))
    v = rng.standard_normal(Dsub)
    v /= np.linalg.norm(v)
    Xhat_np = np.einsum("nm,j->nmj", Z, v).reshape(N, M * Dsub)[:, :D]   # z_p . v^T then ungroup()
    assert _rel(oracle.reconstruct(Z, v, D), Xhat_np) < RTOL


@pytest.mark.parametrize("N,D,Dsub", SHAPES)
def test_residual_is_orthogonal_to_v_and_pythagoras_holds(N, D, Dsub):
    X, _, _ = _case(6, N, D, 4, offset=0.1)
    v = oracle.init_v(X, Dsub)
    Z = oracle.compress(X, v)
    Xhat = oracle.reconstruct(Z, v, D)
    Xp, M = _pad(X, Dsub)
    # The truncated tail of Xhat is compared on the zero-extended width, where the projection lives.
    Xhat_p = np.einsum("nm,j->nmj", Z, v).reshape(N, M * Dsub)
    assert _rel(Xhat_p[:, :D], Xhat) < RTOL
    x = Xp.reshape(N * M, Dsub)
    xh = Xhat_p.reshape(N * M, Dsub)
    r = x - xh
    scale = np.linalg.norm(x, axis=1) + 1e-300
    assert np.max(np.abs(r @ v) / scale) < 1e-13
    nx, nh, nr = (np.sum(a * a, axis=1) for a in (x, xh, r))
    assert np.max(np.abs(nx - nh - nr) / (nx + 1e-300)) < 1e-12
    assert np.all(nr <= nx * (1 + 1e-12)) and np.all(nh <= nx * (1 + 1e-12))
    # energy: sum Z^2 = ||Xhat_p||_F^2 <= ||X||_F^2
    assert abs((Z * Z).sum() - (xh * xh).sum()) <= 1e-12 * (Z * Z).sum()
    assert (Z * Z).sum() <= (X * X).sum() * (1 + 1e-12)


def test_exact_when_subtokens_are_multiples_of_v():
    rng = np.random.default_rng(7)
    N, D, Dsub = 9, 40, 8
    v = rng.standard_normal(Dsub)
    v /= np.linalg.norm(v)
    coef = rng.standard_normal((N, D // Dsub))
    X = np.einsum("nm,j->nmj", coef, v).reshape(N, D)
    Z = oracle.compress(X, v)
    np.testing.assert_allclose(Z, coef, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(oracle.reconstruct(Z, v, D), X, rtol=1e-12, atol=1e-14)


def test_exact_when_subtoken_length_is_one():
    X, _, _ = _case(8, 13, 10, 3, offset=0.4)
    v = oracle.init_v(X, 1)
    assert v.shape == (1,) and abs(abs(v[0]) - 1.0) < RTOL
    Z = oracle.compress(X, v)
    np.testing.assert_allclose(Z, v[0] * X, rtol=RTOL)
    np.testing.assert_allclose(oracle.reconstruct(Z, v, 10), X, rtol=RTOL)


@pytest.mark.parametrize("N,D,Dsub", SHAPES)
def test_projection_is_idempotent(N, D, Dsub):
    X, _, _ = _case(9, N, D, 4, offset=0.1)
    v = oracle.init_v(X, Dsub)
    Z = oracle.compress(X, v)
    Xp, M = _pad(X, Dsub)
    Xhat_p = np.einsum("nm,j->nmj", Z, v).reshape(N, M * Dsub)
    assert _rel(oracle.compress(Xhat_p, v), Z) < 1e-12          # compress(reconstruct(Z)) = Z on the padded width
    if D % Dsub == 0:
        Xhat = oracle.reconstruct(Z, v, D)
        assert _rel(oracle.reconstruct(oracle.compress(Xhat, v), v, D), Xhat) < 1e-12


def test_linearity_and_sign_flip():
    N, D, Dsub, O = 21, 72, 24, 6
    Xa, _, dYa = _case(10, N, D, O)
    Xb, _, dYb = _case(11, N, D, O)
    v = oracle.init_v(Xa + 0.2, Dsub)
    a, b = 0.7, -1.9
    Za, Zb = oracle.compress(Xa, v), oracle.compress(Xb, v)
    assert _rel(oracle.compress(a * Xa + b * Xb, v), a * Za + b * Zb) < 1e-12
    assert _rel(oracle.reconstruct(a * Za + b * Zb, v, D),
                a * oracle.reconstruct(Za, v, D) + b * oracle.reconstruct(Zb, v, D)) < 1e-12
    for fact in (False, True):
        g = lambda dY, Z: oracle.weight_grad(dY, Z, v, D, factored=fact)
        assert _rel(g(a * dYa + b * dYb, Za), a * g(dYa, Za) + b * g(dYb, Za)) < 1e-12
        assert _rel(g(dYa, a * Za + b * Zb), a * g(dYa, Za) + b * g(dYa, Zb)) < 1e-12
    # v -> -v: Z flips sign, Xhat and dW do not care.
    Zm = oracle.compress(Xa, -v)
    assert _rel(Zm, -Za) < RTOL
    assert _rel(oracle.reconstruct(Zm, -v, D), oracle.reconstruct(Za, v, D)) < RTOL
    assert _rel(oracle.weight_grad(dYa, Zm, -v, D), oracle.weight_grad(dYa, Za, v, D)) < RTOL


# --- S5: weight gradient (Algorithm 1 backward; Section 3.2 rank-1 update) ---

@pytest.mark.parametrize("N,D,Dsub,O", [(256, 64, 16, 64), (33, 40, 16, 7), (17, 24, 24, 5), (20, 9, 1, 4),
                                         (15, 50, 32, 9)])
def test_bruteforce_equals_factored_equals_numpy(N, D, Dsub, O):
    X, _, dY = _case(12, N, D, O, offset=0.1)
    v = oracle.init_v(X, Dsub)
    Z = oracle.compress(X, v)
    dW_bf = oracle.weight_grad(dY, Z, v, D)
    dW_fa, P = oracle.weight_grad(dY, Z, v, D, factored=True, return_P=True)
    assert _rel(dW_fa, dW_bf) < 1e-12
    assert _rel(P, dY.T @ Z) < 1e-12
    Xhat = oracle.reconstruct(Z, v, D)
    assert _rel(dW_bf, dY.T @ Xhat) < 1e-12                   # the definition through numpy's matmul


@pytest.mark.parametrize("N,D,Dsub,O", [(64, 48, 16, 10), (31, 32, 32, 6), (40, 56, 8, 3)])
def test_closed_form_exact_gradient_times_block_projector(N, D, Dsub, O):
    # dW_VeLoRA = (dY^T X) (I_M (x) v v^T); for Dsub = D this is the printed g v v^T.
    X, _, dY = _case(13, N, D, O, offset=0.2)
    v = oracle.init_v(X, Dsub)
    M = D // Dsub
    g_exact = dY.T @ X                                           # textbook gradient, numpy
    proj = np.kron(np.eye(M), np.outer(v, v))
    dW = oracle.weight_grad(dY, oracle.compress(X, v), v, D)
    assert _rel(dW, g_exact @ proj) < 1e-12


def test_closed_form_with_a_ragged_last_subtoken():
    N, D, Dsub, O = 25, 44, 16, 5                                # M = 3, last sub-token has 12 entries
    X, _, dY = _case(14, N, D, O, offset=0.2)
    v = oracle.init_v(X, Dsub)
    Xp, M = _pad(X, Dsub)
    proj = np.kron(np.eye(M), np.outer(v, v))
    expect = ((dY.T @ Xp) @ proj)[:, :D]
    assert _rel(oracle.weight_grad(dY, oracle.compress(X, v), v, D), expect) < 1e-12
    assert _rel(oracle.weight_grad(dY, oracle.compress(X, v), v, D, factored=True), expect) < 1e-12


def test_gradient_accumulation_adds_to_the_existing_buffer():
    N, D, Dsub, O = 12, 32, 8, 4
    X, _, dY = _case(15, N, D, O, offset=0.1)
    v = oracle.init_v(X, Dsub)
    Z = oracle.compress(X, v)
    dW0 = np.random.default_rng(16).standard_normal((O, D))
    for fact in (False, True):
        assert _rel(oracle.weight_grad(dY, Z, v, D, dW0=dW0, factored=fact),
                    dW0 + oracle.weight_grad(dY, Z, v, D)) < 1e-12


# --- S2/S6: the dense products (Algorithm 1: out, grad_input) ---

@pytest.mark.parametrize("N,D,O", [(256, 64, 64), (19, 33, 7), (5, 128, 3)])
def test_dense_products_match_numpy(N, D, O):
    X, W, dY = _case(17, N, D, O)
    assert _rel(oracle.linear_forward(X, W), X @ W.T) < 1e-12
    assert _rel(oracle.input_grad(dY, W), dY @ W) < 1e-12


def test_listing_shapes_are_mutually_consistent():
    # out [N,O], grad_input [N,D], grad_weight [O,D]: only W[O,D] used as X W^T fits all three lines.
    X, W, dY = _case(18, 6, 10, 4)
    v = oracle.init_v(X + 0.1, 5)
    assert oracle.linear_forward(X, W).shape == (6, 4)
    assert oracle.input_grad(dY, W).shape == (6, 10)
    assert oracle.weight_grad(dY, oracle.compress(X, v), v, 10).shape == W.shape


# --- planted mistakes: each plausible slip must be caught by a pin above ---

def test_pins_detect_planted_mistakes():
    N, D, Dsub, O = 20, 48, 16, 6
    X, _, dY = _case(19, N, D, O, offset=0.2)
    v = oracle.init_v(X, Dsub)
    Z = oracle.compress(X, v)
    M = D // Dsub
    g_exact = dY.T @ X
    good = g_exact @ np.kron(np.eye(M), np.outer(v, v))
    # transposed operand / wrong index order in the expansion
    bad_transposed = np.einsum("om,j->ojm", dY.T @ Z, v).reshape(O, D)
    # un-normalised v (dropped normalisation)
    s = X.reshape(N * M, Dsub).sum(axis=0)
    bad_unnorm = oracle.weight_grad(dY, oracle.compress(X, s), s, D)
    # per-position mean instead of a shared v would change Z
    for bad in (bad_transposed, bad_unnorm):
        assert _rel(bad, good) > 1e-3
    assert _rel(oracle.weight_grad(dY, Z, v, D), good) < 1e-12


# --- running-average variant of the initialisation (Section 5, ablation on the initialisation strategy) ---

def test_running_average_with_rho_one_is_the_fixed_average_of_that_batch():
    X, _, _ = _case(31, 40, 72, 3, offset=0.3)
    for Dsub in (8, 16, 24):                       # 16 leaves a ragged last sub-token (72 = 4 * 16 + 8)
        a, v = oracle.update_v(X, Dsub, 1.0)
        assert _rel(v, oracle.init_v(X, Dsub)) < 1e-12
        Xp, M = _pad(X, Dsub)
        assert _rel(a, Xp.reshape(-1, Dsub).mean(axis=0)) < 1e-12
        assert abs(np.linalg.norm(v) - 1.0) < 1e-12


def test_running_average_with_rho_one_over_t_is_the_fixed_average_of_all_batches_seen():
    N, D, Dsub, T = 24, 64, 16, 5
    batches = [_case(40 + t, N, D, 2, offset=0.1 * t)[0] for t in range(T)]
    a = None
    for t, X in enumerate(batches, start=1):
        a, v = oracle.update_v(X, Dsub, 1.0 / t, a)
        assert _rel(v, oracle.init_v(np.concatenate(batches[:t], axis=0), Dsub)) < 1e-12


def test_running_average_fixed_points_and_mixing():
    X, _, _ = _case(33, 30, 48, 2, offset=0.5)
    Dsub = 16
    mean, v_mean = oracle.update_v(X, Dsub, 1.0)
    # rho = 0 keeps the state; feeding the same batch again keeps the direction for any rho
    a0 = np.linspace(1.0, 2.0, Dsub)
    a, v = oracle.update_v(X, Dsub, 0.0, a0)
    assert _rel(a, a0) < 1e-15 and _rel(v, a0 / np.linalg.norm(a0)) < 1e-15
    a, v = oracle.update_v(X, Dsub, 0.3, mean)
    assert _rel(a, mean) < 1e-12 and _rel(v, v_mean) < 1e-12
    # the state is the convex combination, written out with numpy
    a, v = oracle.update_v(X, Dsub, 0.25, a0)
    expect = 0.75 * a0 + 0.25 * X.reshape(-1, Dsub).mean(axis=0)
    assert _rel(a, expect) < 1e-12 and _rel(v, expect / np.linalg.norm(expect)) < 1e-12
    # a planted mistake (sum instead of mean, or the weights swapped) is seen by the pins above
    wrong_sum = 0.75 * a0 + 0.25 * X.reshape(-1, Dsub).sum(axis=0)
    wrong_swap = 0.25 * a0 + 0.75 * X.reshape(-1, Dsub).mean(axis=0)
    assert _rel(wrong_sum, a) > 1e-2 and _rel(wrong_swap, a) > 1e-2
    with pytest.raises(oracle.OracleError):
        oracle.update_v(np.zeros((4, 32)), 16, 1.0)


# --- value-format helpers ---

def test_bf16_rounding_helper_matches_bit_level_rounding():
    rng = np.random.default_rng(20)
    a = (rng.standard_normal(20000) * np.exp(3 * rng.standard_normal(20000))).astype(np.float32)
    via_bits = vi.bf16_bits_to_f32(vi.f32_to_bf16_bits(a)).astype(np.float64)
    np.testing.assert_array_equal(oracle.round_to_bf16(a.astype(np.float64)), via_bits)
    # exact ties go to even: 1 + 2^-8 is halfway between 1 and 1 + 2^-7
    assert oracle.round_to_bf16(np.array([1.0 + 2.0 ** -8]))[0] == 1.0
    assert oracle.round_to_bf16(np.array([1.0 + 3 * 2.0 ** -8]))[0] == 1.0 + 2.0 ** -6
    assert oracle.round_to_bf16(np.array([0.0]))[0] == 0.0


def test_generator_is_seeded_and_rounds_once():
    cfg = vi.CONFIGS[2]
    a = vi.make_X(cfg, 0, N=64)
    b = vi.make_X(cfg, 0, N=64)
    np.testing.assert_array_equal(a.bits, b.bits)
    assert a.dtype == "bf16" and a.bits.dtype == np.uint16 and a.shape == (64, 512)
    assert not np.array_equal(a.bits, vi.make_X(cfg, 1, N=64).bits)
    c1 = vi.make_X(vi.CONFIGS[1], 0)
    assert c1.dtype == "f32" and c1.shape == (256, 64)
    t = a.torch()
    assert t.shape == (64, 512) and np.array_equal(t.view(__import__("torch").int16).numpy().view(np.uint16), a.bits)


# ------------------------------------------------------------------ E4M3 rounding helper (8-bit Z storage)
def _e4m3_table():
    """All finite E4M3 values straight from the format's definition: sign, exponent field E (bias 7),
    mantissa field m; E = 0 is subnormal (m/8 * 2^-6); E = 15, m = 7 is NaN; there are no infinities."""
    vals = []
    for code in range(256):
        s, E, m = code >> 7, (code >> 3) & 15, code & 7
        if E == 15 and m == 7:
            continue
        mag = (m / 8.0) * 2.0 ** -6 if E == 0 else (1.0 + m / 8.0) * 2.0 ** (E - 7)
        vals.append((code, -mag if s else mag))
    return vals


def test_round_to_fp8_e4m3_against_the_format_definition():
    table = _e4m3_table()
    assert len(table) == 254
    vals = np.array([v for _, v in table])
    assert vals.max() == 448.0 and np.min(np.abs(vals[vals != 0])) == 2.0 ** -9
    # every representable value is a fixed point
    np.testing.assert_array_equal(oracle.round_to_fp8_e4m3(vals), vals)
    pos = np.array(sorted(v for c, v in table if c < 128))            # 0 .. 448, 127 values
    codes = np.array(sorted(c for c, v in table if c < 128))
    lo, hi = pos[:-1], pos[1:]
    mid = 0.5 * (lo + hi)
    # just below / above a midpoint goes to the nearer neighbour; the midpoint itself to the even code
    np.testing.assert_array_equal(oracle.round_to_fp8_e4m3(mid * (1 - 1e-12)), lo)
    np.testing.assert_array_equal(oracle.round_to_fp8_e4m3(mid * (1 + 1e-12)), hi)
    even = np.where(codes[:-1] % 2 == 0, lo, hi)
    np.testing.assert_array_equal(oracle.round_to_fp8_e4m3(mid), even)
    np.testing.assert_array_equal(oracle.round_to_fp8_e4m3(-mid), -even)
    # saturation, tiny values, specials
    np.testing.assert_array_equal(oracle.round_to_fp8_e4m3([449.0, 464.0, 1e9, -1e9, np.inf, -np.inf]),
                                  [448.0, 448.0, 448.0, -448.0, 448.0, -448.0])
    np.testing.assert_array_equal(oracle.round_to_fp8_e4m3([2.0 ** -10, 2.0 ** -10 * 1.01, 2.0 ** -11]), [0.0, 2.0 ** -9, 0.0])
    assert np.isnan(oracle.round_to_fp8_e4m3(np.nan))


def test_round_to_fp8_e4m3_against_a_library_conversion():
    """torch's float8_e4m3fn cast is an independent implementation of the same rounding (inside the
    finite range; it does not saturate, so values are kept within +-448)."""
    torch = pytest.importorskip("torch")
    if not hasattr(torch, "float8_e4m3fn"):
        pytest.skip("this torch has no float8_e4m3fn")
    rng = np.random.default_rng(5)
    x = np.concatenate([rng.uniform(-448, 448, 20000), rng.standard_normal(20000) * 3,
                        rng.standard_normal(20000) * 0.01, rng.uniform(-2.0 ** -5, 2.0 ** -5, 20000)]).astype(np.float32)
    lib = torch.from_numpy(x).to(torch.float8_e4m3fn).to(torch.float32).numpy().astype(np.float64)
    np.testing.assert_array_equal(oracle.round_to_fp8_e4m3(x.astype(np.float64)), lib)


def test_fp8_z_store_scale_and_error_bound():
    rng = np.random.default_rng(6)
    Z = rng.standard_normal((300, 24)) * np.exp(rng.standard_normal(24))[None, :]
    scale = oracle.zscale_from_batch(Z, headroom=2.0)
    assert abs(scale * 448.0 - 2.0 * np.abs(Z).max()) < 1e-12
    q = oracle.quantize_z_fp8(Z, scale)
    assert np.abs(q).max() <= 448.0 / 2 + 16                      # headroom 2: the batch's own maximum sits at 224
    deq = q * scale
    normal = np.abs(Z) >= scale * 2.0 ** -6
    assert np.all(np.abs(deq - Z)[normal] <= np.abs(Z)[normal] * 2.0 ** -4)      # half a unit of a 4-bit significand
    assert np.all(np.abs(deq - Z)[~normal] <= scale * 2.0 ** -10)                # half the subnormal spacing
    assert oracle.zscale_from_batch(np.zeros((3, 3))) == 1.0
    assert oracle.zscale_from_batch(np.array([[np.nan]])) == 1.0
    # a later batch that exceeds the calibrated range saturates instead of overflowing
    assert oracle.quantize_z_fp8(np.array([1e6 * scale]), scale)[0] == 448.0
