// C-ABI entry points of the VeLoRA library: host-side validation and routing.
// Every argument check happens here, before any launch.
#include "common.cuh"
#include "gemm_tc.cuh"

namespace velora {

int device_info(DeviceInfo* out)
{
    static std::atomic<int> sm_count[64], smem_optin[64];      // 0 = not asked yet (both are positive on any device)
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return VELORA_ERR_CUDA;
    if (dev < 0 || dev >= 64) return VELORA_ERR_UNSUPPORTED;
    DeviceInfo di;
    di.sm_count = sm_count[dev].load(std::memory_order_relaxed);
    di.smem_optin = smem_optin[dev].load(std::memory_order_relaxed);
    if (di.sm_count == 0 || di.smem_optin == 0) {
        if (cudaDeviceGetAttribute(&di.sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
            return VELORA_ERR_CUDA;
        if (cudaDeviceGetAttribute(&di.smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess)
            return VELORA_ERR_CUDA;
        sm_count[dev].store(di.sm_count, std::memory_order_relaxed);
        smem_optin[dev].store(di.smem_optin, std::memory_order_relaxed);
    }
    *out = di;
    return VELORA_OK;
}

static unsigned long long g_launches = 0;

int after_launch()
{
    __atomic_add_fetch(&g_launches, 1ull, __ATOMIC_RELAXED);
    return cudaGetLastError() == cudaSuccess ? VELORA_OK : VELORA_ERR_CUDA;
}

namespace {

bool elem_aligned(const void* p, int dt)
{
    return (reinterpret_cast<uintptr_t>(p) % dtype_size(dt)) == 0;
}

int check_shape(int64_t N, int64_t D, int Dsub)
{
    if (N < 0 || D < 1 || Dsub < 1 || Dsub > D) return VELORA_ERR_INVALID_ARG;
    if (Dsub > VELORA_MAX_DSUB) return VELORA_ERR_UNSUPPORTED;
    if (D > (1 << 30) || N > (static_cast<int64_t>(1) << 40)) return VELORA_ERR_UNSUPPORTED;
    return VELORA_OK;
}

int64_t num_subtokens(int64_t D, int Dsub) { return ceil_div64(D, Dsub); }

int64_t round_up8(int64_t x) { return (x + 7) / 8 * 8; }

size_t align256(size_t x) { return (x + 255) / 256 * 256; }

size_t xhat_bytes(int64_t N, int64_t D)
{
    return kStatusBytes + align256(static_cast<size_t>(N) * round_up8(D) * 4);
}

size_t factored_bytes(int64_t N, int64_t D, int64_t O, int Dsub)
{
    const size_t simt = align256(static_cast<size_t>(O) * num_subtokens(D, Dsub) * sizeof(float));
    const size_t tc = weight_grad_tc_workspace_bytes(N, D, O, Dsub);
    const size_t skinny = weight_grad_skinny_workspace_bytes(N, D, O, Dsub);
    const size_t most = simt > tc ? simt : tc;
    return kStatusBytes + (most > skinny ? most : skinny);
}

// ---- weight gradient routing ----
int weight_grad_impl(const void* dY, int dy_dtype, int64_t N, int64_t O, int64_t lddy,
                     const void* Z, int z_dtype, int64_t ldz, const float* v, int64_t D, int Dsub,
                     void* dW, int dw_dtype, int64_t lddw, int beta, int mode,
                     void* ws, size_t ws_bytes, cudaStream_t stream)
{
    const int64_t M = num_subtokens(D, Dsub);
    int* status = static_cast<int*>(ws);                 // word 0: sticky device error flag
    char* body = static_cast<char*>(ws) + kStatusBytes;
    if (N == 0) {                                        // empty sum: dW = beta * dW
        if (beta) return VELORA_OK;
        const size_t es = dtype_size(dw_dtype);
        return cudaMemset2DAsync(dW, static_cast<size_t>(lddw) * es, 0, static_cast<size_t>(D) * es,
                                 static_cast<size_t>(O), stream) == cudaSuccess ? VELORA_OK : VELORA_ERR_CUDA;
    }
    if (mode == VELORA_WG_FACTORED) {
        if (ws_bytes < factored_bytes(N, D, O, Dsub)) return VELORA_ERR_WORKSPACE;
        // Adapter-shaped layers (O <= 64) first: too few output tiles for the tensor-core kernel to spread.
        int rc = launch_weight_grad_skinny(dY, dy_dtype, N, O, lddy, Z, z_dtype, ldz, v, D, Dsub, dW, dw_dtype, lddw,
                                           beta, body, ws_bytes - kStatusBytes, stream, nullptr, 0);
        if (rc != VELORA_ERR_UNSUPPORTED) return rc;
        rc = launch_weight_grad_tc(dY, dy_dtype, N, O, lddy, Z, z_dtype, ldz, v, D, Dsub,
                                       dW, dw_dtype, lddw, beta, body, ws_bytes - kStatusBytes, status, stream);
        if (rc != VELORA_ERR_UNSUPPORTED) return rc;
        // CUDA-core route: P[O, M] = dY^T Z, then the outer-product expansion.
        float* P = reinterpret_cast<float*>(body);
        rc = launch_gemm_simt(dY, dy_dtype, 1, lddy, Z, z_dtype, 1, ldz, P, VELORA_F32, M, 0, O, M, N, stream);
        if (rc != VELORA_OK) return rc;
        return launch_expand_p(P, 1, 0, M, v, O, D, Dsub, dW, dw_dtype, lddw, beta, stream);
    }
    // Explicit: Xhat into the workspace in dY's storage type, then dW = dY^T Xhat.
    if (ws_bytes < xhat_bytes(N, D)) return VELORA_ERR_WORKSPACE;
    const int64_t ldxh = round_up8(D);
    int rc = launch_reconstruct(Z, z_dtype, ldz, N, D, Dsub, v, body, dy_dtype, ldxh, stream);
    if (rc != VELORA_OK) return rc;
    rc = launch_gemm_tc(GEMM_TN_MN_MN, dY, lddy, body, ldxh, dW, dw_dtype, lddw, beta, O, D, N, dy_dtype, status, stream);
    if (rc != VELORA_ERR_UNSUPPORTED) return rc;
    return launch_gemm_simt(dY, dy_dtype, 1, lddy, body, dy_dtype, 1, ldxh, dW, dw_dtype, lddw, beta, O, D, N, stream);
}

int check_weight_grad_args(const void* dY, int dy_dtype, int64_t N, int64_t O, int64_t lddy,
                           const void* Z, int z_dtype, int64_t ldz, const float* v, int64_t D, int Dsub,
                           void* dW, int dw_dtype, int64_t lddw, int beta, int mode, void* ws)
{
    if (!dW) return VELORA_ERR_INVALID_ARG;
    if (O < 1 || O > (1 << 30)) return VELORA_ERR_INVALID_ARG;
    int rc = check_shape(N, D, Dsub);
    if (rc != VELORA_OK) return rc;
    if (!valid_dtype(dy_dtype) || !valid_z_dtype(z_dtype) || !valid_dtype(dw_dtype)) return VELORA_ERR_UNSUPPORTED;
    if (lddw < D) return VELORA_ERR_INVALID_ARG;
    if ((beta != 0 && beta != 1) || (mode != VELORA_WG_FACTORED && mode != VELORA_WG_EXPLICIT))
        return VELORA_ERR_INVALID_ARG;
    if (!elem_aligned(dW, dw_dtype)) return VELORA_ERR_ALIGNMENT;
    if (N > 0) {                                         /* an empty batch may carry NULL dY, Z and v */
        if (!dY || !Z || !v) return VELORA_ERR_INVALID_ARG;
        if (lddy < O || ldz < num_subtokens(D, Dsub)) return VELORA_ERR_INVALID_ARG;
        if (!elem_aligned(dY, dy_dtype) || !elem_aligned(Z, z_dtype) || !elem_aligned(v, VELORA_F32))
            return VELORA_ERR_ALIGNMENT;
    }
    if (!ws) return VELORA_ERR_WORKSPACE;
    if (!aligned16(ws)) return VELORA_ERR_ALIGNMENT;
    return VELORA_OK;
}

}  // namespace
}  // namespace velora

using namespace velora;

extern "C" {

int velora_version(void) { return 100; }

unsigned long long velora_launch_count(void) { return __atomic_load_n(&g_launches, __ATOMIC_RELAXED); }

int velora_workspace_init(void* ws, size_t ws_bytes, void* stream)
{
    if (!ws || ws_bytes < kStatusBytes) return VELORA_ERR_WORKSPACE;
    if (!aligned16(ws)) return VELORA_ERR_ALIGNMENT;
    return cudaMemsetAsync(ws, 0, kStatusBytes, static_cast<cudaStream_t>(stream)) == cudaSuccess ? VELORA_OK
                                                                                                   : VELORA_ERR_CUDA;
}

int velora_device_error(void* stream)
{
    return read_and_clear_stream_error(static_cast<cudaStream_t>(stream));
}

int velora_selftest_wait_timeout(void* ws, size_t ws_bytes, unsigned long long limit_ns, int* observed, void* stream)
{
    if (!ws || ws_bytes < kStatusBytes) return VELORA_ERR_WORKSPACE;
    if (!aligned16(ws)) return VELORA_ERR_ALIGNMENT;
    if (!observed) return VELORA_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(observed) % sizeof(int)) return VELORA_ERR_ALIGNMENT;
    if (limit_ns < 1000ull || limit_ns > 100000000ull) return VELORA_ERR_INVALID_ARG;   /* 1 us .. 100 ms */
    return launch_wait_timeout_selftest(static_cast<int*>(ws), limit_ns, observed, static_cast<cudaStream_t>(stream));
}

int velora_workspace_status(const void* ws, void* stream)
{
    if (!ws) return VELORA_ERR_WORKSPACE;
    int word = 0;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(&word, ws, sizeof(int), cudaMemcpyDeviceToHost, s) != cudaSuccess) return VELORA_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return VELORA_ERR_CUDA;
    if (word == 0) return VELORA_OK;
    return word == VELORA_ERR_DEGENERATE_V ? VELORA_ERR_DEGENERATE_V : VELORA_ERR_TIMEOUT;
}

const char* velora_status_string(int status)
{
    switch (status) {
        case VELORA_OK: return "ok";
        case VELORA_ERR_INVALID_ARG: return "invalid argument";
        case VELORA_ERR_UNSUPPORTED: return "unsupported dtype or size";
        case VELORA_ERR_ALIGNMENT: return "misaligned pointer";
        case VELORA_ERR_WORKSPACE: return "workspace missing or too small";
        case VELORA_ERR_DEGENERATE_V: return "sub-token sum has zero or non-finite length";
        case VELORA_ERR_TIMEOUT: return "device-side wait timed out";
        case VELORA_ERR_CUDA: return "CUDA runtime error";
        default: return "unknown status";
    }
}

size_t velora_workspace_bytes(int op, int64_t N, int64_t D, int64_t O, int Dsub)
{
    if (N < 0 || D < 1 || Dsub < 1 || Dsub > D || Dsub > VELORA_MAX_DSUB) return 0;
    switch (op) {
        case VELORA_OP_INIT_V: return init_v_workspace_bytes(Dsub);
        case VELORA_OP_WEIGHT_GRAD_FACTORED:
        case VELORA_OP_LINEAR_BACKWARD_FACTORED: return O < 1 ? 0 : factored_bytes(N, D, O, Dsub);
        case VELORA_OP_WEIGHT_GRAD_EXPLICIT:
        case VELORA_OP_LINEAR_BACKWARD_EXPLICIT: return xhat_bytes(N, D);
        case VELORA_OP_LINEAR_FORWARD: return kStatusBytes;
        case VELORA_OP_UPDATE_V: return update_v_workspace_bytes(Dsub);
        case VELORA_OP_Z8_CALIBRATE: return z8_calibrate_workspace_bytes(N, D, Dsub);
        default: return 0;
    }
}

int velora_init_v(const void* X, int x_dtype, int64_t N, int64_t D, int64_t ldx, int Dsub,
                  float* v, void* ws, size_t ws_bytes, void* stream)
{
    int rc = check_shape(N, D, Dsub);
    if (rc != VELORA_OK) return rc;
    if (!valid_dtype(x_dtype)) return VELORA_ERR_UNSUPPORTED;
    if (N == 0) return VELORA_ERR_DEGENERATE_V;      /* an empty batch has no mean; X may be NULL */
    if (!X || !v) return VELORA_ERR_INVALID_ARG;
    if (ldx < D) return VELORA_ERR_INVALID_ARG;
    if (!elem_aligned(X, x_dtype) || !elem_aligned(v, VELORA_F32)) return VELORA_ERR_ALIGNMENT;
    if (!ws || ws_bytes < init_v_workspace_bytes(Dsub)) return VELORA_ERR_WORKSPACE;
    if (!aligned16(ws)) return VELORA_ERR_ALIGNMENT;
    return launch_init_v(X, x_dtype, N, D, ldx, Dsub, v, ws, ws_bytes, static_cast<cudaStream_t>(stream));
}

int velora_compress(const void* X, int x_dtype, int64_t N, int64_t D, int64_t ldx, int Dsub,
                    const float* v, void* Z, int z_dtype, int64_t ldz, void* stream)
{
    int rc = check_shape(N, D, Dsub);
    if (rc != VELORA_OK) return rc;
    if (!valid_dtype(x_dtype) || !valid_z_dtype(z_dtype)) return VELORA_ERR_UNSUPPORTED;
    if (N == 0) return VELORA_OK;                    /* empty tensors may carry NULL pointers */
    if (!X || !v || !Z) return VELORA_ERR_INVALID_ARG;
    if (ldx < D || ldz < num_subtokens(D, Dsub)) return VELORA_ERR_INVALID_ARG;
    if (!elem_aligned(X, x_dtype) || !elem_aligned(Z, z_dtype) || !elem_aligned(v, VELORA_F32))
        return VELORA_ERR_ALIGNMENT;
    return launch_compress(X, x_dtype, N, D, ldx, Dsub, v, Z, z_dtype, ldz, static_cast<cudaStream_t>(stream));
}

int velora_reconstruct(const void* Z, int z_dtype, int64_t ldz, int64_t N, int64_t D, int Dsub,
                       const float* v, void* Xhat, int x_dtype, int64_t ldxhat, void* stream)
{
    int rc = check_shape(N, D, Dsub);
    if (rc != VELORA_OK) return rc;
    if (!valid_dtype(x_dtype) || !valid_z_dtype(z_dtype)) return VELORA_ERR_UNSUPPORTED;
    if (N == 0) return VELORA_OK;
    if (!Z || !v || !Xhat) return VELORA_ERR_INVALID_ARG;
    if (ldxhat < D || ldz < num_subtokens(D, Dsub)) return VELORA_ERR_INVALID_ARG;
    if (!elem_aligned(Xhat, x_dtype) || !elem_aligned(Z, z_dtype) || !elem_aligned(v, VELORA_F32))
        return VELORA_ERR_ALIGNMENT;
    return launch_reconstruct(Z, z_dtype, ldz, N, D, Dsub, v, Xhat, x_dtype, ldxhat,
                              static_cast<cudaStream_t>(stream));
}

int velora_weight_grad(const void* dY, int dy_dtype, int64_t N, int64_t O, int64_t lddy,
                       const void* Z, int z_dtype, int64_t ldz, const float* v, int64_t D, int Dsub,
                       void* dW, int dw_dtype, int64_t lddw, int beta, int mode,
                       void* ws, size_t ws_bytes, void* stream)
{
    int rc = check_weight_grad_args(dY, dy_dtype, N, O, lddy, Z, z_dtype, ldz, v, D, Dsub,
                                    dW, dw_dtype, lddw, beta, mode, ws);
    if (rc != VELORA_OK) return rc;
    const size_t need = velora_workspace_bytes(mode == VELORA_WG_FACTORED ? VELORA_OP_WEIGHT_GRAD_FACTORED
                                                                          : VELORA_OP_WEIGHT_GRAD_EXPLICIT,
                                               N, D, O, Dsub);
    if (ws_bytes < need) return VELORA_ERR_WORKSPACE;
    return weight_grad_impl(dY, dy_dtype, N, O, lddy, Z, z_dtype, ldz, v, D, Dsub, dW, dw_dtype, lddw,
                            beta, mode, ws, ws_bytes, static_cast<cudaStream_t>(stream));
}

int velora_linear_forward(const void* X, int64_t ldx, const void* W, int64_t ldw, const float* v,
                          void* Y, int64_t ldy, void* Z, int z_dtype, int64_t ldz,
                          int dtype, int64_t N, int64_t D, int64_t O, int Dsub,
                          void* ws, size_t ws_bytes, void* stream)
{
    if (O < 1 || O > (1 << 30)) return VELORA_ERR_INVALID_ARG;
    int rc = check_shape(N, D, Dsub);
    if (rc != VELORA_OK) return rc;
    if (!valid_dtype(dtype) || !valid_z_dtype(z_dtype)) return VELORA_ERR_UNSUPPORTED;
    if (N == 0) return VELORA_OK;
    if (!X || !W || !v || !Y || !Z) return VELORA_ERR_INVALID_ARG;
    if (ldx < D || ldw < D || ldy < O || ldz < num_subtokens(D, Dsub)) return VELORA_ERR_INVALID_ARG;
    if (!elem_aligned(X, dtype) || !elem_aligned(W, dtype) || !elem_aligned(Y, dtype) ||
        !elem_aligned(Z, z_dtype) || !elem_aligned(v, VELORA_F32))
        return VELORA_ERR_ALIGNMENT;
    if (!ws || ws_bytes < kStatusBytes) return VELORA_ERR_WORKSPACE;
    if (!aligned16(ws)) return VELORA_ERR_ALIGNMENT;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    rc = launch_linear_forward_tc(X, ldx, W, ldw, v, Y, ldy, Z, z_dtype, ldz, dtype, N, D, O, Dsub,
                                  static_cast<int*>(ws), s);
    if (rc != VELORA_ERR_UNSUPPORTED) return rc;
    rc = launch_gemm_simt(X, dtype, ldx, 1, W, dtype, ldw, 1, Y, dtype, ldy, 0, N, O, D, s);
    if (rc != VELORA_OK) return rc;
    return launch_compress(X, dtype, N, D, ldx, Dsub, v, Z, z_dtype, ldz, s);
}

int velora_linear_backward(const void* dY, int64_t lddy, const void* W, int64_t ldw,
                           const void* Z, int z_dtype, int64_t ldz, const float* v,
                           void* dX, int64_t lddx, void* dW, int dw_dtype, int64_t lddw, int beta, int mode,
                           int dtype, int64_t N, int64_t D, int64_t O, int Dsub,
                           void* ws, size_t ws_bytes, void* stream)
{
    if (O < 1 || O > (1 << 30)) return VELORA_ERR_INVALID_ARG;
    int rc = check_shape(N, D, Dsub);
    if (rc != VELORA_OK) return rc;
    if (!valid_dtype(dtype)) return VELORA_ERR_UNSUPPORTED;
    if (N > 0) {
        if (!dY) return VELORA_ERR_INVALID_ARG;
        if (lddy < O) return VELORA_ERR_INVALID_ARG;
        if (!elem_aligned(dY, dtype)) return VELORA_ERR_ALIGNMENT;
    }
    if (dX && N > 0) {
        if (!W) return VELORA_ERR_INVALID_ARG;
        if (ldw < D || lddx < D) return VELORA_ERR_INVALID_ARG;
        if (!elem_aligned(W, dtype) || !elem_aligned(dX, dtype)) return VELORA_ERR_ALIGNMENT;
    }
    if (dW) {
        rc = check_weight_grad_args(dY, dtype, N, O, lddy, Z, z_dtype, ldz, v, D, Dsub,
                                    dW, dw_dtype, lddw, beta, mode, ws);
        if (rc != VELORA_OK) return rc;
        const size_t need = velora_workspace_bytes(mode == VELORA_WG_FACTORED ? VELORA_OP_LINEAR_BACKWARD_FACTORED
                                                                              : VELORA_OP_LINEAR_BACKWARD_EXPLICIT,
                                                   N, D, O, Dsub);
        if (ws_bytes < need) return VELORA_ERR_WORKSPACE;
    }
    if (!ws || ws_bytes < kStatusBytes) return VELORA_ERR_WORKSPACE;
    if (!aligned16(ws)) return VELORA_ERR_ALIGNMENT;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (dX && N > 0) {
        rc = launch_gemm_tc(GEMM_NN_K_MN, dY, lddy, W, ldw, dX, dtype, lddx, 0, N, D, O, dtype,
                            static_cast<int*>(ws), s);
        if (rc == VELORA_ERR_UNSUPPORTED)
            rc = launch_gemm_simt(dY, dtype, lddy, 1, W, dtype, 1, ldw, dX, dtype, lddx, 0, N, D, O, s);
        if (rc != VELORA_OK) return rc;
    }
    if (dW)
        return weight_grad_impl(dY, dtype, N, O, lddy, Z, z_dtype, ldz, v, D, Dsub, dW, dw_dtype, lddw,
                                beta, mode, ws, ws_bytes, s);
    return VELORA_OK;
}

int velora_dense_product(int kind, const void* A, int64_t lda, const void* B, int64_t ldb,
                         void* C, int c_dtype, int64_t ldc, int beta,
                         int64_t Mdim, int64_t Ndim, int64_t Kdim, int dtype,
                         void* ws, size_t ws_bytes, void* stream)
{
    if (kind != VELORA_PRODUCT_A_BT && kind != VELORA_PRODUCT_A_B && kind != VELORA_PRODUCT_AT_B) return VELORA_ERR_INVALID_ARG;
    if (Mdim < 0 || Ndim < 1 || Kdim < 0 || (beta != 0 && beta != 1)) return VELORA_ERR_INVALID_ARG;
    if (Mdim > (1 << 30) || Ndim > (1 << 30) || Kdim > (1 << 30)) return VELORA_ERR_UNSUPPORTED;
    if (!valid_dtype(dtype) || !valid_dtype(c_dtype)) return VELORA_ERR_UNSUPPORTED;
    if (Mdim == 0) return VELORA_OK;
    if (!C || ldc < Ndim) return VELORA_ERR_INVALID_ARG;
    if (!elem_aligned(C, c_dtype)) return VELORA_ERR_ALIGNMENT;
    if (!ws || ws_bytes < kStatusBytes) return VELORA_ERR_WORKSPACE;
    if (!aligned16(ws)) return VELORA_ERR_ALIGNMENT;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (Kdim == 0) {                                     /* empty sum: C = beta * C */
        if (beta) return VELORA_OK;
        const size_t es = dtype_size(c_dtype);
        return cudaMemset2DAsync(C, static_cast<size_t>(ldc) * es, 0, static_cast<size_t>(Ndim) * es,
                                 static_cast<size_t>(Mdim), s) == cudaSuccess ? VELORA_OK : VELORA_ERR_CUDA;
    }
    if (!A || !B) return VELORA_ERR_INVALID_ARG;
    const bool a_t = kind == VELORA_PRODUCT_AT_B, b_t = kind == VELORA_PRODUCT_A_BT;
    if (lda < (a_t ? Mdim : Kdim) || ldb < (b_t ? Kdim : Ndim)) return VELORA_ERR_INVALID_ARG;
    if (!elem_aligned(A, dtype) || !elem_aligned(B, dtype)) return VELORA_ERR_ALIGNMENT;
    const int tc_kind = kind == VELORA_PRODUCT_A_BT ? GEMM_NT_K_K : (kind == VELORA_PRODUCT_A_B ? GEMM_NN_K_MN : GEMM_TN_MN_MN);
    int rc = launch_gemm_tc(tc_kind, A, lda, B, ldb, C, c_dtype, ldc, beta, Mdim, Ndim, Kdim, dtype,
                            static_cast<int*>(ws), s);
    if (rc != VELORA_ERR_UNSUPPORTED) return rc;
    return launch_gemm_simt(A, dtype, a_t ? 1 : lda, a_t ? lda : 1, B, dtype, b_t ? ldb : 1, b_t ? 1 : ldb,
                            C, c_dtype, ldc, beta, Mdim, Ndim, Kdim, s);
}

size_t velora_host_step_staging_bytes(int64_t N, int64_t D, int64_t O, int Dsub)
{
    if (N < 0 || D < 1 || O < 1 || Dsub < 1 || Dsub > D) return 0;
    const size_t n = static_cast<size_t>(N), d = static_cast<size_t>(D), o = static_cast<size_t>(O);
    const size_t m = static_cast<size_t>(num_subtokens(D, Dsub));
    return align256(n * d * 2) * 2 + align256(n * o * 2) * 2 + align256(o * d * 2) + align256(n * m * 4);
}

int velora_linear_step_host(const void* hX, const void* hdY, void* hY, void* hdX, void* hdW,
                            const void* W, const float* v, void* staging, size_t staging_bytes,
                            int64_t N, int64_t D, int64_t O, int Dsub,
                            void* ws, size_t ws_bytes, void* stream)
{
    if (O < 1 || O > (1 << 30)) return VELORA_ERR_INVALID_ARG;
    int rc = check_shape(N, D, Dsub);
    if (rc != VELORA_OK) return rc;
    if (N == 0) return VELORA_OK;
    if (!hX || !hdY || !W || !v || !staging) return VELORA_ERR_INVALID_ARG;
    if (D % 8 || O % 8) return VELORA_ERR_UNSUPPORTED;          /* dense bf16 rows must be 16-byte multiples */
    if (staging_bytes < velora_host_step_staging_bytes(N, D, O, Dsub)) return VELORA_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(staging) % 256) return VELORA_ERR_ALIGNMENT;
    const size_t n = static_cast<size_t>(N), d = static_cast<size_t>(D), o = static_cast<size_t>(O);
    const int64_t M = num_subtokens(D, Dsub);
    char* p = static_cast<char*>(staging);
    void* dXin = p;  p += align256(n * d * 2);
    void* ddX = p;   p += align256(n * d * 2);
    void* ddY = p;   p += align256(n * o * 2);
    void* dYout = p; p += align256(n * o * 2);
    void* ddW = p;   p += align256(o * d * 2);
    void* dZ = p;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(dXin, hX, n * d * 2, cudaMemcpyHostToDevice, s) != cudaSuccess) return VELORA_ERR_CUDA;
    if (cudaMemcpyAsync(ddY, hdY, n * o * 2, cudaMemcpyHostToDevice, s) != cudaSuccess) return VELORA_ERR_CUDA;
    rc = velora_linear_forward(dXin, D, W, D, v, dYout, O, dZ, VELORA_F32, M, VELORA_BF16, N, D, O, Dsub,
                               ws, ws_bytes, stream);
    if (rc != VELORA_OK) return rc;
    rc = velora_linear_backward(ddY, O, W, D, dZ, VELORA_F32, M, v, ddX, D, ddW, VELORA_BF16, D, 0,
                                VELORA_WG_FACTORED, VELORA_BF16, N, D, O, Dsub, ws, ws_bytes, stream);
    if (rc != VELORA_OK) return rc;
    if (hY && cudaMemcpyAsync(hY, dYout, n * o * 2, cudaMemcpyDeviceToHost, s) != cudaSuccess) return VELORA_ERR_CUDA;
    if (hdX && cudaMemcpyAsync(hdX, ddX, n * d * 2, cudaMemcpyDeviceToHost, s) != cudaSuccess) return VELORA_ERR_CUDA;
    if (hdW && cudaMemcpyAsync(hdW, ddW, o * d * 2, cudaMemcpyDeviceToHost, s) != cudaSuccess) return VELORA_ERR_CUDA;
    return VELORA_OK;
}

int velora_subtoken_sum(const void* X, int x_dtype, int64_t N, int64_t D, int64_t ldx, int Dsub,
                        float* s, void* ws, size_t ws_bytes, void* stream)
{
    int rc = check_shape(N, D, Dsub);
    if (rc != VELORA_OK) return rc;
    if (!valid_dtype(x_dtype)) return VELORA_ERR_UNSUPPORTED;
    if (!s) return VELORA_ERR_INVALID_ARG;
    if (!elem_aligned(s, VELORA_F32)) return VELORA_ERR_ALIGNMENT;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (N == 0)                                           /* an empty shard contributes a zero sum */
        return cudaMemsetAsync(s, 0, sizeof(float) * Dsub, st) == cudaSuccess ? VELORA_OK : VELORA_ERR_CUDA;
    if (!X) return VELORA_ERR_INVALID_ARG;
    if (ldx < D) return VELORA_ERR_INVALID_ARG;
    if (!elem_aligned(X, x_dtype)) return VELORA_ERR_ALIGNMENT;
    if (!ws || ws_bytes < init_v_workspace_bytes(Dsub)) return VELORA_ERR_WORKSPACE;
    if (!aligned16(ws)) return VELORA_ERR_ALIGNMENT;
    return launch_init_v(X, x_dtype, N, D, ldx, Dsub, s, ws, ws_bytes, st, 1);
}

int velora_update_v(const void* X, int x_dtype, int64_t N, int64_t D, int64_t ldx, int Dsub, float rho,
                    float* a, float* v, void* ws, size_t ws_bytes, void* stream)
{
    int rc = check_shape(N, D, Dsub);
    if (rc != VELORA_OK) return rc;
    if (!valid_dtype(x_dtype)) return VELORA_ERR_UNSUPPORTED;
    if (!(rho >= 0.f && rho <= 1.f)) return VELORA_ERR_INVALID_ARG;
    if (N == 0) return VELORA_OK;                         /* an empty batch has no mean: a and v stay */
    if (!X || !a || !v) return VELORA_ERR_INVALID_ARG;
    if (ldx < D) return VELORA_ERR_INVALID_ARG;
    if (!elem_aligned(X, x_dtype) || !elem_aligned(a, VELORA_F32) || !elem_aligned(v, VELORA_F32)) return VELORA_ERR_ALIGNMENT;
    if (!ws || ws_bytes < update_v_workspace_bytes(Dsub)) return VELORA_ERR_WORKSPACE;
    if (!aligned16(ws)) return VELORA_ERR_ALIGNMENT;
    return launch_update_v(X, x_dtype, N, D, ldx, Dsub, rho, a, v, ws, ws_bytes, static_cast<cudaStream_t>(stream));
}

int velora_z8_calibrate(const void* X, int x_dtype, int64_t N, int64_t D, int64_t ldx, int Dsub, const float* v,
                        float headroom, float* zscale, float* v_store, float* v_load,
                        void* ws, size_t ws_bytes, void* stream)
{
    int rc = check_shape(N, D, Dsub);
    if (rc != VELORA_OK) return rc;
    if (!valid_dtype(x_dtype)) return VELORA_ERR_UNSUPPORTED;
    if (!(headroom >= 1.f && headroom <= 1024.f)) return VELORA_ERR_INVALID_ARG;
    if (!v || !zscale || !v_store || !v_load) return VELORA_ERR_INVALID_ARG;
    if (N > 0 && (!X || ldx < D)) return VELORA_ERR_INVALID_ARG;
    if ((N > 0 && !elem_aligned(X, x_dtype)) || !elem_aligned(v, VELORA_F32) || !elem_aligned(zscale, VELORA_F32) ||
        !elem_aligned(v_store, VELORA_F32) || !elem_aligned(v_load, VELORA_F32))
        return VELORA_ERR_ALIGNMENT;
    if (!ws || ws_bytes < z8_calibrate_workspace_bytes(N, D, Dsub)) return VELORA_ERR_WORKSPACE;
    if (!aligned16(ws)) return VELORA_ERR_ALIGNMENT;
    return launch_z8_calibrate(X, x_dtype, N, D, ldx, Dsub, v, headroom, zscale, v_store, v_load, ws, ws_bytes,
                               static_cast<cudaStream_t>(stream));
}

int velora_normalize_v(const float* s, int Dsub, float* v, void* ws, size_t ws_bytes, void* stream)
{
    if (!s || !v || Dsub < 1) return VELORA_ERR_INVALID_ARG;
    if (Dsub > VELORA_MAX_DSUB) return VELORA_ERR_UNSUPPORTED;
    if (!elem_aligned(s, VELORA_F32) || !elem_aligned(v, VELORA_F32)) return VELORA_ERR_ALIGNMENT;
    if (!ws || ws_bytes < kStatusBytes) return VELORA_ERR_WORKSPACE;
    if (!aligned16(ws)) return VELORA_ERR_ALIGNMENT;
    return launch_normalize_v(s, Dsub, v, ws, ws_bytes, static_cast<cudaStream_t>(stream));
}

int velora_weight_grad_p(const void* dY, int dy_dtype, int64_t N, int64_t O, int64_t lddy,
                         const void* Z, int z_dtype, int64_t ldz, int64_t D, int Dsub,
                         float* P, int64_t ldp, int beta, void* ws, size_t ws_bytes, void* stream)
{
    if (O < 1 || O > (1 << 30)) return VELORA_ERR_INVALID_ARG;
    int rc = check_shape(N, D, Dsub);
    if (rc != VELORA_OK) return rc;
    if (!valid_dtype(dy_dtype) || !valid_z_dtype(z_dtype)) return VELORA_ERR_UNSUPPORTED;
    const int64_t M = num_subtokens(D, Dsub);
    if (!P || ldp < M || (beta != 0 && beta != 1)) return VELORA_ERR_INVALID_ARG;
    if (!elem_aligned(P, VELORA_F32)) return VELORA_ERR_ALIGNMENT;
    if (N > 0) {
        if (!dY || !Z) return VELORA_ERR_INVALID_ARG;
        if (lddy < O || ldz < M) return VELORA_ERR_INVALID_ARG;
        if (!elem_aligned(dY, dy_dtype) || !elem_aligned(Z, z_dtype)) return VELORA_ERR_ALIGNMENT;
    }
    if (!ws || ws_bytes < factored_bytes(N, D, O, Dsub)) return VELORA_ERR_WORKSPACE;
    if (!aligned16(ws)) return VELORA_ERR_ALIGNMENT;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int* status = static_cast<int*>(ws);
    char* body = static_cast<char*>(ws) + kStatusBytes;
    if (N > 0) {
        rc = launch_weight_grad_skinny(dY, dy_dtype, N, O, lddy, Z, z_dtype, ldz, nullptr, D, Dsub, nullptr, VELORA_F32, D,
                                       beta, body, ws_bytes - kStatusBytes, st, P, ldp);
        if (rc != VELORA_ERR_UNSUPPORTED) return rc;
    }
    rc = launch_weight_grad_tc(dY, dy_dtype, N, O, lddy, Z, z_dtype, ldz, nullptr, D, Dsub, nullptr, VELORA_F32, D, beta,
                               body, ws_bytes - kStatusBytes, status, st, P, ldp);
    if (rc != VELORA_ERR_UNSUPPORTED) return rc;
    if (N == 0 && beta) return VELORA_OK;
    return launch_gemm_simt(dY, dy_dtype, 1, lddy, Z, z_dtype, 1, ldz, P, VELORA_F32, ldp, beta, O, M, N, st);
}

int velora_expand_p(const float* P, int64_t ldp, const float* v, int64_t O, int64_t D, int Dsub,
                    void* dW, int dw_dtype, int64_t lddw, int beta, void* stream)
{
    if (O < 1 || O > (1 << 30)) return VELORA_ERR_INVALID_ARG;
    int rc = check_shape(0, D, Dsub);
    if (rc != VELORA_OK) return rc;
    if (!P || !v || !dW) return VELORA_ERR_INVALID_ARG;
    if (!valid_dtype(dw_dtype)) return VELORA_ERR_UNSUPPORTED;
    if (ldp < num_subtokens(D, Dsub) || lddw < D || (beta != 0 && beta != 1)) return VELORA_ERR_INVALID_ARG;
    if (!elem_aligned(P, VELORA_F32) || !elem_aligned(v, VELORA_F32) || !elem_aligned(dW, dw_dtype))
        return VELORA_ERR_ALIGNMENT;
    return launch_expand_p(P, 1, 0, ldp, v, O, D, Dsub, dW, dw_dtype, lddw, beta, static_cast<cudaStream_t>(stream));
}

}  // extern "C"
