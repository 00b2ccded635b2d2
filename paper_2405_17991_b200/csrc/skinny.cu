// Adapter-shaped layers (Section 4: VeLoRA on the down projections of trainable adapters, output width
// O = the adapter rank, 4 .. 64): the factored weight gradient of Algorithm 1 for a tiny O.
//     P[o, m] = sum_n dY[n, o] * Z[n, m]            (O x M <= 64 x 256 values, a few MFLOP)
//     dW[o, m*Dsub + j] = beta*dW + P[o, m] * v[j]
// With one or two output tiles the tensor-core kernel of weight_grad_tc.cu cannot spread over the SMs (at
// most 8 CTAs pull on dY and Z); here every SM takes a slice of the tokens and forms its own partial P on
// the CUDA cores, a second kernel adds the partials in a fixed order, and the common expansion kernel
// writes dW.  All sums are fp32, products are formed from the stored values (Z is not rounded to bf16).
#include "common.cuh"

namespace velora {

namespace {

constexpr int SK_THREADS = 256;
constexpr int SK_CHUNK = 32;          // tokens staged in shared memory at a time
constexpr int SK_MAX_O = 64;
constexpr int SK_MAX_M = 256;

// Thread (warp w, lane l) owns outputs o = w + 8 i (i < OI), m = l + 32 j (j < MJ).
template <typename YT, typename ZT, int OI, int MJ>
__global__ void __launch_bounds__(SK_THREADS)
wg_skinny_partial_kernel(const YT* __restrict__ dY, int64_t lddy, const ZT* __restrict__ Z, int64_t ldz,
                         int N, int O, int M, int tokens_per_cta, float* __restrict__ partials)
{
    __shared__ float sdy[SK_CHUNK][8 * OI];
    __shared__ float sz[SK_CHUNK][32 * MJ];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_begin = blockIdx.x * tokens_per_cta;
    const int n_end = (n_begin + tokens_per_cta < N) ? n_begin + tokens_per_cta : N;
    float acc[OI][MJ];
#pragma unroll
    for (int i = 0; i < OI; ++i)
#pragma unroll
        for (int j = 0; j < MJ; ++j) acc[i][j] = 0.f;

    for (int n0 = n_begin; n0 < n_end; n0 += SK_CHUNK) {
        for (int idx = threadIdx.x; idx < SK_CHUNK * 8 * OI; idx += SK_THREADS) {
            const int r = idx / (8 * OI), o = idx - r * (8 * OI);
            const int n = n0 + r;
            sdy[r][o] = (n < n_end && o < O) ? Elem<YT>::load(dY + static_cast<int64_t>(n) * lddy + o) : 0.f;
        }
        for (int idx = threadIdx.x; idx < SK_CHUNK * 32 * MJ; idx += SK_THREADS) {
            const int r = idx / (32 * MJ), m = idx - r * (32 * MJ);
            const int n = n0 + r;
            sz[r][m] = (n < n_end && m < M) ? Elem<ZT>::load(Z + static_cast<int64_t>(n) * ldz + m) : 0.f;
        }
        __syncthreads();
#pragma unroll 4
        for (int r = 0; r < SK_CHUNK; ++r) {
            float y[OI], z[MJ];
#pragma unroll
            for (int i = 0; i < OI; ++i) y[i] = sdy[r][warp + 8 * i];
#pragma unroll
            for (int j = 0; j < MJ; ++j) z[j] = sz[r][lane + 32 * j];
#pragma unroll
            for (int i = 0; i < OI; ++i)
#pragma unroll
                for (int j = 0; j < MJ; ++j) acc[i][j] = fmaf(y[i], z[j], acc[i][j]);
        }
        __syncthreads();
    }
    float* out = partials + static_cast<int64_t>(blockIdx.x) * O * M;
#pragma unroll
    for (int i = 0; i < OI; ++i)
#pragma unroll
        for (int j = 0; j < MJ; ++j) {
            const int o = warp + 8 * i, m = lane + 32 * j;
            if (o < O && m < M) out[o * M + m] = acc[i][j];
        }
}

// P[o*ldp + m] = beta * P + sum over the partials, added in a fixed order, eight loads in flight.
__global__ void __launch_bounds__(SK_THREADS)
wg_skinny_reduce_kernel(const float* __restrict__ partials, int parts, int O, int M, float* __restrict__ P,
                        int64_t ldp, int beta)
{
    const int total = O * M;
    for (int idx = blockIdx.x * SK_THREADS + threadIdx.x; idx < total; idx += gridDim.x * SK_THREADS) {
        float s = 0.f;
        for (int b = 0; b < parts; b += 8) {
            float x[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) x[u] = (b + u < parts) ? partials[static_cast<int64_t>(b + u) * total + idx] : 0.f;
#pragma unroll
            for (int u = 0; u < 8; ++u) s += x[u];
        }
        const int o = idx / M, m = idx - o * M;
        float* p = P + static_cast<int64_t>(o) * ldp + m;
        *p = beta ? *p + s : s;
    }
}

struct SkinnyPlan {
    bool ok;
    int M, oi, mj, tokens_per_cta, parts;
    size_t partial_bytes, p_bytes;
};

SkinnyPlan skinny_plan(int64_t N, int64_t D, int64_t O, int Dsub, int sm_count)
{
    SkinnyPlan p{};
    const int64_t M = ceil_div64(D, Dsub);
    if (O < 1 || O > SK_MAX_O || M > SK_MAX_M || N < 1 || N > (1 << 30)) return p;
    p.M = static_cast<int>(M);
    p.oi = static_cast<int>((O + 7) / 8);
    p.oi = p.oi <= 2 ? 2 : (p.oi <= 4 ? 4 : 8);
    p.mj = static_cast<int>((M + 31) / 32);
    p.mj = p.mj <= 2 ? 2 : (p.mj <= 4 ? 4 : 8);
    int64_t tpc = ceil_div64(N, sm_count);
    tpc = ceil_div64(tpc, SK_CHUNK) * SK_CHUNK;
    p.tokens_per_cta = static_cast<int>(tpc);
    p.parts = static_cast<int>(ceil_div64(N, tpc));
    p.partial_bytes = ((static_cast<size_t>(p.parts) * O * M * sizeof(float) + 255) / 256) * 256;
    p.p_bytes = ((static_cast<size_t>(O) * M * sizeof(float) + 255) / 256) * 256;
    p.ok = true;
    return p;
}

template <typename YT, typename ZT>
int launch_partial(const SkinnyPlan& p, const void* dY, int64_t lddy, const void* Z, int64_t ldz, int N, int O,
                   float* partials, cudaStream_t stream)
{
#define VELORA_SK_CASE(OIV, MJV)                                                                                  \
    if (p.oi == OIV && p.mj == MJV) {                                                                             \
        wg_skinny_partial_kernel<YT, ZT, OIV, MJV><<<p.parts, SK_THREADS, 0, stream>>>(                           \
            static_cast<const YT*>(dY), lddy, static_cast<const ZT*>(Z), ldz, N, O, p.M, p.tokens_per_cta, partials); \
        return after_launch();                                                                                    \
    }
    VELORA_SK_CASE(2, 2) VELORA_SK_CASE(2, 4) VELORA_SK_CASE(2, 8)
    VELORA_SK_CASE(4, 2) VELORA_SK_CASE(4, 4) VELORA_SK_CASE(4, 8)
    VELORA_SK_CASE(8, 2) VELORA_SK_CASE(8, 4) VELORA_SK_CASE(8, 8)
#undef VELORA_SK_CASE
    return VELORA_ERR_UNSUPPORTED;
}

}  // namespace

size_t weight_grad_skinny_workspace_bytes(int64_t N, int64_t D, int64_t O, int Dsub)
{
    const SkinnyPlan p = skinny_plan(N > 0 ? N : 1, D, O, Dsub, 148);
    // The token range is always cut into at most 148 slices, whatever the device, so the size is fixed.
    return p.ok ? p.partial_bytes + p.p_bytes : 0;
}

// Returns VELORA_ERR_UNSUPPORTED (nothing launched) when the shape is not adapter-like (O > 64 or M > 256).
// P_out != NULL: only the factor, P_out = beta * P_out + dY^T Z (dW, v unused).
int launch_weight_grad_skinny(const void* dY, int dy_dtype, int64_t N, int64_t O, int64_t lddy,
                              const void* Z, int z_dtype, int64_t ldz, const float* v, int64_t D, int Dsub,
                              void* dW, int dw_dtype, int64_t lddw, int beta,
                              void* ws, size_t ws_bytes, cudaStream_t stream, float* P_out, int64_t ldp_out)
{
    const SkinnyPlan p = skinny_plan(N, D, O, Dsub, 148);
    if (!p.ok) return VELORA_ERR_UNSUPPORTED;
    if (ws_bytes < p.partial_bytes + p.p_bytes) return VELORA_ERR_WORKSPACE;
    float* partials = static_cast<float*>(ws);
    float* P = reinterpret_cast<float*>(static_cast<char*>(ws) + p.partial_bytes);
    const int n = static_cast<int>(N), o = static_cast<int>(O);
    int rc;
    if (dy_dtype == VELORA_BF16)
        rc = z_dtype == VELORA_BF16 ? launch_partial<__nv_bfloat16, __nv_bfloat16>(p, dY, lddy, Z, ldz, n, o, partials, stream)
                                    : launch_partial<__nv_bfloat16, float>(p, dY, lddy, Z, ldz, n, o, partials, stream);
    else
        rc = z_dtype == VELORA_BF16 ? launch_partial<float, __nv_bfloat16>(p, dY, lddy, Z, ldz, n, o, partials, stream)
                                    : launch_partial<float, float>(p, dY, lddy, Z, ldz, n, o, partials, stream);
    if (rc != VELORA_OK) return rc;
    const int total = o * p.M;
    const int grid = (total + SK_THREADS - 1) / SK_THREADS;
    if (P_out) {
        wg_skinny_reduce_kernel<<<grid, SK_THREADS, 0, stream>>>(partials, p.parts, o, p.M, P_out, ldp_out, beta);
        return after_launch();
    }
    wg_skinny_reduce_kernel<<<grid, SK_THREADS, 0, stream>>>(partials, p.parts, o, p.M, P, p.M, 0);
    rc = after_launch();
    if (rc != VELORA_OK) return rc;
    return launch_expand_p(P, 1, 0, p.M, v, O, D, Dsub, dW, dw_dtype, lddw, beta, stream);
}

}  // namespace velora
