// CUDA-core GEMM with arbitrary element strides and fp32 accumulation.
//   C[m, n] = beta * C[m, n] + sum_k A(m, k) * B(n, k)
// It computes the dense products of Algorithm 1 (arxiv 2405.17991) for the
// all-fp32 case, where tensor cores would drop mantissa bits, and for operand
// layouts the tensor-core kernels do not take (rows that are not 16-byte
// multiples).  64x64 output tile, 16-deep k slices, 4x4 outputs per thread.
#include "common.cuh"

namespace velora {
namespace {

constexpr int TM = 64, TN = 64, TK = 16, THREADS = 256;

template <typename AT, typename BT, typename CT>
__global__ void __launch_bounds__(THREADS)
gemm_simt_kernel(const AT* __restrict__ A, int64_t a_sm, int64_t a_sk,
                 const BT* __restrict__ B, int64_t b_sn, int64_t b_sk,
                 CT* __restrict__ C, int64_t ldc, int beta,
                 int64_t Mdim, int64_t Ndim, int64_t Kdim)
{
    __shared__ float As[TK][TM + 4];
    __shared__ float Bs[TK][TN + 4];
    const int t = threadIdx.x;
    const int tx = t % 16, ty = t / 16;
    const int64_t m0 = static_cast<int64_t>(blockIdx.y) * TM;
    const int64_t n0 = static_cast<int64_t>(blockIdx.x) * TN;
    const bool a_kfast = (a_sk == 1);
    const bool b_kfast = (b_sk == 1);

    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

    for (int64_t k0 = 0; k0 < Kdim; k0 += TK) {
#pragma unroll
        for (int i = 0; i < (TM * TK) / THREADS; ++i) {
            const int idx = t + THREADS * i;
            const int kk = a_kfast ? idx % TK : idx / TM;
            const int mm = a_kfast ? idx / TK : idx % TM;
            const int64_t m = m0 + mm, k = k0 + kk;
            As[kk][mm] = (m < Mdim && k < Kdim) ? Elem<AT>::load(A + m * a_sm + k * a_sk) : 0.f;
        }
#pragma unroll
        for (int i = 0; i < (TN * TK) / THREADS; ++i) {
            const int idx = t + THREADS * i;
            const int kk = b_kfast ? idx % TK : idx / TN;
            const int nn = b_kfast ? idx / TK : idx % TN;
            const int64_t n = n0 + nn, k = k0 + kk;
            Bs[kk][nn] = (n < Ndim && k < Kdim) ? Elem<BT>::load(B + n * b_sn + k * b_sk) : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < TK; ++kk) {
            float a[4], b[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) a[i] = As[kk][ty * 4 + i];
#pragma unroll
            for (int j = 0; j < 4; ++j) b[j] = Bs[kk][tx * 4 + j];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int64_t m = m0 + ty * 4 + i;
        if (m >= Mdim) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int64_t n = n0 + tx * 4 + j;
            if (n >= Ndim) continue;
            CT* p = C + m * ldc + n;
            float r = acc[i][j];
            if (beta) r += Elem<CT>::load(p);
            Elem<CT>::store(p, r);
        }
    }
}

template <typename AT, typename BT>
int dispatch_c(const void* A, int64_t a_sm, int64_t a_sk, const void* B, int64_t b_sn, int64_t b_sk,
               void* C, int c_dtype, int64_t ldc, int beta, int64_t Mdim, int64_t Ndim, int64_t Kdim,
               dim3 grid, cudaStream_t stream)
{
    if (c_dtype == VELORA_BF16)
        gemm_simt_kernel<AT, BT, __nv_bfloat16><<<grid, THREADS, 0, stream>>>(
            static_cast<const AT*>(A), a_sm, a_sk, static_cast<const BT*>(B), b_sn, b_sk,
            static_cast<__nv_bfloat16*>(C), ldc, beta, Mdim, Ndim, Kdim);
    else
        gemm_simt_kernel<AT, BT, float><<<grid, THREADS, 0, stream>>>(
            static_cast<const AT*>(A), a_sm, a_sk, static_cast<const BT*>(B), b_sn, b_sk,
            static_cast<float*>(C), ldc, beta, Mdim, Ndim, Kdim);
    return after_launch();
}

}  // namespace

int launch_gemm_simt(const void* A, int a_dtype, int64_t a_sm, int64_t a_sk,
                     const void* B, int b_dtype, int64_t b_sn, int64_t b_sk,
                     void* C, int c_dtype, int64_t ldc, int beta,
                     int64_t Mdim, int64_t Ndim, int64_t Kdim, cudaStream_t stream)
{
    if (Mdim <= 0 || Ndim <= 0) return VELORA_OK;
    const int64_t gx = ceil_div64(Ndim, TN), gy = ceil_div64(Mdim, TM);
    if (gy > 65535) return VELORA_ERR_UNSUPPORTED;
    dim3 grid(static_cast<unsigned>(gx), static_cast<unsigned>(gy));
    if (b_dtype == VELORA_FP8_E4M3) {                    // Z in its 8-bit store as the second operand of dY^T Z
        if (a_dtype == VELORA_BF16)
            return dispatch_c<__nv_bfloat16, e4m3_t>(A, a_sm, a_sk, B, b_sn, b_sk, C, c_dtype, ldc, beta, Mdim, Ndim, Kdim, grid, stream);
        return dispatch_c<float, e4m3_t>(A, a_sm, a_sk, B, b_sn, b_sk, C, c_dtype, ldc, beta, Mdim, Ndim, Kdim, grid, stream);
    }
    if (a_dtype == VELORA_BF16 && b_dtype == VELORA_BF16)
        return dispatch_c<__nv_bfloat16, __nv_bfloat16>(A, a_sm, a_sk, B, b_sn, b_sk, C, c_dtype, ldc, beta, Mdim, Ndim, Kdim, grid, stream);
    if (a_dtype == VELORA_BF16 && b_dtype == VELORA_F32)
        return dispatch_c<__nv_bfloat16, float>(A, a_sm, a_sk, B, b_sn, b_sk, C, c_dtype, ldc, beta, Mdim, Ndim, Kdim, grid, stream);
    if (a_dtype == VELORA_F32 && b_dtype == VELORA_BF16)
        return dispatch_c<float, __nv_bfloat16>(A, a_sm, a_sk, B, b_sn, b_sk, C, c_dtype, ldc, beta, Mdim, Ndim, Kdim, grid, stream);
    return dispatch_c<float, float>(A, a_sm, a_sk, B, b_sn, b_sk, C, c_dtype, ldc, beta, Mdim, Ndim, Kdim, grid, stream);
}

}  // namespace velora
