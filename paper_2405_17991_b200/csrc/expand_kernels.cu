// "Row of scalars times v": the write-bound half of the VeLoRA path (arxiv 2405.17991).
//   out[r, m*Dsub + j] = beta * out[r, m*Dsub + j] + (sum_s S[s][r][m]) * v[j]
// With one split and beta = 0 this is reconstruct + ungroup (Section 3.1, Eq. 2: Xhat = Z (x) v);
// with several splits it is the expansion of the factored weight gradient (dW = P (x) v, the per
// sub-token form of Section 3.2's g v v^T), where S holds partial products dY^T Z over disjoint token
// ranges that are summed here in a fixed order.
//
// A warp takes one output row and 32 consecutive sub-tokens.  Lane l loads the scalars of sub-token
// m0 + l (one coalesced load per split, all independent), then the warp walks the 32 sub-tokens,
// 32 / LPS of them per store instruction (LPS = Dsub / 8 lanes cover one sub-token), each scalar
// handed to its lanes by shuffle.  A lane keeps its 8-element slice of v in registers and its output
// pointer advances by a constant, so one store instruction costs one shuffle, eight multiplies, four
// packs and the store; every store instruction writes one contiguous 512-byte span.
#include "common.cuh"

namespace velora {
namespace {

constexpr unsigned kFull = 0xffffffffu;

template <typename T> __device__ __forceinline__ float load_scalar(const T* p);
template <> __device__ __forceinline__ float load_scalar<float>(const float* p) { return __ldg(p); }
template <> __device__ __forceinline__ float load_scalar<__nv_bfloat16>(const __nv_bfloat16* p)
{
    return __bfloat162float(*p);
}
template <> __device__ __forceinline__ float load_scalar<e4m3_t>(const e4m3_t* p) { return e4m3_to_float(*p); }

template <typename WT> struct Out8;
template <> struct Out8<__nv_bfloat16> {
    static __device__ __forceinline__ void store(__nv_bfloat16* p, float (&y)[8], int beta)
    {
        uint4* q = reinterpret_cast<uint4*>(p);
        if (beta) {
            const uint4 old = *q;
            y[0] += bf16_lo(old.x); y[1] += bf16_hi(old.x);
            y[2] += bf16_lo(old.y); y[3] += bf16_hi(old.y);
            y[4] += bf16_lo(old.z); y[5] += bf16_hi(old.z);
            y[6] += bf16_lo(old.w); y[7] += bf16_hi(old.w);
        }
        uint4 o;
        o.x = pack_bf16x2(y[0], y[1]);
        o.y = pack_bf16x2(y[2], y[3]);
        o.z = pack_bf16x2(y[4], y[5]);
        o.w = pack_bf16x2(y[6], y[7]);
        __stcs(q, o);
    }
};
template <> struct Out8<float> {
    static __device__ __forceinline__ void store(float* p, float (&y)[8], int beta)
    {
        float4* q = reinterpret_cast<float4*>(p);
        if (beta) {
            const float4 a = q[0], b = q[1];
            y[0] += a.x; y[1] += a.y; y[2] += a.z; y[3] += a.w;
            y[4] += b.x; y[5] += b.y; y[6] += b.z; y[7] += b.w;
        }
        __stcs(q, make_float4(y[0], y[1], y[2], y[3]));
        __stcs(q + 1, make_float4(y[4], y[5], y[6], y[7]));
    }
};

// MODE 0: M is a multiple of 32 and Dsub divides D (no checks in the store loop).
// MODE 1: Dsub divides D, the last block of 32 sub-tokens is partial (one compare per store).
// MODE 2: ragged last sub-token as well (column checks, element-wise tail).
template <int LPS, int CH, int MODE, typename ST, typename WT>
__global__ void __launch_bounds__(kStreamThreads)
expand_rows_vec_kernel(const ST* __restrict__ S, int splits, int64_t split_stride, int lds,
                       const float* __restrict__ v, int R, int D, int M, int mblocks,
                       WT* __restrict__ out, int64_t ldo, int beta)
{
    constexpr int L = LPS * CH;                  // 16-byte chunks per sub-token
    constexpr int SPW = 32 / LPS;                // sub-tokens per store instruction
    const int lane = threadIdx.x & 31;
    const int q = lane & (LPS - 1);
    const int sub = lane / LPS;
    // Programmatic stream serialisation (see common.cuh): resident early, nothing read or written before the wait.
    pdl_trigger();
    pdl_wait();
    float vr[CH][8];
#pragma unroll
    for (int i = 0; i < CH; ++i)
#pragma unroll
        for (int e = 0; e < 8; ++e) vr[i][e] = __ldg(v + 8 * (q + LPS * i) + e);

    // One warp per output row at a time.  The row's scalars are fetched for up to PB blocks of 32 sub-tokens
    // before the first store, so a row costs one load latency per PB blocks instead of one per block (a row of
    // 172 sub-tokens went through six dependent round trips to memory before).
    constexpr int PB = 4;
    const int warps = gridDim.x * (kStreamThreads / 32);
    for (int r = blockIdx.x * (kStreamThreads / 32) + (threadIdx.x >> 5); r < R; r += warps)
    for (int mb0 = 0; mb0 < mblocks; mb0 += PB) {
        float pb[PB];
#pragma unroll
        for (int b = 0; b < PB; ++b) {
            const int m = (mb0 + b) * 32 + lane;
            float p = 0.f;
            if (mb0 + b < mblocks && (MODE == 0 || m < M)) {
                const ST* sp = S + static_cast<int64_t>(r) * lds + m;
#pragma unroll 4
                for (int s = 0; s < splits; ++s) p += load_scalar<ST>(sp + s * split_stride);   // fixed order
            }
            pb[b] = p;
        }
#pragma unroll
        for (int b = 0; b < PB; ++b) {
            const int m0 = (mb0 + b) * 32;
            if (mb0 + b >= mblocks) break;
            const float p = pb[b];
            // Element pointer of this lane's first chunk; each step moves on by SPW sub-tokens.
            WT* ptr = out + static_cast<int64_t>(r) * ldo + (static_cast<int64_t>(m0 + sub) * L + q) * 8;
#pragma unroll 8
            for (int it = 0; it < LPS; ++it, ptr += SPW * L * 8) {
                const int ms = it * SPW + sub;
                const float pm = __shfl_sync(kFull, p, ms);
                if (MODE != 0 && m0 + ms >= M) continue;
#pragma unroll
                for (int i = 0; i < CH; ++i) {
                    float y[8];
#pragma unroll
                    for (int e = 0; e < 8; ++e) y[e] = pm * vr[i][e];
                    if (MODE != 2) {
                        Out8<WT>::store(ptr + i * LPS * 8, y, beta);
                    } else {
                        const int col = ((m0 + ms) * L + q + LPS * i) * 8;
                        if (col + 8 <= D) {
                            Out8<WT>::store(ptr + i * LPS * 8, y, beta);
                        } else {
#pragma unroll
                            for (int e = 0; e < 8; ++e)
                                if (col + e < D) {
                                    WT* pe = ptr + i * LPS * 8 + e;
                                    float f = y[e];
                                    if (beta) f += Elem<WT>::load(pe);
                                    Elem<WT>::store(pe, f);
                                }
                        }
                    }
                }
            }
        }
    }
}

template <int LPS, int CH, typename ST, typename WT>
int launch_mode(int mode, int grid, const void* S, int splits, int64_t split_stride, int lds, const float* v,
                int R, int D, int M, int mblocks, void* out, int64_t ldo, int beta, cudaStream_t stream)
{
    const ST* s = static_cast<const ST*>(S);
    WT* o = static_cast<WT*>(out);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(grid), 1, 1);
    cfg.blockDim = dim3(kStreamThreads, 1, 1);
    cfg.stream = stream;
    cudaLaunchAttribute attr = pdl_attribute();
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    cudaError_t e;
    if (mode == 0)
        e = cudaLaunchKernelEx(&cfg, expand_rows_vec_kernel<LPS, CH, 0, ST, WT>, s, splits, split_stride, lds, v, R, D, M, mblocks, o, ldo, beta);
    else if (mode == 1)
        e = cudaLaunchKernelEx(&cfg, expand_rows_vec_kernel<LPS, CH, 1, ST, WT>, s, splits, split_stride, lds, v, R, D, M, mblocks, o, ldo, beta);
    else
        e = cudaLaunchKernelEx(&cfg, expand_rows_vec_kernel<LPS, CH, 2, ST, WT>, s, splits, split_stride, lds, v, R, D, M, mblocks, o, ldo, beta);
    if (e != cudaSuccess) {
        cudaGetLastError();
        return VELORA_ERR_CUDA;
    }
    return after_launch();
}

template <typename ST, typename WT>
int launch_shape(int lps, int ch, int mode, int grid, const void* S, int splits, int64_t split_stride, int lds,
                 const float* v, int R, int D, int M, int mblocks, void* out, int64_t ldo, int beta, cudaStream_t stream)
{
#define VELORA_EXPAND_CASE(LPSV, CHV)                                                                          \
    if (lps == LPSV && ch == CHV)                                                                              \
        return launch_mode<LPSV, CHV, ST, WT>(mode, grid, S, splits, split_stride, lds, v, R, D, M, mblocks, out, ldo, beta, stream)
    VELORA_EXPAND_CASE(1, 1);
    VELORA_EXPAND_CASE(2, 1);
    VELORA_EXPAND_CASE(4, 1);
    VELORA_EXPAND_CASE(8, 1);
    VELORA_EXPAND_CASE(16, 1);
    VELORA_EXPAND_CASE(32, 1);
    VELORA_EXPAND_CASE(32, 2);
    VELORA_EXPAND_CASE(32, 4);
#undef VELORA_EXPAND_CASE
    return VELORA_ERR_UNSUPPORTED;
}

}  // namespace

int launch_expand_rows_vec(const void* S, int s_dtype, int splits, int64_t split_stride, int64_t lds, const float* v,
                           int64_t R, int64_t D, int Dsub, void* out, int out_dtype, int64_t ldo, int beta,
                           cudaStream_t stream)
{
    if (Dsub % 8) return VELORA_ERR_UNSUPPORTED;
    const int L = Dsub / 8;
    if (L < 1 || L > 128 || (L & (L - 1))) return VELORA_ERR_UNSUPPORTED;
    if (!aligned16(out) || (ldo * static_cast<int64_t>(dtype_size(out_dtype))) % 16) return VELORA_ERR_UNSUPPORTED;
    if (R < 1 || R >= (1 << 30) || lds >= (1 << 30) || D >= (1 << 30)) return VELORA_ERR_UNSUPPORTED;
    if ((s_dtype == VELORA_BF16 || s_dtype == VELORA_FP8_E4M3) && out_dtype != VELORA_BF16) return VELORA_ERR_UNSUPPORTED;
    const int lps = L < 32 ? L : 32, ch = L / lps;
    const int M = static_cast<int>(ceil_div64(D, Dsub));
    const int mblocks = (M + 31) / 32;
    const int mode = (D % Dsub) ? 2 : ((M % 32) ? 1 : 0);
    DeviceInfo di;
    int rc = device_info(&di);
    if (rc != VELORA_OK) return rc;
    int64_t ctas = ceil_div64(R, kStreamThreads / 32);
    const int64_t cap = static_cast<int64_t>(di.sm_count) * kStreamCtasPerSm;
    if (ctas > cap) ctas = cap;
    const int grid = static_cast<int>(ctas < 1 ? 1 : ctas);
    const int r = static_cast<int>(R), d = static_cast<int>(D), ld = static_cast<int>(lds);
    if (s_dtype == VELORA_BF16)
        return launch_shape<__nv_bfloat16, __nv_bfloat16>(lps, ch, mode, grid, S, splits, split_stride, ld, v, r, d, M, mblocks, out, ldo, beta, stream);
    if (s_dtype == VELORA_FP8_E4M3)
        return launch_shape<e4m3_t, __nv_bfloat16>(lps, ch, mode, grid, S, splits, split_stride, ld, v, r, d, M, mblocks, out, ldo, beta, stream);
    if (out_dtype == VELORA_BF16)
        return launch_shape<float, __nv_bfloat16>(lps, ch, mode, grid, S, splits, split_stride, ld, v, r, d, M, mblocks, out, ldo, beta, stream);
    return launch_shape<float, float>(lps, ch, mode, grid, S, splits, split_stride, ld, v, r, d, M, mblocks, out, ldo, beta, stream);
}

}  // namespace velora
