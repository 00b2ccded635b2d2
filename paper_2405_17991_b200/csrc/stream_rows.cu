// Row-streaming kernels for bf16 inputs with 16-byte aligned rows and Dsub = 8 * 2^k (8 .. 1024):
// compress (arxiv 2405.17991, Section 3.1 Eq. 1) and the partial sums of init_v (Section 3.2).
//
// Both are bound by the one pass over X, so the kernel is as plain as a read stream can be: a warp owns a
// token row and walks it in rounds of U = 8 load instructions, each of which reads one contiguous 512-byte
// span (32 lanes x 16 bytes = 32 chunks of 8 elements); all eight are issued before the first is used.  With
// 8 CTAs of 256 threads per SM that keeps 128-256 KB per SM in flight with no shared memory, no barrier and
// no set-up to speak of -- measured against a TMA-fed shared-memory ring (three 32 KB stages per CTA, two
// CTAs per SM) this form is faster by about 4 us per call on a 67 MB input and by 2 us on a 180 MB one, and
// runs within a few per cent of a kernel that only reads.
//
// A sub-token of length Dsub = 8 * L covers L consecutive chunks: LPS = min(L, 32) adjacent lanes hold one
// part of it, and for L > 32 the CH = L / 32 consecutive load instructions of a round complete it.  A lane's
// position inside the sub-token never changes (rounds advance by multiples of 32 * CH chunks), so its slice
// of v lives in registers.  compress: fp32 products and sums, xor-shuffle reduction over the LPS lanes,
// the lane at position 0 stores Z[row, m].  init_v: the lane adds what it loads into 8 * CH running sums; the
// CTA then adds the sums of the lanes that share a position in a fixed order and writes one row of partials.
//
// Columns at or beyond D count as zeros: chunks past the row's end are not loaded and a last chunk that
// straddles D is masked, which is the zero extension of a ragged last sub-token.
#include "common.cuh"
#include "gemm_tc.cuh"

namespace velora {
namespace {

constexpr int RW_THREADS = 256;
constexpr int RW_WARPS = RW_THREADS / 32;
constexpr int RW_U = 8;                          // load instructions in flight per warp

template <typename ZT> __device__ __forceinline__ void put_z(ZT* p, float z);
template <> __device__ __forceinline__ void put_z<float>(float* p, float z) { *p = z; }
template <> __device__ __forceinline__ void put_z<__nv_bfloat16>(__nv_bfloat16* p, float z) { *p = __float2bfloat16_rn(z); }
template <> __device__ __forceinline__ void put_z<e4m3_t>(e4m3_t* p, float z) { *p = float_to_e4m3(z); }

// Chunk c of a row: 8 elements; zeros beyond column D.  d8 = D / 8 whole chunks, tail = D % 8.
__device__ __forceinline__ uint4 load_row_chunk(const uint4* __restrict__ row, int c, int d8, int tail)
{
    if (c < d8) return __ldcs(row + c);
    uint4 x = make_uint4(0u, 0u, 0u, 0u);
    if (c == d8 && tail) {
        x = __ldcs(row + c);                     // inside the row's pitch (a multiple of 8 elements)
        uint32_t w[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            if (2 * i >= tail) w[i] = 0u;
            else if (2 * i + 1 >= tail) w[i] &= 0x0000ffffu;
        }
        x = make_uint4(w[0], w[1], w[2], w[3]);
    }
    return x;
}

template <int LPS, int CH, bool INIT, typename ZT>
__global__ void __launch_bounds__(RW_THREADS)
stream_rows_kernel(const uint4* __restrict__ X, int N, int D, int64_t ldx_chunks, int M,
                   const float* __restrict__ v, ZT* __restrict__ Z, int64_t ldz, float* __restrict__ partials)
{
    static_assert(CH == 1 || LPS == 32, "several chunks per lane only for sub-tokens wider than a warp's span");
    static_assert(RW_U % CH == 0, "a round must hold whole sub-tokens");
    // Programmatic stream serialisation (common.cuh): resident early, nothing read or written before the wait.
    pdl_trigger();
    pdl_wait();
    const int lane = threadIdx.x & 31;
    const int q = lane & (LPS - 1);               // position of this lane's chunk inside a 32-chunk part
    constexpr int SPI = 32 / LPS;                 // sub-tokens per load instruction (CH == 1)
    const int d8 = D >> 3, tail = D & 7;
    const int cpr = d8 + (tail ? 1 : 0);          // chunks that hold data

    float vr[CH][8];                              // compress: slice of v; init_v: running sums
#pragma unroll
    for (int i = 0; i < CH; ++i)
#pragma unroll
        for (int e = 0; e < 8; ++e) vr[i][e] = INIT ? 0.f : __ldg(v + 8 * (q + LPS * i) + e);

    const int warps = gridDim.x * RW_WARPS;
    for (int row = blockIdx.x * RW_WARPS + (threadIdx.x >> 5); row < N; row += warps) {
        const uint4* rp = X + static_cast<int64_t>(row) * ldx_chunks;
        ZT* zrow = INIT ? nullptr : Z + static_cast<int64_t>(row) * ldz;
        for (int c0 = 0; c0 < cpr; c0 += 32 * RW_U) {
            uint4 d[RW_U];
#pragma unroll
            for (int u = 0; u < RW_U; ++u) d[u] = load_row_chunk(rp, c0 + 32 * u + lane, d8, tail);
            float part = 0.f;                     // CH > 1: sum over the parts of one sub-token so far
#pragma unroll
            for (int u = 0; u < RW_U; ++u) {
                const int i = u % CH;             // which part of the sub-token this instruction read
                float x[8];
                x[0] = bf16_lo(d[u].x); x[1] = bf16_hi(d[u].x);
                x[2] = bf16_lo(d[u].y); x[3] = bf16_hi(d[u].y);
                x[4] = bf16_lo(d[u].z); x[5] = bf16_hi(d[u].z);
                x[6] = bf16_lo(d[u].w); x[7] = bf16_hi(d[u].w);
                if (INIT) {
#pragma unroll
                    for (int e = 0; e < 8; ++e) vr[i][e] += x[e];
                } else {
                    float a0 = x[0] * vr[i][0], a1 = x[1] * vr[i][1];
                    a0 = fmaf(x[2], vr[i][2], a0); a1 = fmaf(x[3], vr[i][3], a1);
                    a0 = fmaf(x[4], vr[i][4], a0); a1 = fmaf(x[5], vr[i][5], a1);
                    a0 = fmaf(x[6], vr[i][6], a0); a1 = fmaf(x[7], vr[i][7], a1);
                    part = (i == 0) ? a0 + a1 : part + (a0 + a1);
                    if (i == CH - 1) {
                        float k = part;
#pragma unroll
                        for (int off = LPS / 2; off >= 1; off >>= 1) k += __shfl_xor_sync(0xffffffffu, k, off);
                        // first chunk of the sub-token: c0 + 32 * (u - i); its index m = that / (LPS * CH) (+ lane / LPS)
                        const int m = (c0 + 32 * (u - i)) / (LPS * CH) + (CH == 1 ? lane / LPS : 0);
                        if (q == 0 && m < M) put_z<ZT>(zrow + m, k);
                    }
                }
            }
        }
    }

    if constexpr (INIT) {
        // Fixed-order sum over the lanes of the CTA that share a position.
        __shared__ float sacc[RW_THREADS * 8 * CH];
#pragma unroll
        for (int i = 0; i < CH; ++i)
#pragma unroll
            for (int e = 0; e < 8; ++e) sacc[(threadIdx.x * CH + i) * 8 + e] = vr[i][e];
        __syncthreads();
        constexpr int Dsub = 8 * LPS * CH;
        for (int j = threadIdx.x; j < Dsub; j += RW_THREADS) {
            const int chunk = j >> 3, e = j & 7;
            const int qq = chunk % LPS, i = chunk / LPS;
            float sum = 0.f;
            for (int t = qq; t < RW_THREADS; t += LPS) sum += sacc[(t * CH + i) * 8 + e];
            partials[static_cast<int64_t>(blockIdx.x) * Dsub + j] = sum;
        }
    }
}

struct RowsPlan {
    bool ok;
    int lps, ch, M, grid;
};

RowsPlan plan_rows(const void* X, int64_t N, int64_t D, int64_t ldx, int Dsub, int sm_count, int max_grid)
{
    RowsPlan p{};
    if (Dsub < 8 || Dsub > 1024 || (Dsub & (Dsub - 1))) return p;
    if (!aligned16(X) || ldx % 8 || ldx < ((D + 7) / 8) * 8) return p;
    if (N < 1 || N >= (1 << 30) || D >= (1 << 30)) return p;
    const int L = Dsub / 8;
    p.lps = L < 32 ? L : 32;
    p.ch = L / p.lps;
    p.M = static_cast<int>(ceil_div64(D, Dsub));
    int64_t grid = ceil_div64(N, RW_WARPS);
    const int64_t cap = static_cast<int64_t>(sm_count) * kStreamCtasPerSm;
    if (grid > cap) grid = cap;
    if (max_grid > 0 && grid > max_grid) grid = max_grid;
    p.grid = static_cast<int>(grid);
    p.ok = true;
    return p;
}

template <int LPS, int CH, bool INIT, typename ZT>
int launch_rows(const RowsPlan& p, const void* X, int64_t N, int64_t D, int64_t ldx, const float* v, ZT* Z, int64_t ldz,
                float* partials, cudaStream_t stream)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(p.grid), 1, 1);
    cfg.blockDim = dim3(RW_THREADS, 1, 1);
    cfg.stream = stream;
    cudaLaunchAttribute attr = pdl_attribute();
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, stream_rows_kernel<LPS, CH, INIT, ZT>, static_cast<const uint4*>(X), static_cast<int>(N),
                           static_cast<int>(D), ldx / 8, p.M, v, Z, ldz, partials) != cudaSuccess) {
        cudaGetLastError();
        return VELORA_ERR_CUDA;
    }
    return after_launch();
}

template <bool INIT, typename ZT>
int dispatch_rows(const RowsPlan& p, const void* X, int64_t N, int64_t D, int64_t ldx, const float* v, ZT* Z, int64_t ldz,
                  float* partials, cudaStream_t stream)
{
#define VELORA_ROWS_CASE(LPSV, CHV) \
    if (p.lps == LPSV && p.ch == CHV) return launch_rows<LPSV, CHV, INIT, ZT>(p, X, N, D, ldx, v, Z, ldz, partials, stream)
    VELORA_ROWS_CASE(1, 1);
    VELORA_ROWS_CASE(2, 1);
    VELORA_ROWS_CASE(4, 1);
    VELORA_ROWS_CASE(8, 1);
    VELORA_ROWS_CASE(16, 1);
    VELORA_ROWS_CASE(32, 1);
    VELORA_ROWS_CASE(32, 2);
    VELORA_ROWS_CASE(32, 4);
#undef VELORA_ROWS_CASE
    return VELORA_ERR_UNSUPPORTED;
}

}  // namespace

int launch_compress_rows(const void* X, int64_t N, int64_t D, int64_t ldx, int Dsub, const float* v,
                         void* Z, int z_dtype, int64_t ldz, cudaStream_t stream)
{
    DeviceInfo di;
    const int rc = device_info(&di);
    if (rc != VELORA_OK) return rc;
    const RowsPlan p = plan_rows(X, N, D, ldx, Dsub, di.sm_count, 0);
    if (!p.ok) return VELORA_ERR_UNSUPPORTED;
    if (z_dtype == VELORA_F32)
        return dispatch_rows<false, float>(p, X, N, D, ldx, v, static_cast<float*>(Z), ldz, nullptr, stream);
    if (z_dtype == VELORA_FP8_E4M3)
        return dispatch_rows<false, e4m3_t>(p, X, N, D, ldx, v, static_cast<e4m3_t*>(Z), ldz, nullptr, stream);
    return dispatch_rows<false, __nv_bfloat16>(p, X, N, D, ldx, v, static_cast<__nv_bfloat16*>(Z), ldz, nullptr, stream);
}

int launch_init_v_partials_rows(const void* X, int64_t N, int64_t D, int64_t ldx, int Dsub,
                                float* partials, int max_partials, int* num_partials, cudaStream_t stream)
{
    DeviceInfo di;
    const int rc = device_info(&di);
    if (rc != VELORA_OK) return rc;
    // Four CTAs of this kernel are resident per SM (its registers), so a grid of four per SM is one wave of CTAs
    // that each walk a few rows; a larger grid would only add partial rows for the finalize kernel to add up.
    int cap = di.sm_count * 4;
    if (max_partials > 0 && cap > max_partials) cap = max_partials;
    const RowsPlan p = plan_rows(X, N, D, ldx, Dsub, di.sm_count, cap);
    if (!p.ok) return VELORA_ERR_UNSUPPORTED;
    *num_partials = p.grid;
    return dispatch_rows<true, float>(p, X, N, D, ldx, nullptr, static_cast<float*>(nullptr), 0, partials, stream);
}

}  // namespace velora
