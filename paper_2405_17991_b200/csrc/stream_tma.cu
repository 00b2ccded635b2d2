// TMA-staged streaming kernels: compress (arxiv 2405.17991, Section 3.1 Eq. 1) and the partial sums
// of init_v (Section 3.2) for bf16 inputs with 16-byte aligned rows and Dsub in {8, 16, ..., 256}.
//
// These kernels are bound by the HBM read of X, so the design goal is bytes in flight, not math.
// Two persistent CTAs per SM each keep a ring of three 32 KB stages in shared memory.  A single producer
// thread issues 2-d TMA tile loads (boxes of 16 rows x 256 columns, no swizzle) that complete on
// mbarriers, so up to 192 KB per SM are in flight regardless of what the consumers do.  Sixteen consumer
// warps per CTA read the landed tiles with conflict-free 16-byte shared-memory loads (a warp instruction reads
// one 512-byte tile row), form the dot products with a slice of v held in registers, reduce over the
// Dsub/8 lanes of a sub-token with xor shuffles and write Z.  Rows beyond N and columns beyond D are
// zero-filled by TMA, which is exactly the zero extension of a ragged last sub-token: the kernel has
// no bounds checks on its loads.  Every barrier wait is bounded (one second) and a timeout is
// recorded in a device word that velora_device_error() reads.
#include "gemm_tc.cuh"
#include "tc_common.cuh"

namespace velora {

using namespace tc;

namespace {

constexpr int ST_R = 16;                          // rows per box
constexpr int ST_COLS = 256;                      // columns per box (512 bytes)
constexpr int ST_NB = 4;                          // boxes per stage
constexpr int ST_BOX_BYTES = ST_R * ST_COLS * 2;  // 8 KB
constexpr int ST_STAGE_BYTES = ST_NB * ST_BOX_BYTES;
constexpr int ST_STAGES = 3;                      // per CTA; two CTAs share an SM
constexpr int ST_CONSUMERS = 16;                  // warps, one tile row each
constexpr int ST_THREADS = (ST_CONSUMERS + 1) * 32;
constexpr int ST_ROWS_PER_WARP = ST_R / ST_CONSUMERS;
constexpr size_t ST_SMEM = 1024 + static_cast<size_t>(ST_STAGES) * ST_STAGE_BYTES + 256;

__device__ int g_stream_error = 0;

__device__ __forceinline__ uint4 lds128(uint32_t addr)
{
    uint4 r;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "r"(addr));
    return r;
}

template <typename ZT> __device__ __forceinline__ void put_z(ZT* p, float z);
template <> __device__ __forceinline__ void put_z<float>(float* p, float z) { *p = z; }
template <> __device__ __forceinline__ void put_z<__nv_bfloat16>(__nv_bfloat16* p, float z) { *p = __float2bfloat16_rn(z); }

// LPS = Dsub / 8 lanes per sub-token (power of two, <= 32).  INIT = false: compress, writes Z.
// INIT = true: init_v partial sums, writes partials[blockIdx.x][Dsub].
template <int LPS, bool INIT, typename ZT>
__global__ void __launch_bounds__(ST_THREADS, 2)
stream_tma_kernel(const __grid_constant__ CUtensorMap tmX, int N, int M, int ncb, int cgroups, int units,
                  const float* __restrict__ v, ZT* __restrict__ Z, int64_t ldz, float* __restrict__ partials)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (base - raw);
    uint8_t* tail = smem + ST_STAGES * ST_STAGE_BYTES;
    const uint32_t bars = base + ST_STAGES * ST_STAGE_BYTES;
    const uint32_t full = bars, empty = bars + 8 * ST_STAGES;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tail + 16 * ST_STAGES);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int s = 0; s < ST_STAGES; ++s) {
            mbar_init(full + 8 * s, 1);
            mbar_init(empty + 8 * s, ST_CONSUMERS);
        }
        *abort_flag = 0;
        fence_mbar_init();
        prefetch_tensormap(&tmX);
    }
    __syncthreads();

    bool failed = false;
    float acc[8];                                 // INIT: running sums at this lane's fixed positions
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[e] = 0.f;

    if (warp == 0) {
        // ------------------------------------------------ producer
        if (lane == 0) {
            int it = 0;
            for (int u = blockIdx.x; u < units; u += gridDim.x, ++it) {
                const int s = it % ST_STAGES;
                const uint32_t ph = (it / ST_STAGES) & 1u;
                if (!mbar_wait(empty + 8 * s, ph ^ 1u, abort_flag)) { failed = true; break; }
                const int rb = u / cgroups, cg = u - rb * cgroups;
                const int nb = (ncb - cg * ST_NB < ST_NB) ? ncb - cg * ST_NB : ST_NB;
                mbar_arrive_expect_tx(full + 8 * s, static_cast<uint32_t>(nb * ST_BOX_BYTES));
                for (int b = 0; b < nb; ++b)
                    tma_load_2d(base + s * ST_STAGE_BYTES + b * ST_BOX_BYTES, &tmX, full + 8 * s,
                                (cg * ST_NB + b) * ST_COLS, rb * ST_R);
            }
            if (failed) {
                *abort_flag = 1;
                const int back = it < ST_STAGES ? it : ST_STAGES;     // own copies still in flight
                for (int j = 1; j <= back; ++j) {
                    const int jt = it - j;
                    const unsigned long long t0 = globaltimer_ns();
                    while (!mbar_try_wait(full + 8 * (jt % ST_STAGES), (jt / ST_STAGES) & 1u))
                        if (globaltimer_ns() - t0 > kWaitLimitNs) break;
                }
            }
        }
    } else {
        // ------------------------------------------------ consumers
        const int cw = warp - 1;
        const int q = lane & (LPS - 1);           // this lane's 8 elements sit at positions 8q .. 8q+7
        float vr[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) vr[e] = INIT ? 0.f : __ldg(v + 8 * q + e);
        constexpr int SUBS_PER_BOX = 32 / LPS;    // sub-tokens per 256-column tile row

        int it = 0;
        for (int u = blockIdx.x; u < units; u += gridDim.x, ++it) {
            const int s = it % ST_STAGES;
            const uint32_t ph = (it / ST_STAGES) & 1u;
            if (!mbar_wait(full + 8 * s, ph, abort_flag)) { failed = true; break; }
            const int rb = u / cgroups, cg = u - rb * cgroups;
            const int nb = (ncb - cg * ST_NB < ST_NB) ? ncb - cg * ST_NB : ST_NB;
            const uint32_t st = base + s * ST_STAGE_BYTES + lane * 16;

            static_assert(ST_ROWS_PER_WARP == 1 && ST_NB == 4, "the reduction below handles four boxes of one row");
            const int row = rb * ST_R + cw;
            uint4 d[ST_NB];
#pragma unroll
            for (int b = 0; b < ST_NB; ++b)
                d[b] = (b < nb) ? lds128(st + b * ST_BOX_BYTES + cw * (ST_COLS * 2)) : make_uint4(0u, 0u, 0u, 0u);
            float dot[ST_NB];
#pragma unroll
            for (int b = 0; b < ST_NB; ++b) {
                float x[8];
                x[0] = bf16_lo(d[b].x); x[1] = bf16_hi(d[b].x);
                x[2] = bf16_lo(d[b].y); x[3] = bf16_hi(d[b].y);
                x[4] = bf16_lo(d[b].z); x[5] = bf16_hi(d[b].z);
                x[6] = bf16_lo(d[b].w); x[7] = bf16_hi(d[b].w);
                if (INIT) {
#pragma unroll
                    for (int e = 0; e < 8; ++e) acc[e] += x[e];
                } else {
                    dot[b] = 0.f;
#pragma unroll
                    for (int e = 0; e < 8; ++e) dot[b] = fmaf(x[e], vr[e], dot[b]);
                }
            }
            if (!INIT) {
                const int mbase = cg * ST_NB * SUBS_PER_BOX + lane / LPS;
                if (LPS >= 4) {
                    // Four sums over LPS lanes in four shuffles: the halves of the lane group trade two of
                    // their four values, then the quarters trade one, then a plain butterfly finishes; the
                    // lane ends up holding the complete sum of box `mine`.
                    const bool hi1 = (lane & (LPS / 2)) != 0;
                    float k0 = hi1 ? dot[2] : dot[0], k1 = hi1 ? dot[3] : dot[1];
                    const float s0 = hi1 ? dot[0] : dot[2], s1 = hi1 ? dot[1] : dot[3];
                    k0 += __shfl_xor_sync(0xffffffffu, s0, LPS / 2);
                    k1 += __shfl_xor_sync(0xffffffffu, s1, LPS / 2);
                    const bool hi2 = (lane & (LPS / 4)) != 0;
                    float k = hi2 ? k1 : k0;
                    const float sx = hi2 ? k0 : k1;
                    k += __shfl_xor_sync(0xffffffffu, sx, LPS / 4);
#pragma unroll
                    for (int off = LPS / 8; off >= 1; off >>= 1) k += __shfl_xor_sync(0xffffffffu, k, off);
                    const int mine = (hi1 ? 2 : 0) + (hi2 ? 1 : 0);
                    const int m = mbase + mine * SUBS_PER_BOX;
                    if ((lane & (LPS / 4 - 1)) == 0 && mine < nb && row < N && m < M)
                        put_z<ZT>(Z + static_cast<int64_t>(row) * ldz + m, k);
                } else {
#pragma unroll
                    for (int b = 0; b < ST_NB; ++b) {
                        float k = dot[b];
#pragma unroll
                        for (int off = LPS / 2; off >= 1; off >>= 1) k += __shfl_xor_sync(0xffffffffu, k, off);
                        const int m = mbase + b * SUBS_PER_BOX;
                        if (q == 0 && b < nb && row < N && m < M) put_z<ZT>(Z + static_cast<int64_t>(row) * ldz + m, k);
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(empty + 8 * s);   // this warp has read its rows of the stage
        }
        if (failed) *abort_flag = 1;
    }
    if (failed) atomicExch(&g_stream_error, VELORA_ERR_TIMEOUT);

    if (INIT) {
        // Fixed-order reduction over the consumer lanes that share a position, through the (now idle) ring.
        __syncthreads();
        float* sacc = reinterpret_cast<float*>(smem);           // [ST_CONSUMERS * 32][8]
        if (warp > 0) {
#pragma unroll
            for (int e = 0; e < 8; ++e) sacc[((warp - 1) * 32 + lane) * 8 + e] = acc[e];
        }
        __syncthreads();
        const int Dsub = LPS * 8;
        for (int j = threadIdx.x; j < Dsub; j += ST_THREADS) {
            const int qq = j >> 3, e = j & 7;
            float sum = 0.f;
            for (int t = qq; t < ST_CONSUMERS * 32; t += LPS) sum += sacc[t * 8 + e];
            partials[static_cast<int64_t>(blockIdx.x) * Dsub + j] = sum;
        }
    }
}

struct StreamPlan {
    bool ok;
    int lps, M, ncb, cgroups, units, grid;
};

StreamPlan plan_stream(const void* X, int64_t N, int64_t D, int64_t ldx, int Dsub, int sm_count)
{
    StreamPlan p{};
    if (Dsub < 8 || Dsub > 256 || (Dsub & (Dsub - 1))) return p;
    if (!tc_operand_ok(X, ldx) || N < 1 || N > (1 << 30) || D > (1 << 30)) return p;
    p.lps = Dsub / 8;
    p.M = static_cast<int>(ceil_div64(D, Dsub));
    p.ncb = static_cast<int>(ceil_div64(D, ST_COLS));
    p.cgroups = (p.ncb + ST_NB - 1) / ST_NB;
    const int64_t units = ceil_div64(N, ST_R) * p.cgroups;
    if (units > (1 << 30)) return p;
    p.units = static_cast<int>(units);
    p.grid = p.units < 2 * sm_count ? p.units : 2 * sm_count;
    p.ok = true;
    return p;
}

template <int LPS, bool INIT, typename ZT>
int launch_stream(const CUtensorMap& tm, const StreamPlan& p, int N, const float* v, ZT* Z, int64_t ldz,
                  float* partials, cudaStream_t stream)
{
    static bool configured[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return VELORA_ERR_CUDA;
    auto kern = stream_tma_kernel<LPS, INIT, ZT>;
    if (!configured[dev]) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(ST_SMEM)) != cudaSuccess)
            return VELORA_ERR_CUDA;
        configured[dev] = true;
    }
    kern<<<p.grid, ST_THREADS, ST_SMEM, stream>>>(tm, N, p.M, p.ncb, p.cgroups, p.units, v, Z, ldz, partials);
    return after_launch();
}

#define VELORA_DISPATCH_LPS(LPSV, CALL)                \
    switch (LPSV) {                                    \
        case 1: return CALL(1);                        \
        case 2: return CALL(2);                        \
        case 4: return CALL(4);                        \
        case 8: return CALL(8);                        \
        case 16: return CALL(16);                      \
        case 32: return CALL(32);                      \
        default: return VELORA_ERR_UNSUPPORTED;        \
    }

}  // namespace

int launch_compress_tma(const void* X, int64_t N, int64_t D, int64_t ldx, int Dsub, const float* v,
                        void* Z, int z_dtype, int64_t ldz, int* /*status*/, cudaStream_t stream)
{
    DeviceInfo di;
    int rc = device_info(&di);
    if (rc != VELORA_OK) return rc;
    if (static_cast<size_t>(di.smem_optin) < ST_SMEM) return VELORA_ERR_UNSUPPORTED;
    const StreamPlan p = plan_stream(X, N, D, ldx, Dsub, di.sm_count);
    if (!p.ok) return VELORA_ERR_UNSUPPORTED;
    CUtensorMap tm;
    rc = make_tmap_bf16_2d(&tm, X, D, N, ldx, ST_COLS, ST_R, false);
    if (rc != VELORA_OK) return rc;
    const int n = static_cast<int>(N);
    if (z_dtype == VELORA_F32) {
#define CALL_F32(L) launch_stream<L, false, float>(tm, p, n, v, static_cast<float*>(Z), ldz, nullptr, stream)
        VELORA_DISPATCH_LPS(p.lps, CALL_F32)
#undef CALL_F32
    }
#define CALL_BF16(L) launch_stream<L, false, __nv_bfloat16>(tm, p, n, v, static_cast<__nv_bfloat16*>(Z), ldz, nullptr, stream)
    VELORA_DISPATCH_LPS(p.lps, CALL_BF16)
#undef CALL_BF16
}

int launch_init_v_partials_tma(const void* X, int64_t N, int64_t D, int64_t ldx, int Dsub,
                               float* partials, int max_partials, int* num_partials, int* /*status*/,
                               cudaStream_t stream)
{
    DeviceInfo di;
    int rc = device_info(&di);
    if (rc != VELORA_OK) return rc;
    if (static_cast<size_t>(di.smem_optin) < ST_SMEM) return VELORA_ERR_UNSUPPORTED;
    StreamPlan p = plan_stream(X, N, D, ldx, Dsub, di.sm_count);
    if (!p.ok) return VELORA_ERR_UNSUPPORTED;
    if (p.grid > max_partials) p.grid = max_partials;
    CUtensorMap tm;
    rc = make_tmap_bf16_2d(&tm, X, D, N, ldx, ST_COLS, ST_R, false);
    if (rc != VELORA_OK) return rc;
    *num_partials = p.grid;
    const int n = static_cast<int>(N);
#define CALL_INIT(L) launch_stream<L, true, float>(tm, p, n, nullptr, static_cast<float*>(nullptr), 0, partials, stream)
    VELORA_DISPATCH_LPS(p.lps, CALL_INIT)
#undef CALL_INIT
}

int read_and_clear_stream_error(cudaStream_t stream)
{
    int word = 0;
    if (cudaMemcpyFromSymbolAsync(&word, g_stream_error, sizeof(int), 0, cudaMemcpyDeviceToHost, stream) != cudaSuccess)
        return VELORA_ERR_CUDA;
    if (cudaStreamSynchronize(stream) != cudaSuccess) return VELORA_ERR_CUDA;
    if (word != 0) {
        const int zero = 0;
        if (cudaMemcpyToSymbolAsync(g_stream_error, &zero, sizeof(int), 0, cudaMemcpyHostToDevice, stream) != cudaSuccess)
            return VELORA_ERR_CUDA;
        cudaStreamSynchronize(stream);
        return VELORA_ERR_TIMEOUT;
    }
    return VELORA_OK;
}

}  // namespace velora
