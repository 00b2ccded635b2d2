// HBM-bound streaming kernels of the VeLoRA path: init_v, compress, reconstruct and the expansion
// of the factored weight gradient (arxiv 2405.17991, Section 3.1 Eq. 1 / Eq. 2, Section 3.2).
//
// The common case (bf16 rows that are 16-byte aligned, Dsub = 8 * 2^k) is served by stream_rows.cu
// (compress, init_v) and expand_kernels.cu (reconstruct, expansion of the factored weight gradient).  This
// file holds the kernels for everything else and the routing between all of them.
//
// Element kernels cover everything else (fp32 data, Dsub not a multiple of 8, unaligned rows) with
// the same arithmetic, one element per lane.
#include "common.cuh"
#include "gemm_tc.cuh"

namespace velora {

namespace {

constexpr unsigned kFull = 0xffffffffu;

template <typename ZT> __device__ __forceinline__ void store_z(ZT* p, float z);
template <> __device__ __forceinline__ void store_z<float>(float* p, float z) { *p = z; }
template <> __device__ __forceinline__ void store_z<__nv_bfloat16>(__nv_bfloat16* p, float z) { *p = __float2bfloat16_rn(z); }
template <> __device__ __forceinline__ void store_z<e4m3_t>(e4m3_t* p, float z) { *p = float_to_e4m3(z); }

template <typename ZT> __device__ __forceinline__ float load_z(const ZT* p);
template <> __device__ __forceinline__ float load_z<float>(const float* p) { return __ldg(p); }
template <> __device__ __forceinline__ float load_z<__nv_bfloat16>(const __nv_bfloat16* p)
{
    return __bfloat162float(*p);
}
template <> __device__ __forceinline__ float load_z<e4m3_t>(const e4m3_t* p) { return e4m3_to_float(*p); }

// ------------------------------------------------------------------ init_v (element-wise) partial sums
// CTA b owns rows [b*rows_per_cta, ...).  For each block of up to 256 positions j, thread t adds
// X[row, m*Dsub + j] over its rows and over m = slot, slot + slots, ...; slots share a position and are
// summed in fixed order through shared memory.
template <typename XT>
__global__ void __launch_bounds__(kStreamThreads)
init_v_partial_elem_kernel(const XT* __restrict__ X, int64_t N, int D, int64_t ldx, int Dsub, int M,
                           int64_t rows_per_cta, float* __restrict__ partials /* [gridDim.x][Dsub] */)
{
    __shared__ float sred[kStreamThreads];
    const int64_t r0 = blockIdx.x * rows_per_cta;
    const int64_t r1 = (r0 + rows_per_cta < N) ? r0 + rows_per_cta : N;
    for (int j0 = 0; j0 < Dsub; j0 += kStreamThreads) {
        const int width = (Dsub - j0 < kStreamThreads) ? Dsub - j0 : kStreamThreads;
        const int slots = kStreamThreads / width;
        const int j = j0 + threadIdx.x % width;
        const int slot = threadIdx.x / width;
        float acc = 0.f;
        if (slot < slots)
            for (int64_t r = r0; r < r1; ++r)
                for (int m = slot; m < M; m += slots) {
                    const int d = m * Dsub + j;
                    if (d < D) acc += Elem<XT>::load(X + r * ldx + d);
                }
        sred[threadIdx.x] = acc;
        __syncthreads();
        if (threadIdx.x < width) {
            float s = 0.f;
            for (int k = 0; k < slots; ++k) s += sred[k * width + threadIdx.x];
            partials[static_cast<int64_t>(blockIdx.x) * Dsub + j] = s;
        }
        __syncthreads();
    }
}

// ------------------------------------------------------------------ init_v finalize: one CTA
// s[j] = sum over CTAs (fixed order, fp64), norm, v = s / ||s||.  status[0] = 0 ok, 1 degenerate.
// The partial rows come from up to ~1200 CTAs and sit in L2; adding them is a chain of load latencies, so
// the CTA is as wide as it can be (1024 threads) and a thread owns VEC consecutive positions (one 16-byte
// load for VEC = 4): for a block of up to 1024 position groups the threads split the partial rows into
// `slots` interleaved sets (eight independent loads in flight each), then one thread per group adds the
// sets in order.  The order depends only on the sizes, so the result is run-to-run identical.
constexpr int kFinThreads = 1024;

template <int VEC>
__global__ void __launch_bounds__(kFinThreads)
init_v_finalize_kernel(const float* __restrict__ partials, int num_partials, int Dsub,
                       float* __restrict__ v, int* __restrict__ status, int normalize)
{
    __shared__ double s_sum[VELORA_MAX_DSUB];
    __shared__ double s_red[kFinThreads * VEC];
    __shared__ double s_warp[kFinThreads / 32];
    const int groups = Dsub / VEC;                             // VEC divides Dsub (host)
    for (int g0 = 0; g0 < groups; g0 += kFinThreads) {
        const int width = (groups - g0 < kFinThreads) ? groups - g0 : kFinThreads;
        const int slots = kFinThreads / width;
        const int g = g0 + threadIdx.x % width;
        const int slot = threadIdx.x / width;
        double s[VEC];
#pragma unroll
        for (int e = 0; e < VEC; ++e) s[e] = 0.0;
        if (slot < slots)
            for (int b = slot; b < num_partials; b += 8 * slots) {     // eight loads in flight, added in order
                float x[8][VEC];
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    const int bu = b + u * slots;
                    const float* src = partials + static_cast<int64_t>(bu) * Dsub + g * VEC;
                    if (bu >= num_partials) {
#pragma unroll
                        for (int e = 0; e < VEC; ++e) x[u][e] = 0.f;
                    } else if (VEC == 4) {
                        const float4 t = *reinterpret_cast<const float4*>(src);
                        x[u][0] = t.x; x[u][1 % VEC] = t.y; x[u][2 % VEC] = t.z; x[u][3 % VEC] = t.w;
                    } else {
                        x[u][0] = *src;
                    }
                }
#pragma unroll
                for (int u = 0; u < 8; ++u)
#pragma unroll
                    for (int e = 0; e < VEC; ++e) s[e] += static_cast<double>(x[u][e]);
            }
#pragma unroll
        for (int e = 0; e < VEC; ++e) s_red[threadIdx.x * VEC + e] = s[e];
        __syncthreads();
        if (threadIdx.x < width) {
#pragma unroll
            for (int e = 0; e < VEC; ++e) {
                double t = 0.0;
                for (int k = 0; k < slots; ++k) t += s_red[(k * width + threadIdx.x) * VEC + e];
                s_sum[g * VEC + e] = t;
            }
        }
        __syncthreads();
    }
    if (!normalize) {                                          // the plain sub-token sum s (multi-rank use)
        for (int j = threadIdx.x; j < Dsub; j += kFinThreads) v[j] = static_cast<float>(s_sum[j]);
        return;
    }
    // ||s||^2: fixed tree (xor shuffles inside a warp, then the 32 warp sums in order)
    double sq = 0.0;
    for (int j = threadIdx.x; j < Dsub; j += kFinThreads) sq += s_sum[j] * s_sum[j];
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, off);
    if ((threadIdx.x & 31) == 0) s_warp[threadIdx.x >> 5] = sq;
    __syncthreads();
    double t = 0.0;
    for (int i = 0; i < kFinThreads / 32; ++i) t += s_warp[i];
    const double norm = sqrt(t);
    const bool ok = (norm > 0.0) && isfinite(norm);
    if (threadIdx.x == 0) status[0] = ok ? 0 : 1;
    if (ok)
        for (int j = threadIdx.x; j < Dsub; j += kFinThreads) v[j] = static_cast<float>(s_sum[j] / norm);
}

// Partial rows start 16-byte aligned and are Dsub floats apart: four positions per load when Dsub allows it.
inline void launch_init_v_finalize(const float* partials, int num_partials, int Dsub, float* v, int* status,
                                   int normalize, cudaStream_t stream)
{
    if (Dsub % 4 == 0 && aligned16(partials))
        init_v_finalize_kernel<4><<<1, kFinThreads, 0, stream>>>(partials, num_partials, Dsub, v, status, normalize);
    else
        init_v_finalize_kernel<1><<<1, kFinThreads, 0, stream>>>(partials, num_partials, Dsub, v, status, normalize);
}

// Running-average variant of the initialisation (Section 5, ablation on the initialisation strategy):
//   a <- (1 - rho) * a + rho * s / count,   v <- a / ||a||_2      (rho == 1: a is not read)
// s is this batch's sub-token sum.  One CTA; fp64 like init_v_finalize_kernel.  A zero or non-finite norm
// leaves a and v as they were and raises the workspace's sticky status word.
__global__ void __launch_bounds__(kStreamThreads)
update_v_kernel(const float* __restrict__ s, double inv_count, float rho, int Dsub,
                float* __restrict__ a, float* __restrict__ v, int* __restrict__ sticky)
{
    __shared__ double s_a[VELORA_MAX_DSUB];
    __shared__ double s_red[kStreamThreads];
    __shared__ double s_norm;
    double sq = 0.0;
    for (int j = threadIdx.x; j < Dsub; j += kStreamThreads) {
        const double mean = static_cast<double>(s[j]) * inv_count;
        const double an = (rho == 1.f) ? mean
                                       : (1.0 - static_cast<double>(rho)) * static_cast<double>(a[j]) + static_cast<double>(rho) * mean;
        s_a[j] = an;
        sq += an * an;
    }
    s_red[threadIdx.x] = sq;
    __syncthreads();
    if (threadIdx.x == 0) {
        double t = 0.0;
        for (int i = 0; i < kStreamThreads; ++i) t += s_red[i];
        s_norm = sqrt(t);
    }
    __syncthreads();
    const double norm = s_norm;
    if (!((norm > 0.0) && isfinite(norm))) {
        if (threadIdx.x == 0) atomicCAS(sticky, 0, VELORA_ERR_DEGENERATE_V);
        return;
    }
    for (int j = threadIdx.x; j < Dsub; j += kStreamThreads) {
        a[j] = static_cast<float>(s_a[j]);
        v[j] = static_cast<float>(s_a[j] / norm);
    }
}

// ------------------------------------------------------------------ compress / reconstruct (element-wise)
template <typename XT, typename ZT>
__global__ void __launch_bounds__(kStreamThreads)
compress_elem_kernel(const XT* __restrict__ X, int64_t N, int D, int64_t ldx, int Dsub, int M,
                     const float* __restrict__ v, ZT* __restrict__ Z, int64_t ldz)
{
    const int lane = threadIdx.x & 31;
    const int64_t warps = static_cast<int64_t>(gridDim.x) * (kStreamThreads / 32);
    const int64_t total = N * M;
    for (int64_t g = static_cast<int64_t>(blockIdx.x) * (kStreamThreads / 32) + (threadIdx.x >> 5); g < total; g += warps) {
        const int64_t row = g / M;
        const int m = static_cast<int>(g - row * M);
        const XT* xp = X + row * ldx + static_cast<int64_t>(m) * Dsub;
        const int len = (D - m * Dsub < Dsub) ? D - m * Dsub : Dsub;
        float acc = 0.f;
        for (int j = lane; j < len; j += 32) acc = fmaf(Elem<XT>::load(xp + j), __ldg(v + j), acc);
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) acc += __shfl_xor_sync(kFull, acc, off);
        if (lane == 0) store_z<ZT>(Z + row * ldz + m, acc);
    }
}

template <typename ZT, typename XT>
__global__ void __launch_bounds__(kStreamThreads)
reconstruct_elem_kernel(const ZT* __restrict__ Z, int64_t ldz, int64_t N, int D, int Dsub,
                        const float* __restrict__ v, XT* __restrict__ Xhat, int64_t ldx)
{
    const int64_t total = N * D;
    const int64_t stride = static_cast<int64_t>(gridDim.x) * kStreamThreads;
    for (int64_t idx = static_cast<int64_t>(blockIdx.x) * kStreamThreads + threadIdx.x; idx < total; idx += stride) {
        const int64_t row = idx / D;
        const int d = static_cast<int>(idx - row * D);
        const int m = d / Dsub;
        const int j = d - m * Dsub;
        Elem<XT>::store(Xhat + row * ldx + d, load_z<ZT>(Z + row * ldz + m) * __ldg(v + j));
    }
}

// ------------------------------------------------------------------ expansion of the factored weight gradient
// (Section 3.2's rank-1 form, per sub-token):
//   dW[o, m*Dsub + j] = beta*dW[o, m*Dsub + j] + (sum_s P[s][o][m]) * v[j]
// P holds `splits` partial products dY^T Z over disjoint token ranges, summed here in a fixed order.
template <typename WT>
__global__ void __launch_bounds__(kStreamThreads)
expand_p_elem_kernel(const float* __restrict__ P, int splits, int64_t split_stride, int64_t ldp,
                     const float* __restrict__ v, int64_t O, int D, int Dsub,
                     WT* __restrict__ dW, int64_t lddw, int beta)
{
    const int64_t total = O * D;
    const int64_t stride = static_cast<int64_t>(gridDim.x) * kStreamThreads;
    for (int64_t idx = static_cast<int64_t>(blockIdx.x) * kStreamThreads + threadIdx.x; idx < total; idx += stride) {
        const int64_t o = idx / D;
        const int d = static_cast<int>(idx - o * D);
        const int m = d / Dsub;
        const int j = d - m * Dsub;
        float p = 0.f;
        for (int s = 0; s < splits; ++s) p += __ldg(P + s * split_stride + o * ldp + m);
        float r = p * __ldg(v + j);
        if (beta) r += Elem<WT>::load(dW + o * lddw + d);
        Elem<WT>::store(dW + o * lddw + d, r);
    }
}

// ------------------------------------------------------------------ sub-tokens shorter than a 16-byte chunk
// Dsub in {1, 2, 4} (the paper's smallest setting, sub-token length 4 with rank-4 adapters): a 16-byte chunk of
// a row holds 8 / Dsub whole sub-tokens, so a thread needs no partner: one 128-bit load, 8 / Dsub dot
// products (compress) or 8 / Dsub scalars times v (reconstruct), coalesced stores.  Four chunks per thread are
// in flight.  Columns beyond D inside the last chunk of a row (row pitch padded to 8) are treated as zeros.
template <int DS, typename ZT>
__global__ void __launch_bounds__(kStreamThreads)
compress_small_kernel(const uint4* __restrict__ X, int64_t N, int D, int64_t ldc, int M,
                      const float* __restrict__ v, ZT* __restrict__ Z, int64_t ldz)
{
    constexpr int PER = 8 / DS;
    float vr[DS];
#pragma unroll
    for (int j = 0; j < DS; ++j) vr[j] = __ldg(v + j);
    const int chunks = (D + 7) / 8;
    const int64_t total = N * chunks;
    const int64_t stride = static_cast<int64_t>(gridDim.x) * kStreamThreads;
    for (int64_t base = static_cast<int64_t>(blockIdx.x) * kStreamThreads + threadIdx.x; base < total; base += 4 * stride) {
        uint4 d[4];
        int64_t row[4];
        int c[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int64_t idx = base + u * stride;
            row[u] = idx / chunks;
            c[u] = static_cast<int>(idx - row[u] * chunks);
            d[u] = idx < total ? __ldg(X + row[u] * ldc + c[u]) : make_uint4(0u, 0u, 0u, 0u);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            if (base + u * stride >= total) break;
            float x[8];
            x[0] = bf16_lo(d[u].x); x[1] = bf16_hi(d[u].x);
            x[2] = bf16_lo(d[u].y); x[3] = bf16_hi(d[u].y);
            x[4] = bf16_lo(d[u].z); x[5] = bf16_hi(d[u].z);
            x[6] = bf16_lo(d[u].w); x[7] = bf16_hi(d[u].w);
#pragma unroll
            for (int e = 0; e < 8; ++e)
                if (8 * c[u] + e >= D) x[e] = 0.f;
#pragma unroll
            for (int k = 0; k < PER; ++k) {
                float z = 0.f;
#pragma unroll
                for (int j = 0; j < DS; ++j) z = fmaf(x[k * DS + j], vr[j], z);
                const int m = c[u] * PER + k;
                if (m < M) Elem<ZT>::store(Z + row[u] * ldz + m, z);
            }
        }
    }
}

template <int DS, typename ZT>
__global__ void __launch_bounds__(kStreamThreads)
reconstruct_small_kernel(const ZT* __restrict__ Z, int64_t ldz, int64_t N, int D, int M,
                         const float* __restrict__ v, uint4* __restrict__ Xhat, int64_t ldc)
{
    constexpr int PER = 8 / DS;
    float vr[DS];
#pragma unroll
    for (int j = 0; j < DS; ++j) vr[j] = __ldg(v + j);
    const int chunks = (D + 7) / 8;                       // D is a multiple of 8 here (whole 16-byte stores)
    const int64_t total = N * chunks;
    const int64_t stride = static_cast<int64_t>(gridDim.x) * kStreamThreads;
    for (int64_t idx = static_cast<int64_t>(blockIdx.x) * kStreamThreads + threadIdx.x; idx < total; idx += stride) {
        const int64_t row = idx / chunks;
        const int c = static_cast<int>(idx - row * chunks);
        float y[8];
#pragma unroll
        for (int k = 0; k < PER; ++k) {
            const int m = c * PER + k;
            const float z = m < M ? Elem<ZT>::load(Z + row * ldz + m) : 0.f;
#pragma unroll
            for (int j = 0; j < DS; ++j) y[k * DS + j] = z * vr[j];
        }
        uint4 o;
        o.x = pack_bf16x2(y[0], y[1]);
        o.y = pack_bf16x2(y[2], y[3]);
        o.z = pack_bf16x2(y[4], y[5]);
        o.w = pack_bf16x2(y[6], y[7]);
        __stcs(Xhat + row * ldc + c, o);
    }
}

// ------------------------------------------------------------------ any sub-token length that is a multiple of 8
// The paper's sub-token size ablation uses D/8 .. D/64 of a 768-wide layer: 96, 48, 24 (Section 5), none a
// power of two.  compress: a warp walks a row in windows of 32 chunks (512 contiguous bytes per load
// instruction); a lane multiplies its chunk with its slice of v, then the lanes of a sub-token are added up
// by a segmented shuffle reduction (the key is the sub-token index), and what a sub-token has collected when
// the window ends is carried into the next window by the same warp.  Sums run in a fixed order.
template <typename ZT>
__global__ void __launch_bounds__(kStreamThreads)
compress_seg_kernel(const uint4* __restrict__ X, int N, int D, int64_t ldc, int Dsub, int M,
                    const float* __restrict__ v, ZT* __restrict__ Z, int64_t ldz)
{
    extern __shared__ float sv_seg[];
    for (int j = threadIdx.x; j < Dsub; j += kStreamThreads) sv_seg[j] = __ldg(v + j);
    __syncthreads();
    const int lane = threadIdx.x & 31;
    const int chunks = (D + 7) / 8;
    const int warps = gridDim.x * (kStreamThreads / 32);
    for (int row = blockIdx.x * (kStreamThreads / 32) + (threadIdx.x >> 5); row < N; row += warps) {
        const uint4* xr = X + static_cast<int64_t>(row) * ldc;
        float carry = 0.f;
        int carry_m = -1;
        for (int w0 = 0; w0 < chunks; w0 += 128) {          // four windows (2 KB of the row) in flight
            uint4 d[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int c = w0 + 32 * u + lane;
                d[u] = c < chunks ? __ldg(xr + c) : make_uint4(0u, 0u, 0u, 0u);
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int wbase = w0 + 32 * u;
                if (wbase >= chunks) break;
                const int c = wbase + lane;
                const bool valid = c < chunks;
                const int m = valid ? (8 * c) / Dsub : -2 - lane;
                float p = 0.f;
                if (valid) {
                    const int j0 = 8 * c - m * Dsub;
                    const float4 va = *reinterpret_cast<const float4*>(sv_seg + j0);
                    const float4 vb = *reinterpret_cast<const float4*>(sv_seg + j0 + 4);
                    float x[8];
                    x[0] = bf16_lo(d[u].x); x[1] = bf16_hi(d[u].x);
                    x[2] = bf16_lo(d[u].y); x[3] = bf16_hi(d[u].y);
                    x[4] = bf16_lo(d[u].z); x[5] = bf16_hi(d[u].z);
                    x[6] = bf16_lo(d[u].w); x[7] = bf16_hi(d[u].w);
#pragma unroll
                    for (int e = 0; e < 8; ++e)
                        if (8 * c + e >= D) x[e] = 0.f;              // padding of the row pitch is not data
                    p = x[0] * va.x;
                    p = fmaf(x[1], va.y, p); p = fmaf(x[2], va.z, p); p = fmaf(x[3], va.w, p);
                    p = fmaf(x[4], vb.x, p); p = fmaf(x[5], vb.y, p); p = fmaf(x[6], vb.z, p); p = fmaf(x[7], vb.w, p);
                }
                // After the five steps the first lane of every run of equal keys holds the run's sum.
#pragma unroll
                for (int off = 1; off < 32; off <<= 1) {
                    const float p2 = __shfl_down_sync(0xffffffffu, p, off);
                    const int m2 = __shfl_down_sync(0xffffffffu, m, off);
                    if (lane + off < 32 && m2 == m) p += p2;
                }
                const int m_left = __shfl_up_sync(0xffffffffu, m, 1);
                const bool head = valid && (lane == 0 || m_left != m);
                if (lane == 0 && m == carry_m) p += carry;           // the sub-token began in an earlier window
                // Last chunk of sub-token m: the one before the next sub-token starts, or the row's last chunk.
                int end_chunk = ((m + 1) * Dsub) / 8 - 1;
                if (end_chunk > chunks - 1) end_chunk = chunks - 1;
                const bool ends_here = end_chunk <= wbase + 31;
                if (head && ends_here && m < M) Elem<ZT>::store(Z + static_cast<int64_t>(row) * ldz + m, p);
                const unsigned heads = __ballot_sync(0xffffffffu, head);
                const int last_head = 31 - __clz(heads);             // heads != 0: lane 0 of a live window is valid
                const float p_last = __shfl_sync(0xffffffffu, p, last_head);
                const int m_last = __shfl_sync(0xffffffffu, m, last_head);
                const int open = __shfl_sync(0xffffffffu, ends_here ? 0 : 1, last_head);
                carry = p_last;
                carry_m = open ? m_last : -1;
            }
        }
    }
}

__device__ __forceinline__ void store8(__nv_bfloat16* p, float (&y)[8], int beta)
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
__device__ __forceinline__ void store8(float* p, float (&y)[8], int beta)
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

// out[r, 8c .. 8c+7] = beta * out + (sum_s S[s][r][m(c)]) * v[...]: one thread per 16-byte-aligned group of eight
// outputs, for any Dsub that is a multiple of 8 (a group then lies inside one sub-token).  Serves reconstruct
// (one split, beta = 0) and the expansion of the factor P where the power-of-two kernel does not apply.
template <typename ST, typename WT>
__global__ void __launch_bounds__(kStreamThreads)
expand_any_kernel(const ST* __restrict__ S, int splits, int64_t split_stride, int64_t lds, const float* __restrict__ v,
                  int64_t R, int D, int Dsub, WT* __restrict__ out, int64_t ldo, int beta)
{
    extern __shared__ float sv_any[];
    for (int j = threadIdx.x; j < Dsub; j += kStreamThreads) sv_any[j] = __ldg(v + j);
    __syncthreads();
    const int chunks = D / 8;                                 // D is a multiple of 8 here
    const int64_t total = R * chunks;
    const int64_t stride = static_cast<int64_t>(gridDim.x) * kStreamThreads;
    for (int64_t idx = static_cast<int64_t>(blockIdx.x) * kStreamThreads + threadIdx.x; idx < total; idx += stride) {
        const int64_t r = idx / chunks;
        const int c = static_cast<int>(idx - r * chunks);
        const int m = (8 * c) / Dsub;
        const int j0 = 8 * c - m * Dsub;
        float z = 0.f;
        for (int sp = 0; sp < splits; ++sp) z += Elem<ST>::load(S + sp * split_stride + r * lds + m);   // fixed order
        const float4 va = *reinterpret_cast<const float4*>(sv_any + j0);
        const float4 vb = *reinterpret_cast<const float4*>(sv_any + j0 + 4);
        float y[8] = {z * va.x, z * va.y, z * va.z, z * va.w, z * vb.x, z * vb.y, z * vb.z, z * vb.w};
        store8(out + r * ldo + 8 * c, y, beta);                // 16-byte aligned: checked on the host
    }
}

// ------------------------------------------------------------------ host side
bool rows_vectorisable(const void* p, int64_t ld_elems)
{
    return aligned16(p) && (ld_elems % 8 == 0);
}

int stream_grid(int64_t items, int per_thread, int* grid)
{
    DeviceInfo di;
    const int rc = device_info(&di);
    if (rc != VELORA_OK) return rc;
    int64_t ctas = ceil_div64(items, static_cast<int64_t>(kStreamThreads) * per_thread);
    const int64_t cap = static_cast<int64_t>(di.sm_count) * kStreamCtasPerSm;
    if (ctas > cap) ctas = cap;
    if (ctas < 1) ctas = 1;
    *grid = static_cast<int>(ctas);
    return VELORA_OK;
}

int check_launch()
{
    return after_launch();
}

}  // namespace

size_t init_v_workspace_bytes(int Dsub)
{
    return kStatusBytes + static_cast<size_t>(kInitVMaxCtas) * static_cast<size_t>(Dsub) * sizeof(float);
}

namespace {
int read_degenerate_flag(const int* status, cudaStream_t stream)
{
    int host_status = -1;
    if (cudaMemcpyAsync(&host_status, status, sizeof(int), cudaMemcpyDeviceToHost, stream) != cudaSuccess)
        return VELORA_ERR_CUDA;
    if (cudaStreamSynchronize(stream) != cudaSuccess) return VELORA_ERR_CUDA;
    if (host_status == 0) return VELORA_OK;
    return host_status == 1 ? VELORA_ERR_DEGENERATE_V : VELORA_ERR_CUDA;
}
}  // namespace

int launch_normalize_v(const float* s, int Dsub, float* v, void* ws, size_t ws_bytes, cudaStream_t stream)
{
    if (ws_bytes < kStatusBytes) return VELORA_ERR_WORKSPACE;
    int* status = static_cast<int*>(ws) + 1;
    launch_init_v_finalize(s, 1, Dsub, v, status, 1, stream);
    if (check_launch() != VELORA_OK) return VELORA_ERR_CUDA;
    return read_degenerate_flag(status, stream);
}

size_t update_v_workspace_bytes(int Dsub)
{
    return init_v_workspace_bytes(Dsub) + ((static_cast<size_t>(Dsub) * sizeof(float) + 255) / 256) * 256;
}

int launch_update_v(const void* X, int x_dtype, int64_t N, int64_t D, int64_t ldx, int Dsub, float rho,
                    float* a, float* v, void* ws, size_t ws_bytes, cudaStream_t stream)
{
    if (ws_bytes < update_v_workspace_bytes(Dsub)) return VELORA_ERR_WORKSPACE;
    float* s = reinterpret_cast<float*>(static_cast<char*>(ws) + init_v_workspace_bytes(Dsub));
    const int rc = launch_init_v(X, x_dtype, N, D, ldx, Dsub, s, ws, init_v_workspace_bytes(Dsub), stream, 1);
    if (rc != VELORA_OK) return rc;
    const double count = static_cast<double>(N) * static_cast<double>(ceil_div64(D, Dsub));
    update_v_kernel<<<1, kStreamThreads, 0, stream>>>(s, 1.0 / count, rho, Dsub, a, v, static_cast<int*>(ws));
    return check_launch();
}

int launch_init_v(const void* X, int x_dtype, int64_t N, int64_t D, int64_t ldx, int Dsub,
                  float* v, void* ws, size_t ws_bytes, cudaStream_t stream, int sum_only)
{
    if (ws_bytes < init_v_workspace_bytes(Dsub)) return VELORA_ERR_WORKSPACE;
    int* status = static_cast<int*>(ws) + 1;             // word 1: degenerate-sum flag of this call
    float* partials = reinterpret_cast<float*>(static_cast<char*>(ws) + kStatusBytes);
    const int M = static_cast<int>(ceil_div64(D, Dsub));
    int num_partials = 0;

    int rows_rc = VELORA_ERR_UNSUPPORTED;
    if (x_dtype == VELORA_BF16)
        rows_rc = launch_init_v_partials_rows(X, N, D, ldx, Dsub, partials, kInitVMaxCtas, &num_partials, stream);
    if (rows_rc != VELORA_ERR_UNSUPPORTED) {
        if (rows_rc != VELORA_OK) return rows_rc;
    } else {
        DeviceInfo di;
        int rc = device_info(&di);
        if (rc != VELORA_OK) return rc;
        int64_t grid = static_cast<int64_t>(di.sm_count) * 4;
        if (grid > kInitVMaxCtas) grid = kInitVMaxCtas;
        if (grid > N) grid = N;
        const int64_t rows_per_cta = ceil_div64(N, grid);
        grid = ceil_div64(N, rows_per_cta);
        num_partials = static_cast<int>(grid);
        if (x_dtype == VELORA_BF16)
            init_v_partial_elem_kernel<__nv_bfloat16><<<static_cast<int>(grid), kStreamThreads, 0, stream>>>(
                static_cast<const __nv_bfloat16*>(X), N, static_cast<int>(D), ldx, Dsub, M, rows_per_cta, partials);
        else
            init_v_partial_elem_kernel<float><<<static_cast<int>(grid), kStreamThreads, 0, stream>>>(
                static_cast<const float*>(X), N, static_cast<int>(D), ldx, Dsub, M, rows_per_cta, partials);
    }
    if (check_launch() != VELORA_OK) return VELORA_ERR_CUDA;
    launch_init_v_finalize(partials, num_partials, Dsub, v, status, sum_only ? 0 : 1, stream);
    if (check_launch() != VELORA_OK) return VELORA_ERR_CUDA;
    if (sum_only) return VELORA_OK;                            // v holds s; nothing to report, no synchronisation
    return read_degenerate_flag(status, stream);
}

int launch_compress(const void* X, int x_dtype, int64_t N, int64_t D, int64_t ldx, int Dsub,
                    const float* v, void* Z, int z_dtype, int64_t ldz, cudaStream_t stream)
{
    const int M = static_cast<int>(ceil_div64(D, Dsub));
    if (x_dtype == VELORA_BF16) {                        // aligned rows, Dsub = 8 * 2^k: the row-streaming kernel
        const int rc = launch_compress_rows(X, N, D, ldx, Dsub, v, Z, z_dtype, ldz, stream);
        if (rc != VELORA_ERR_UNSUPPORTED) return rc;
    }
    const bool z8 = z_dtype == VELORA_FP8_E4M3;          // 8-bit Z: the TMA kernel above or the element kernel below
    if (!z8 && x_dtype == VELORA_BF16 && (Dsub == 1 || Dsub == 2 || Dsub == 4) && rows_vectorisable(X, ldx) && D < (1 << 30)) {
        int grid = 0;
        const int rc = stream_grid(N * ceil_div64(D, 8), 4, &grid);
        if (rc != VELORA_OK) return rc;
#define CALL_SMALL(DSV)                                                                                     \
        if (z_dtype == VELORA_F32)                                                                          \
            compress_small_kernel<DSV, float><<<grid, kStreamThreads, 0, stream>>>(                         \
                static_cast<const uint4*>(X), N, static_cast<int>(D), ldx / 8, M, v, static_cast<float*>(Z), ldz); \
        else                                                                                                \
            compress_small_kernel<DSV, __nv_bfloat16><<<grid, kStreamThreads, 0, stream>>>(                 \
                static_cast<const uint4*>(X), N, static_cast<int>(D), ldx / 8, M, v, static_cast<__nv_bfloat16*>(Z), ldz)
        if (Dsub == 1) { CALL_SMALL(1); } else if (Dsub == 2) { CALL_SMALL(2); } else { CALL_SMALL(4); }
#undef CALL_SMALL
        return check_launch();
    }
    if (!z8 && x_dtype == VELORA_BF16 && Dsub % 8 == 0 && rows_vectorisable(X, ldx) && N < (1 << 30) && D < (1 << 28)) {
        // any other multiple of 8 (96, 48, 24 ...): segmented reduction over the lanes of a sub-token
        int sgrid = 0;
        const int src = stream_grid(N * 32, 1, &sgrid);
        if (src != VELORA_OK) return src;
        const size_t smem = static_cast<size_t>(Dsub) * sizeof(float);
        if (z_dtype == VELORA_F32)
            compress_seg_kernel<float><<<sgrid, kStreamThreads, smem, stream>>>(
                static_cast<const uint4*>(X), static_cast<int>(N), static_cast<int>(D), ldx / 8, Dsub, M, v, static_cast<float*>(Z), ldz);
        else
            compress_seg_kernel<__nv_bfloat16><<<sgrid, kStreamThreads, smem, stream>>>(
                static_cast<const uint4*>(X), static_cast<int>(N), static_cast<int>(D), ldx / 8, Dsub, M, v,
                static_cast<__nv_bfloat16*>(Z), ldz);
        return check_launch();
    }
    int grid = 0;
    int rc = stream_grid(N * M * 32, 1, &grid);
    if (rc != VELORA_OK) return rc;
#define CALL_ELEM(XT, ZT)                                                                                 \
    compress_elem_kernel<XT, ZT><<<grid, kStreamThreads, 0, stream>>>(                                    \
        static_cast<const XT*>(X), N, static_cast<int>(D), ldx, Dsub, M, v, static_cast<ZT*>(Z), ldz)
    if (x_dtype == VELORA_BF16 && z_dtype == VELORA_F32) CALL_ELEM(__nv_bfloat16, float);
    else if (x_dtype == VELORA_BF16 && z8) CALL_ELEM(__nv_bfloat16, e4m3_t);
    else if (x_dtype == VELORA_BF16) CALL_ELEM(__nv_bfloat16, __nv_bfloat16);
    else if (z_dtype == VELORA_F32) CALL_ELEM(float, float);
    else if (z8) CALL_ELEM(float, e4m3_t);
    else CALL_ELEM(float, __nv_bfloat16);
#undef CALL_ELEM
    return check_launch();
}

// Per-chunk expansion for any Dsub that is a multiple of 8; VELORA_ERR_UNSUPPORTED (nothing launched) otherwise.
static int launch_expand_any(const void* S, int s_dtype, int splits, int64_t split_stride, int64_t lds, const float* v,
                             int64_t R, int64_t D, int Dsub, void* out, int out_dtype, int64_t ldo, int beta,
                             cudaStream_t stream)
{
    if (Dsub % 8 || D % 8 || D >= (1 << 28) || R < 1) return VELORA_ERR_UNSUPPORTED;
    if (!aligned16(out) || (ldo * static_cast<int64_t>(dtype_size(out_dtype))) % 16) return VELORA_ERR_UNSUPPORTED;
    if (s_dtype == VELORA_BF16 && out_dtype != VELORA_BF16) return VELORA_ERR_UNSUPPORTED;
    int grid = 0;
    const int rc = stream_grid(R * (D / 8), 2, &grid);
    if (rc != VELORA_OK) return rc;
    const size_t smem = static_cast<size_t>(Dsub) * sizeof(float);
    const int d = static_cast<int>(D);
    if (s_dtype == VELORA_BF16)
        expand_any_kernel<__nv_bfloat16, __nv_bfloat16><<<grid, kStreamThreads, smem, stream>>>(
            static_cast<const __nv_bfloat16*>(S), splits, split_stride, lds, v, R, d, Dsub, static_cast<__nv_bfloat16*>(out), ldo, beta);
    else if (out_dtype == VELORA_BF16)
        expand_any_kernel<float, __nv_bfloat16><<<grid, kStreamThreads, smem, stream>>>(
            static_cast<const float*>(S), splits, split_stride, lds, v, R, d, Dsub, static_cast<__nv_bfloat16*>(out), ldo, beta);
    else
        expand_any_kernel<float, float><<<grid, kStreamThreads, smem, stream>>>(
            static_cast<const float*>(S), splits, split_stride, lds, v, R, d, Dsub, static_cast<float*>(out), ldo, beta);
    return check_launch();
}

int launch_reconstruct(const void* Z, int z_dtype, int64_t ldz, int64_t N, int64_t D, int Dsub,
                       const float* v, void* Xhat, int x_dtype, int64_t ldxhat, cudaStream_t stream)
{
    if (x_dtype == VELORA_BF16) {                        // Xhat = Z (x) v is the one-split, beta = 0 expansion
        const int rc = launch_expand_rows_vec(Z, z_dtype, 1, 0, ldz, v, N, D, Dsub, Xhat, x_dtype, ldxhat, 0, stream);
        if (rc != VELORA_ERR_UNSUPPORTED) return rc;
    }
    const bool z8 = z_dtype == VELORA_FP8_E4M3;          // 8-bit Z: the vector expansion above or the element kernel below
    if (!z8 && x_dtype == VELORA_BF16 && (Dsub == 1 || Dsub == 2 || Dsub == 4) && D % 8 == 0 && rows_vectorisable(Xhat, ldxhat) &&
        D < (1 << 30)) {
        const int M = static_cast<int>(ceil_div64(D, Dsub));
        int grid = 0;
        const int rc = stream_grid(N * (D / 8), 1, &grid);
        if (rc != VELORA_OK) return rc;
#define CALL_SMALL(DSV)                                                                                     \
        if (z_dtype == VELORA_F32)                                                                          \
            reconstruct_small_kernel<DSV, float><<<grid, kStreamThreads, 0, stream>>>(                      \
                static_cast<const float*>(Z), ldz, N, static_cast<int>(D), M, v, static_cast<uint4*>(Xhat), ldxhat / 8); \
        else                                                                                                \
            reconstruct_small_kernel<DSV, __nv_bfloat16><<<grid, kStreamThreads, 0, stream>>>(              \
                static_cast<const __nv_bfloat16*>(Z), ldz, N, static_cast<int>(D), M, v, static_cast<uint4*>(Xhat), ldxhat / 8)
        if (Dsub == 1) { CALL_SMALL(1); } else if (Dsub == 2) { CALL_SMALL(2); } else { CALL_SMALL(4); }
#undef CALL_SMALL
        return check_launch();
    }
    if (!z8) {
        const int arc = launch_expand_any(Z, z_dtype, 1, 0, ldz, v, N, D, Dsub, Xhat, x_dtype, ldxhat, 0, stream);
        if (arc != VELORA_ERR_UNSUPPORTED) return arc;
    }
    int grid = 0;
    int rc = stream_grid(N * D, 4, &grid);
    if (rc != VELORA_OK) return rc;
#define CALL_ELEM(ZT, XT)                                                                                 \
    reconstruct_elem_kernel<ZT, XT><<<grid, kStreamThreads, 0, stream>>>(                                 \
        static_cast<const ZT*>(Z), ldz, N, static_cast<int>(D), Dsub, v, static_cast<XT*>(Xhat), ldxhat)
    if (z_dtype == VELORA_F32 && x_dtype == VELORA_BF16) CALL_ELEM(float, __nv_bfloat16);
    else if (z_dtype == VELORA_F32) CALL_ELEM(float, float);
    else if (z8 && x_dtype == VELORA_BF16) CALL_ELEM(e4m3_t, __nv_bfloat16);
    else if (z8) CALL_ELEM(e4m3_t, float);
    else if (x_dtype == VELORA_BF16) CALL_ELEM(__nv_bfloat16, __nv_bfloat16);
    else CALL_ELEM(__nv_bfloat16, float);
#undef CALL_ELEM
    return check_launch();
}

int launch_expand_p(const float* P, int splits, int64_t split_stride, int64_t ldp, const float* v,
                    int64_t O, int64_t D, int Dsub, void* dW, int dw_dtype, int64_t lddw, int beta,
                    cudaStream_t stream)
{
    int rc = launch_expand_rows_vec(P, VELORA_F32, splits, split_stride, ldp, v, O, D, Dsub, dW, dw_dtype, lddw, beta, stream);
    if (rc != VELORA_ERR_UNSUPPORTED) return rc;
    rc = launch_expand_any(P, VELORA_F32, splits, split_stride, ldp, v, O, D, Dsub, dW, dw_dtype, lddw, beta, stream);
    if (rc != VELORA_ERR_UNSUPPORTED) return rc;
    int grid = 0;
    rc = stream_grid(O * D, 4, &grid);
    if (rc != VELORA_OK) return rc;
    if (dw_dtype == VELORA_BF16)
        expand_p_elem_kernel<__nv_bfloat16><<<grid, kStreamThreads, 0, stream>>>(
            P, splits, split_stride, ldp, v, O, static_cast<int>(D), Dsub, static_cast<__nv_bfloat16*>(dW), lddw, beta);
    else
        expand_p_elem_kernel<float><<<grid, kStreamThreads, 0, stream>>>(
            P, splits, split_stride, ldp, v, O, static_cast<int>(D), Dsub, static_cast<float*>(dW), lddw, beta);
    return check_launch();
}

}  // namespace velora
// ------------------------------------------------------------------ scale of the 8-bit Z store
namespace velora {
namespace {

// Largest |z| of a contiguous fp32 array, as the bit pattern of a non-negative float (those order like
// unsigned integers; a NaN's pattern is above every finite one, so it surfaces as "not finite").
__global__ void __launch_bounds__(kStreamThreads) z_amax_kernel(const float* __restrict__ Z, int64_t count, unsigned int* amax_bits)
{
    unsigned int best = 0u;
    const int64_t stride = static_cast<int64_t>(gridDim.x) * kStreamThreads;
    for (int64_t i = static_cast<int64_t>(blockIdx.x) * kStreamThreads + threadIdx.x; i < count; i += stride) {
        const unsigned int b = __float_as_uint(__ldg(Z + i)) & 0x7fffffffu;
        best = b > best ? b : best;
    }
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) {
        const unsigned int o = __shfl_xor_sync(kFull, best, off);
        best = o > best ? o : best;
    }
    if ((threadIdx.x & 31) == 0 && best) atomicMax(amax_bits, best);     // a maximum: the order of arrival does not matter
}

__global__ void __launch_bounds__(kStreamThreads) z8_scale_kernel(const unsigned int* amax_bits, float headroom, const float* __restrict__ v,
                                                                   int Dsub, float* zscale, float* v_store, float* v_load)
{
    const float amax = __uint_as_float(*amax_bits);
    float scale = 1.f;
    if (amax > 0.f && amax <= 3.0e38f) scale = headroom * amax / 448.f;
    if (!(scale > 0.f) || !(scale <= 3.0e38f)) scale = 1.f;
    if (threadIdx.x == 0) *zscale = scale;
    for (int j = threadIdx.x; j < Dsub; j += kStreamThreads) {
        const float x = __ldg(v + j);
        v_store[j] = x / scale;
        v_load[j] = x * scale;
    }
}

}  // namespace

size_t z8_calibrate_workspace_bytes(int64_t N, int64_t D, int Dsub)
{
    const size_t zbytes = static_cast<size_t>(N) * static_cast<size_t>(ceil_div64(D, Dsub)) * sizeof(float);
    return kStatusBytes + 256 + (zbytes + 255) / 256 * 256;
}

int launch_z8_calibrate(const void* X, int x_dtype, int64_t N, int64_t D, int64_t ldx, int Dsub, const float* v,
                        float headroom, float* zscale, float* v_store, float* v_load,
                        void* ws, size_t ws_bytes, cudaStream_t stream)
{
    if (ws_bytes < z8_calibrate_workspace_bytes(N, D, Dsub)) return VELORA_ERR_WORKSPACE;
    unsigned int* amax_bits = reinterpret_cast<unsigned int*>(static_cast<char*>(ws) + kStatusBytes);
    float* Z = reinterpret_cast<float*>(static_cast<char*>(ws) + kStatusBytes + 256);
    const int64_t M = ceil_div64(D, Dsub);
    if (cudaMemsetAsync(amax_bits, 0, sizeof(unsigned int), stream) != cudaSuccess) return VELORA_ERR_CUDA;
    if (N > 0) {
        int rc = launch_compress(X, x_dtype, N, D, ldx, Dsub, v, Z, VELORA_F32, M, stream);
        if (rc != VELORA_OK) return rc;
        int grid = 0;
        rc = stream_grid(N * M, 4, &grid);
        if (rc != VELORA_OK) return rc;
        z_amax_kernel<<<grid, kStreamThreads, 0, stream>>>(Z, N * M, amax_bits);
        if (check_launch() != VELORA_OK) return VELORA_ERR_CUDA;
    }
    z8_scale_kernel<<<1, kStreamThreads, 0, stream>>>(amax_bits, headroom, v, Dsub, zscale, v_store, v_load);
    return check_launch();
}

}  // namespace velora
// ------------------------------------------------------------------ velora_init_v without a workspace
// Scratch for velora_init_v_static: the status header plus one row of partial sums per CTA, for
// sub-tokens of up to VELORA_INIT_V_STATIC_MAX_DSUB elements.  It is part of the loaded module, so
// every GPU that loads the library carries these ~1.2 MB until the process exits.
namespace velora {
namespace {
constexpr size_t kStaticScratchBytes =
    kStatusBytes + static_cast<size_t>(kInitVMaxCtas) * VELORA_INIT_V_STATIC_MAX_DSUB * sizeof(float);
static __device__ __align__(256) unsigned char g_init_v_scratch[kStaticScratchBytes];

// Device address of g_init_v_scratch on the current device.  In host code the array's name is only a
// handle for the runtime, never a pointer a kernel may use; the real address is asked for once per
// device, with that device current, and remembered.
int static_scratch_address(void** out)
{
    static std::atomic<void*> cached[64];          // two threads' first calls both store the same address
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return VELORA_ERR_CUDA;
    if (dev < 0 || dev >= 64) return VELORA_ERR_UNSUPPORTED;
    void* p = cached[dev].load(std::memory_order_relaxed);
    if (!p) {
        if (cudaGetSymbolAddress(&p, g_init_v_scratch) != cudaSuccess || !p) return VELORA_ERR_CUDA;
        cached[dev].store(p, std::memory_order_relaxed);
    }
    *out = p;
    return VELORA_OK;
}
}  // namespace
}  // namespace velora

extern "C" int velora_init_v_static(const void* X, int x_dtype, int64_t N, int64_t D, int64_t ldx, int Dsub,
                                    float* v, void* stream)
{
    using namespace velora;
    if (N < 0 || D < 1 || Dsub < 1 || Dsub > D) return VELORA_ERR_INVALID_ARG;
    if (Dsub > VELORA_INIT_V_STATIC_MAX_DSUB) return VELORA_ERR_UNSUPPORTED;   // beyond the built-in scratch
    if (D > (1 << 30) || N > (static_cast<int64_t>(1) << 40)) return VELORA_ERR_UNSUPPORTED;
    if (!valid_dtype(x_dtype)) return VELORA_ERR_UNSUPPORTED;
    if (N == 0) return VELORA_ERR_DEGENERATE_V;
    if (!X || !v) return VELORA_ERR_INVALID_ARG;
    if (ldx < D) return VELORA_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(X) % dtype_size(x_dtype) || reinterpret_cast<uintptr_t>(v) % sizeof(float))
        return VELORA_ERR_ALIGNMENT;
    void* scratch = nullptr;
    const int rc = static_scratch_address(&scratch);
    if (rc != VELORA_OK) return rc;
    // Every partial-sum row that is read was written by this call, and the result word is rewritten
    // by every call, so nothing in the shared scratch has to be cleared first.
    return launch_init_v(X, x_dtype, N, D, ldx, Dsub, v, scratch, kStaticScratchBytes,
                         static_cast<cudaStream_t>(stream));
}
