// Factored weight gradient on the sm_100a tensor cores (arxiv 2405.17991, Algorithm 1 backward with
// the rank-1 identity of Section 3.2 applied per sub-token):
//     P[o, m] = sum_n dY[n, o] * Z[n, m],      dW[o, m*Dsub + j] = beta*dW + P[o, m] * v[j].
// The reconstructed input is never formed.  The work is bound by HBM traffic (read dY once, write dW
// once); the contraction over tokens is small next to it and runs on tcgen05 so that it hides under
// the dY stream.
//
//   z_to_bf16_kernel   Z (fp32 or bf16, any pitch) -> Zb[N, pitch] bf16, pitch = round_up(M, 64), zero
//                      padded, so that TMA can fetch 64-wide MN-major slabs.
//   wg_kernel          grid (O/128, S): CTA (t, s) multiplies dY[:, 128t : 128t+128]^T with Zb over its
//                      share of the tokens.  Both operands are MN-major (tokens are the K dimension and
//                      rows of dY / Zb are tokens): 64 x 64 TMA boxes, MN-major matrix descriptors, no
//                      transpose; fp32 accumulator in TMEM.  Splitting the token range keeps every SM
//                      pulling on dY.
//     CLUSTER = true   the S CTAs of an output tile form a thread-block cluster.  Each parks its partial
//                      product in its own shared memory; after a cluster barrier CTA s adds the S
//                      partials of its share of the 128 rows through distributed shared memory, in a
//                      fixed order, and streams dW = P (x) v for those rows.  One launch, no partials in
//                      global memory, every SM takes part in the write.
//                      Two launch shapes: two CTAs of six warps per SM (ring of 2..4 stages), or, where the
//                      partial products are large and the row blocks few, one CTA of twelve warps per SM with
//                      half as many splits (half the reduction traffic, four stages, as many warps writing).
//     CLUSTER = false  the partials go to the workspace and launch_expand_p sums and expands them
//                      (shapes the cluster form does not take: Dsub not 8 * 2^k, unaligned dW rows).
// Summing the partials in a fixed order keeps the result run-to-run identical.
#include <cooperative_groups.h>

#include "gemm_tc.cuh"
#include "tc_common.cuh"

namespace velora {

using namespace tc;

namespace {

constexpr int WG_BM = 128, WG_BK = 64, WG_STAGES = 4;   // WG_STAGES: most ring stages (2..4 are used)
constexpr int WG_A_BYTES = WG_BM * WG_BK * 2;         // 16 KB: two 64-wide slabs of dY^T
constexpr int WG_SLAB = 64 * WG_BK * 2;               // 8 KB
constexpr int WG_THREADS = 192;
constexpr int WG_MAX_SPLITS = 8;                      // also the portable cluster size limit
constexpr int WG_MAX_M = 256;

inline int64_t round_up(int64_t x, int64_t m) { return (x + m - 1) / m * m; }

template <typename ZT>
__global__ void __launch_bounds__(256)
z_to_bf16_kernel(const ZT* __restrict__ Z, int64_t ldz, int64_t N, int M, int pitch, uint4* __restrict__ Zb)
{
    // The kernel that consumes Zb may be launched now: it waits (griddepcontrol.wait) before its first
    // read of Zb, and meanwhile sets up and starts pulling dY.  Z itself may come from the kernel before.
    pdl_trigger();
    pdl_wait();
    const int chunks = pitch / 8;
    const int64_t total = N * chunks;
    const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
    for (int64_t idx = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; idx < total; idx += stride) {
        const int64_t n = idx / chunks;
        const int c0 = static_cast<int>(idx - n * chunks) * 8;
        float f[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) f[e] = (c0 + e < M) ? Elem<ZT>::load(Z + n * ldz + c0 + e) : 0.f;
        uint4 o;
        o.x = pack_bf16x2(f[0], f[1]);
        o.y = pack_bf16x2(f[2], f[3]);
        o.z = pack_bf16x2(f[4], f[5]);
        o.w = pack_bf16x2(f[6], f[7]);
        Zb[idx] = o;
    }
}

struct WgArgs {
    float* partials;          // CLUSTER = false: [S][O][ldp]
    int64_t split_stride;
    int O, n_slabs, npad, tmem_cols, kblocks, kb_per_split, ldp;
    int stages;               // ring depth, 2..WG_STAGES: as deep as still lets two CTAs share an SM
    int tail_off;             // barriers etc. sit this far into the aligned shared memory (past ring and partial)
    int* status;
    // CLUSTER = true: the expansion
    const float* v;
    void* dW;
    int64_t lddw;
    int D, M, beta, splits;
};

template <typename WT> struct WgOut8;
template <> struct WgOut8<__nv_bfloat16> {
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
template <> struct WgOut8<float> {
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

// Four consecutive floats at the same shared-memory offset in CTA `rank` of the cluster.
__device__ __forceinline__ float4 ld_cluster_f32x4(uint32_t local_addr, uint32_t rank)
{
    uint32_t remote;
    float4 x;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_addr), "r"(rank));
    asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];"
                 : "=f"(x.x), "=f"(x.y), "=f"(x.z), "=f"(x.w) : "r"(remote) : "memory");
    return x;
}

// LPS, CH, WT describe the expansion (CLUSTER = true only): Dsub = 8 * LPS * CH, dW element type.
template <bool CLUSTER, int LPS, int CH, typename WT, int NT = WG_THREADS>
__global__ void __launch_bounds__(NT, NT == WG_THREADS ? 2 : 1)
wg_kernel(const __grid_constant__ CUtensorMap tmY, const __grid_constant__ CUtensorMap tmZ, const WgArgs a)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (base - raw);
    const int stage_bytes = WG_A_BYTES + a.n_slabs * WG_SLAB;
    uint8_t* tail = smem + a.tail_off;
    const uint32_t bars = base + a.tail_off;
    const uint32_t full = bars, empty = bars + 8 * WG_STAGES, tfull = bars + 16 * WG_STAGES;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tail + 16 * WG_STAGES + 16);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tail + 16 * WG_STAGES + 24);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int o0 = blockIdx.x * WG_BM;
    const int split = blockIdx.y;                            // = rank in the cluster when CLUSTER
    const int kb0 = split * a.kb_per_split;
    const int kb1 = (kb0 + a.kb_per_split < a.kblocks) ? kb0 + a.kb_per_split : a.kblocks;
    const int nkb = kb1 - kb0;                               // >= 1 by construction on the host

    if (threadIdx.x == 0) {
        for (int s = 0; s < WG_STAGES; ++s) {
            mbar_init(full + 8 * s, 1);
            mbar_init(empty + 8 * s, 1);
        }
        mbar_init(tfull, 1);
        *abort_flag = 0;
        fence_mbar_init();
        prefetch_tensormap(&tmY);
        prefetch_tensormap(&tmZ);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(tmem_slot), static_cast<uint32_t>(a.tmem_cols));
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    // Partial product of this CTA in its own shared memory (CLUSTER): rows of ldsp floats over the ring,
    // which is idle once the accumulator is complete.
    const int ldsp = a.npad + 4;

    bool failed = false;
    if (warp == 0) {
        if (lane == 0) {
            // The ring starts empty: fill it with dY tiles first, then wait for the kernel that writes Zb
            // (launched just before this one, which may overlap its tail) and add the Zb slabs.
            const int pre = nkb < a.stages ? nkb : a.stages;
            for (int it = 0; it < pre; ++it) {
                mbar_arrive_expect_tx(full + 8 * it, static_cast<uint32_t>(stage_bytes));
                const int k0 = (kb0 + it) * WG_BK;
                tma_load_2d(base + it * stage_bytes, &tmY, full + 8 * it, o0, k0);
                tma_load_2d(base + it * stage_bytes + WG_SLAB, &tmY, full + 8 * it, o0 + 64, k0);
            }
            pdl_wait();
            for (int it = 0; it < pre; ++it)
                for (int i = 0; i < a.n_slabs; ++i)
                    tma_load_2d(base + it * stage_bytes + WG_A_BYTES + i * WG_SLAB, &tmZ, full + 8 * it, 64 * i,
                                (kb0 + it) * WG_BK);
            int it = pre;
            uint32_t s = 0, ph = 1;                          // stage and phase parity of iteration `it` (= stages here)
            for (; it < nkb; ++it) {
                if (!mbar_wait(empty + 8 * s, ph ^ 1u, abort_flag)) { failed = true; break; }
                mbar_arrive_expect_tx(full + 8 * s, static_cast<uint32_t>(stage_bytes));
                const int k0 = (kb0 + it) * WG_BK;
                const uint32_t a_dst = base + s * stage_bytes;
                tma_load_2d(a_dst, &tmY, full + 8 * s, o0, k0);
                tma_load_2d(a_dst + WG_SLAB, &tmY, full + 8 * s, o0 + 64, k0);
                for (int i = 0; i < a.n_slabs; ++i)
                    tma_load_2d(a_dst + WG_A_BYTES + i * WG_SLAB, &tmZ, full + 8 * s, 64 * i, k0);
                if (++s == static_cast<uint32_t>(a.stages)) { s = 0; ph ^= 1u; }
            }
            if (failed) {
                *abort_flag = 1;
                const int back = it < a.stages ? it : a.stages;   // copies of this CTA still in flight
                for (int j = 1; j <= back; ++j) {
                    const int jt = it - j;
                    const unsigned long long t0 = globaltimer_ns();
                    while (!mbar_try_wait(full + 8 * (jt % a.stages), (jt / a.stages) & 1u))
                        if (globaltimer_ns() - t0 > kWaitLimitNs) break;
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_bf16(WG_BM, a.npad, true, true);
            uint32_t s = 0, ph = 0;
            for (int it = 0; it < nkb; ++it) {
                if (!mbar_wait(full + 8 * s, ph, abort_flag)) { failed = true; break; }
                tc_fence_after_sync();
                const uint32_t a_addr = base + s * stage_bytes, b_addr = a_addr + WG_A_BYTES;
#pragma unroll
                for (int j = 0; j < WG_BK / 16; ++j) {
                    const uint64_t da = umma_smem_desc(a_addr + j * 2048, WG_SLAB, 1024);
                    const uint64_t db = umma_smem_desc(b_addr + j * 2048, WG_SLAB, 1024);
                    umma_bf16(tmem_base, da, db, idesc, (it | j) != 0);
                }
                umma_commit(empty + 8 * s);
                if (++s == static_cast<uint32_t>(a.stages)) { s = 0; ph ^= 1u; }
            }
            if (!failed) umma_commit(tfull);
            else *abort_flag = 1;
        }
    } else if (warp < 6) {
        const int quarter = warp & 3;
        if (!mbar_wait_warp(tfull, 0u, abort_flag, 256)) {
            failed = true;
            *abort_flag = 1;
        } else {
            tc_fence_after_sync();
            const int trow = quarter * 32 + lane;
            const int o = o0 + trow;
            const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
            float* prow = CLUSTER ? reinterpret_cast<float*>(smem) + trow * ldsp
                                  : a.partials + split * a.split_stride + static_cast<int64_t>(o) * a.ldp;
            for (int c = 0; c * 32 < a.npad; ++c) {
                uint32_t r[32];
                tmem_ld_32x32(taddr + c * 32, r);
                tmem_ld_wait();
                if (CLUSTER || o < a.O) {
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        if (c * 32 + 4 * i < a.npad)               // npad is a multiple of 16
                            *reinterpret_cast<float4*>(prow + c * 32 + 4 * i) =
                                make_float4(__uint_as_float(r[4 * i]), __uint_as_float(r[4 * i + 1]),
                                            __uint_as_float(r[4 * i + 2]), __uint_as_float(r[4 * i + 3]));
                }
            }
        }
    }
    if (failed && a.status) atomicExch(a.status, VELORA_ERR_TIMEOUT);

    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    if (warp == 1) {
        __syncwarp();
        tmem_dealloc(tmem_base, static_cast<uint32_t>(a.tmem_cols));
    }

    if (CLUSTER) {
        // Every CTA reaches both cluster barriers whatever happened above (a timed-out role only skips
        // its own loop), so the cluster cannot deadlock on a CTA that gave up.
        namespace cg = cooperative_groups;
        cg::cluster_group cluster = cg::this_cluster();
        cluster.sync();                                      // all partials of the tile are in shared memory

        constexpr int L = LPS * CH;
        constexpr int SPW = 32 / LPS;
        const int q = lane & (LPS - 1), sub = lane / LPS;
        float vr[CH][8];
#pragma unroll
        for (int i = 0; i < CH; ++i)
#pragma unroll
            for (int e = 0; e < 8; ++e) vr[i][e] = __ldg(a.v + 8 * (q + LPS * i) + e);

        const int rows_per = (WG_BM + a.splits - 1) / a.splits;
        const int r_begin = split * rows_per;
        const int r_end = (r_begin + rows_per < WG_BM) ? r_begin + rows_per : WG_BM;
        WT* dW = static_cast<WT*>(a.dW);

        // Sum the partials of this CTA's rows, all threads at once and all loads of an element in flight
        // together (a remote load takes a good part of a microsecond; issued one after the other they
        // outlast the whole dY stream).  The sum replaces this CTA's own partial of those rows, which no
        // other CTA reads.
        float* sp = reinterpret_cast<float*>(smem);
        if (a.splits > 1) {
            const int c4n = a.npad / 4;
            for (int idx = threadIdx.x; idx < (r_end - r_begin) * c4n; idx += NT) {
                const int r = idx / c4n, c4 = idx - r * c4n;
                const int off = (r_begin + r) * ldsp + c4 * 4;
                const uint32_t laddr = base + static_cast<uint32_t>(off * 4);
                float4 x[WG_MAX_SPLITS];
#pragma unroll
                for (int s = 0; s < WG_MAX_SPLITS; ++s)
                    x[s] = (s < a.splits) ? ld_cluster_f32x4(laddr, static_cast<uint32_t>(s)) : make_float4(0.f, 0.f, 0.f, 0.f);
                float4 t = x[0];
#pragma unroll
                for (int s = 1; s < WG_MAX_SPLITS; ++s) {          // fixed order
                    t.x += x[s].x; t.y += x[s].y; t.z += x[s].z; t.w += x[s].w;
                }
                *reinterpret_cast<float4*>(sp + off) = t;
            }
            __syncthreads();
        }
        for (int trow = r_begin + warp; trow < r_end; trow += NT / 32) {
            const int o = o0 + trow;
            if (o >= a.O) break;
            for (int m0 = 0; m0 < a.M; m0 += 32) {
                const float p = (m0 + lane < a.M) ? sp[trow * ldsp + m0 + lane] : 0.f;
                WT* ptr = dW + static_cast<int64_t>(o) * a.lddw + (static_cast<int64_t>(m0 + sub) * L + q) * 8;
#pragma unroll 8
                for (int it = 0; it < LPS; ++it, ptr += SPW * L * 8) {
                    const int ms = it * SPW + sub;
                    const float pm = __shfl_sync(0xffffffffu, p, ms);
                    if (m0 + ms >= a.M) continue;
#pragma unroll
                    for (int i = 0; i < CH; ++i) {
                        const int col = ((m0 + ms) * L + q + LPS * i) * 8;
                        float y[8];
#pragma unroll
                        for (int e = 0; e < 8; ++e) y[e] = pm * vr[i][e];
                        if (col + 8 <= a.D) {
                            WgOut8<WT>::store(ptr + i * LPS * 8, y, a.beta);
                        } else {
#pragma unroll
                            for (int e = 0; e < 8; ++e)
                                if (col + e < a.D) {
                                    WT* pe = ptr + i * LPS * 8 + e;
                                    float f = y[e];
                                    if (a.beta) f += Elem<WT>::load(pe);
                                    Elem<WT>::store(pe, f);
                                }
                        }
                    }
                }
            }
        }
        cluster.sync();                                      // nobody leaves while its partial is still being read
    }
}

// P[o, m] = beta * P[o, m] + sum_s partials[s][o][m], splits added in a fixed order.
__global__ void __launch_bounds__(256)
reduce_partials_kernel(const float* __restrict__ partials, int splits, int64_t split_stride, int ldpart,
                       int O, int M, float* __restrict__ P, int64_t ldp, int beta)
{
    const int64_t total = static_cast<int64_t>(O) * M;
    const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
    for (int64_t idx = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; idx < total; idx += stride) {
        const int o = static_cast<int>(idx / M);
        const int m = static_cast<int>(idx - static_cast<int64_t>(o) * M);
        float p = beta ? P[o * ldp + m] : 0.f;
        for (int s = 0; s < splits; ++s) p += __ldg(partials + s * split_stride + static_cast<int64_t>(o) * ldpart + m);
        P[o * ldp + m] = p;
    }
}

struct WgPlan {
    bool ok;
    int M, npad, pitch, n_slabs, tmem_cols, kblocks, splits, kb_per_split, tiles_o, stages, tail_off;
    bool after_conversion;    // the launch follows z_to_bf16_kernel in the stream
    bool fat;                 // one CTA of twelve warps per SM instead of two CTAs of six
    size_t zb_bytes, part_bytes, smem;
};

WgPlan make_plan(int64_t N, int64_t D, int64_t O, int Dsub, int sm_count)
{
    WgPlan p{};
    const int64_t M = ceil_div64(D, Dsub);
    if (M > WG_MAX_M || N < 1 || N > (1 << 30) || O > (1 << 30)) return p;
    p.M = static_cast<int>(M);
    p.npad = static_cast<int>(round_up(M, 16));
    p.pitch = static_cast<int>(round_up(M, 64));
    p.n_slabs = p.pitch / 64;
    p.tmem_cols = 32;
    while (p.tmem_cols < p.npad) p.tmem_cols *= 2;
    p.kblocks = static_cast<int>(ceil_div64(N, WG_BK));
    p.tiles_o = static_cast<int>(ceil_div64(O, WG_BM));
    // Shared memory holds the ring and, afterwards, the CTA's partial product (128 rows of npad + 4 floats).
    // The ring is as deep as still lets two CTAs share an SM (down to two stages: with two CTAs pulling,
    // as many bytes are in flight per SM as with one CTA and four stages, and twice the warps write dW).
    const size_t stage_bytes = WG_A_BYTES + static_cast<size_t>(p.n_slabs) * WG_SLAB;
    const size_t partial_bytes = static_cast<size_t>(WG_BM) * (p.npad + 4) * 4;
    auto smem_for = [&](int stages) {
        const size_t body = stages * stage_bytes > partial_bytes ? stages * stage_bytes : partial_bytes;
        return 1024 + ((body + 1023) / 1024) * 1024 + 256;
    };
    p.stages = WG_STAGES;
    // One CTA per SM with twelve warps and half as many splits where the partial products are large (more than
    // 64 sub-tokens) and there are few row blocks: the traffic of the cluster reduction halves, the ring is twice as
    // deep and as many warps write dW (47 against 51 us on a 4096 x 11008 gradient with 172 sub-tokens).
    p.fat = p.npad > 64 && static_cast<int64_t>(p.tiles_o) * 4 <= sm_count;
    const bool fat = p.fat;
    if (!fat)
    while (p.stages > 2 && 2 * (smem_for(p.stages) + 1024) > 228 * 1024) --p.stages;
    if (2 * (smem_for(p.stages) + 1024) > 228 * 1024) { p.stages = WG_STAGES; p.fat = true; }      // one CTA per SM either way: twelve warps
    p.smem = smem_for(p.stages);
    p.tail_off = static_cast<int>(p.smem - 1024 - 256);
    const int64_t slots = static_cast<int64_t>(sm_count) * ((!fat && 2 * (p.smem + 1024) <= 228 * 1024) ? 2 : 1);
    // Pick the split count that fills whole waves of SMs best; ties go to fewer splits (fewer partials).
    int best = 1;
    double best_eff = 0.0;
    for (int s = 1; s <= WG_MAX_SPLITS && s <= p.kblocks; ++s) {
        const int64_t ctas = static_cast<int64_t>(p.tiles_o) * s;
        const int64_t waves = ceil_div64(ctas, slots);
        const double eff = static_cast<double>(ctas) / static_cast<double>(waves * slots) - 0.01 * s;
        if (eff > best_eff + 1e-9) { best_eff = eff; best = s; }
    }
    p.kb_per_split = static_cast<int>(ceil_div64(p.kblocks, best));
    p.splits = static_cast<int>(ceil_div64(p.kblocks, p.kb_per_split));
    p.zb_bytes = static_cast<size_t>(round_up(static_cast<int64_t>(N) * p.pitch * 2, 256));
    p.part_bytes = static_cast<size_t>(WG_MAX_SPLITS) * static_cast<size_t>(O) * p.npad * sizeof(float);
    p.ok = true;
    return p;
}

template <bool CLUSTER, int LPS, int CH, typename WT, int NT = WG_THREADS>
int launch_wg(const CUtensorMap& tmY, const CUtensorMap& tmZ, const WgArgs& a, const WgPlan& p, int smem_optin,
              cudaStream_t stream)
{
    static DeviceOnce configured;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return VELORA_ERR_CUDA;
    auto kern = wg_kernel<CLUSTER, LPS, CH, WT, NT>;
    if (!configured.get(dev)) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_optin) != cudaSuccess)
            return VELORA_ERR_CUDA;
        configured.set(dev);
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(p.tiles_o), static_cast<unsigned>(p.splits), 1);
    cfg.blockDim = dim3(NT, 1, 1);
    cfg.dynamicSmemBytes = p.smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 1;
    attr[0].val.clusterDim.y = CLUSTER ? static_cast<unsigned>(p.splits) : 1u;
    attr[0].val.clusterDim.z = 1;
    // Programmatic dependent launch, only behind this file's own Z conversion (which is launched the
    // ordinary way, so everything before it has completed): the kernel may then start while the conversion
    // is finishing, pulls dY at once and reads Zb only after pdl_wait().  Behind any other kernel it is
    // launched the ordinary way, because dY is read before the wait.
    attr[1] = pdl_attribute();
    cfg.attrs = attr;
    cfg.numAttrs = p.after_conversion ? 2 : 1;
    if (cudaLaunchKernelEx(&cfg, kern, tmY, tmZ, a) != cudaSuccess) {
        cudaGetLastError();
        return VELORA_ERR_CUDA;
    }
    return after_launch();
}

}  // namespace

size_t weight_grad_tc_workspace_bytes(int64_t N, int64_t D, int64_t O, int Dsub)
{
    const WgPlan p = make_plan(N > 0 ? N : 1, D, O, Dsub, 148);
    if (!p.ok) return 0;
    return p.zb_bytes + static_cast<size_t>(round_up(static_cast<int64_t>(p.part_bytes), 256));
}

int launch_weight_grad_tc(const void* dY, int dy_dtype, int64_t N, int64_t O, int64_t lddy,
                          const void* Z, int z_dtype, int64_t ldz, const float* v, int64_t D, int Dsub,
                          void* dW, int dw_dtype, int64_t lddw, int beta,
                          void* ws, size_t ws_bytes, int* status, cudaStream_t stream,
                          float* P_out, int64_t ldp_out)
{
    if (dy_dtype != VELORA_BF16 || N < 1) return VELORA_ERR_UNSUPPORTED;
    if (!tc_operand_ok(dY, lddy)) return VELORA_ERR_UNSUPPORTED;
    DeviceInfo di;
    int rc = device_info(&di);
    if (rc != VELORA_OK) return rc;
    const WgPlan p = make_plan(N, D, O, Dsub, di.sm_count);
    if (!p.ok) return VELORA_ERR_UNSUPPORTED;
    if (ws_bytes < weight_grad_tc_workspace_bytes(N, D, O, Dsub) || !aligned16(ws)) return VELORA_ERR_WORKSPACE;
    if (p.smem > static_cast<size_t>(di.smem_optin)) return VELORA_ERR_UNSUPPORTED;

    uint4* Zb = static_cast<uint4*>(ws);
    float* partials = reinterpret_cast<float*>(static_cast<char*>(ws) + p.zb_bytes);

    // 1. Z -> bf16, padded to whole 64-wide slabs.  A bf16 Z whose rows TMA can address is read in place
    //    (columns beyond M are zero-filled by the tensor map).
    const bool z_in_place = z_dtype == VELORA_BF16 && tc_operand_ok(Z, ldz);
    if (!z_in_place) {
        const int64_t items = N * (p.pitch / 8);
        int64_t grid = ceil_div64(items, 256);
        const int64_t cap = static_cast<int64_t>(di.sm_count) * 8;
        if (grid > cap) grid = cap;
        if (z_dtype == VELORA_F32)
            z_to_bf16_kernel<float><<<static_cast<int>(grid), 256, 0, stream>>>(
                static_cast<const float*>(Z), ldz, N, p.M, p.pitch, Zb);
        else if (z_dtype == VELORA_FP8_E4M3)                  // every E4M3 value is a bf16 value: exact
            z_to_bf16_kernel<e4m3_t><<<static_cast<int>(grid), 256, 0, stream>>>(
                static_cast<const e4m3_t*>(Z), ldz, N, p.M, p.pitch, Zb);
        else
            z_to_bf16_kernel<__nv_bfloat16><<<static_cast<int>(grid), 256, 0, stream>>>(
                static_cast<const __nv_bfloat16*>(Z), ldz, N, p.M, p.pitch, Zb);
        rc = after_launch();
        if (rc != VELORA_OK) return rc;
    }

    WgPlan plan = p;
    plan.after_conversion = !z_in_place;
    CUtensorMap tmY, tmZ;
    rc = make_tmap_bf16_2d(&tmY, dY, O, N, lddy, 64, WG_BK);
    if (rc != VELORA_OK) return rc;
    rc = z_in_place ? make_tmap_bf16_2d(&tmZ, Z, p.M, N, ldz, 64, WG_BK)
                    : make_tmap_bf16_2d(&tmZ, Zb, p.pitch, N, p.pitch, 64, WG_BK);
    if (rc != VELORA_OK) return rc;

    WgArgs a{};
    a.partials = partials;
    a.split_stride = static_cast<int64_t>(O) * p.npad;
    a.O = static_cast<int>(O);
    a.n_slabs = p.n_slabs;
    a.npad = p.npad;
    a.tmem_cols = p.tmem_cols;
    a.kblocks = p.kblocks;
    a.kb_per_split = p.kb_per_split;
    a.stages = p.stages;
    a.tail_off = p.tail_off;
    a.ldp = p.npad;
    a.status = status;
    a.v = v;
    a.dW = dW;
    a.lddw = lddw;
    a.D = static_cast<int>(D);
    a.M = p.M;
    a.beta = beta;
    a.splits = p.splits;

    if (P_out) {
        // The factor alone: P = beta * P + dY^T Z (kept across micro-batches, expanded once by the caller).
        rc = launch_wg<false, 1, 1, float>(tmY, tmZ, a, plan, di.smem_optin, stream);
        if (rc != VELORA_OK) return rc;
        const int64_t total = O * p.M;
        int64_t grid = ceil_div64(total, 256);
        const int64_t cap = static_cast<int64_t>(di.sm_count) * 8;
        if (grid > cap) grid = cap;
        reduce_partials_kernel<<<static_cast<int>(grid), 256, 0, stream>>>(
            partials, p.splits, a.split_stride, p.npad, static_cast<int>(O), p.M, P_out, ldp_out, beta);
        return after_launch();
    }
    // 2a. one launch: cluster of the tile's splits, reduction through distributed shared memory
    const int L = (Dsub % 8 == 0) ? Dsub / 8 : 0;
    const bool vec = L >= 1 && L <= 128 && (L & (L - 1)) == 0 && aligned16(dW) &&
                     (lddw * static_cast<int64_t>(dtype_size(dw_dtype))) % 16 == 0 &&
                     static_cast<size_t>(WG_BM) * (p.npad + 4) * 4 <= static_cast<size_t>(p.tail_off);
    if (vec) {
        const int lps = L < 32 ? L : 32, ch = L / lps;
        rc = VELORA_ERR_CUDA;
#define VELORA_WG_CASE(LPSV, CHV)                                                                             \
        if (lps == LPSV && ch == CHV) {                                                                       \
            if (plan.fat)                                                                                     \
                rc = dw_dtype == VELORA_BF16                                                                  \
                         ? launch_wg<true, LPSV, CHV, __nv_bfloat16, 2 * WG_THREADS>(tmY, tmZ, a, plan, di.smem_optin, stream) \
                         : launch_wg<true, LPSV, CHV, float, 2 * WG_THREADS>(tmY, tmZ, a, plan, di.smem_optin, stream);        \
            else                                                                                              \
                rc = dw_dtype == VELORA_BF16                                                                  \
                         ? launch_wg<true, LPSV, CHV, __nv_bfloat16>(tmY, tmZ, a, plan, di.smem_optin, stream)   \
                         : launch_wg<true, LPSV, CHV, float>(tmY, tmZ, a, plan, di.smem_optin, stream);          \
        }
        VELORA_WG_CASE(1, 1);
        VELORA_WG_CASE(2, 1);
        VELORA_WG_CASE(4, 1);
        VELORA_WG_CASE(8, 1);
        VELORA_WG_CASE(16, 1);
        VELORA_WG_CASE(32, 1);
        VELORA_WG_CASE(32, 2);
        VELORA_WG_CASE(32, 4);
#undef VELORA_WG_CASE
        if (rc == VELORA_OK) return rc;          // a refused cluster launch falls through to the three-launch route
    }
    // 2b. partial products to the workspace, then 3. dW = (sum of partials) (x) v
    rc = launch_wg<false, 1, 1, float>(tmY, tmZ, a, plan, di.smem_optin, stream);
    if (rc != VELORA_OK) return rc;
    return launch_expand_p(partials, p.splits, static_cast<int64_t>(O) * p.npad, p.npad, v, O, D, Dsub,
                           dW, dw_dtype, lddw, beta, stream);
}

}  // namespace velora
