// Adapter-shaped layers (Section 4: VeLoRA on the down projections of trainable adapters, output width
// O = the adapter rank, 4 .. 64).  Two things live here, both from Algorithm 1 with a tiny O:
//
//  1. the factored weight gradient
//     P[o, m] = sum_n dY[n, o] * Z[n, m]            (O x M <= 64 x 256 values, a few MFLOP)
//     dW[o, m*Dsub + j] = beta*dW + P[o, m] * v[j]
// With one or two output tiles the tensor-core kernel of weight_grad_tc.cu cannot spread over the SMs (at
// most 8 CTAs pull on dY and Z); here the tokens are cut into up to 512 slices, each CTA forms the partial P of
// its slice on the CUDA cores, a second kernel adds the partials in a fixed order, and the common expansion
// kernel writes dW.  All sums are fp32, products are formed from the stored values (Z is not rounded to bf16).
//
//  2. the forward, Y = X W^T and Z = compress(X, v) in one pass over X (further down).
#include "common.cuh"
#include "gemm_fuse.cuh"
#include "gemm_tc.cuh"
#include "tc_common.cuh"

namespace velora {

using namespace tc;

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

// P[o*ldp + m] = beta * P + sum over the partials.  A block takes 32 consecutive elements; its eight warps
// each add every eighth partial (four loads in flight), then the eight sums are added in a fixed order: a
// thread per element walking all the partials one after the other took 12 us for 148 of them.
__global__ void __launch_bounds__(SK_THREADS)
wg_skinny_reduce_kernel(const float* __restrict__ partials, int parts, int O, int M, float* __restrict__ P,
                        int64_t ldp, int beta)
{
    __shared__ float sred[8][32];
    const int total = O * M;
    const int lane = threadIdx.x & 31, slice = threadIdx.x >> 5;
    const int idx = blockIdx.x * 32 + lane;
    float s = 0.f;
    if (idx < total) {
        for (int b = slice; b < parts; b += 32) {
            float x[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) x[u] = (b + 8 * u < parts) ? partials[static_cast<int64_t>(b + 8 * u) * total + idx] : 0.f;
#pragma unroll
            for (int u = 0; u < 4; ++u) s += x[u];
        }
    }
    sred[slice][lane] = s;
    __syncthreads();
    if (slice == 0 && idx < total) {
        float t = sred[0][lane];
#pragma unroll
        for (int w = 1; w < 8; ++w) t += sred[w][lane];
        const int o = idx / M, m = idx - o * M;
        float* p = P + static_cast<int64_t>(o) * ldp + m;
        *p = beta ? *p + t : t;
    }
}

// ------------------------------------------------------------------ forward of an adapter-shaped layer
// Y[N, O] = X W^T and Z = compress(X, v) for O <= 64 in ONE pass over X (Algorithm 1, forward).  The work is
// one HBM read of X; the product runs on tcgen05 with the roles of the operands swapped so that tokens are
// the N dimension of the MMA and 64-token tiles give every SM a CTA:
//     D[o, t] (TMEM, 128 lanes x 64 columns) += W_tile[o, k] * X_tile[t, k]      (M = 128, N = 64, K = 16)
// Only the first O lanes of the accumulator mean anything: the A descriptor spans 128 rows of shared memory
// but only round_up(O, 8) rows are loaded; whatever lies behind them feeds lanes that are never read.
// A stage holds 256 columns of the 64 tokens as four 8 KB tiles (64 rows x 128 bytes, 128-byte swizzle) plus
// the four W tiles.  Where D is a multiple of 64 ONE three-dimensional TMA box (64 elements x 64 rows x 4
// column chunks) brings the X tiles in, 512 contiguous bytes per token row: with one box per 128-byte-wide
// tile the same pass ran at 2.5 TB/s however deep the ring was.  Warp 0 produces, warp 1 issues the MMAs, the
// other sixteen warps compress: four sets of four warps take the stages in turn (a sub-token that spans
// several stages stays with one set; spreading the four tiles of a stage over the sets instead was slower,
// every set then waking for every stage).  Within a set a warp takes 16 of the 64 token rows; eight lanes per row
// read the row's eight 16-byte chunks of a tile in one instruction, multiply with their slice of v and add up
// over the lanes of a sub-token with shuffles.  They read the tiles in place and release the stage together
// with the MMA's commit (the kernel waits on HBM, so a stage held a little longer costs nothing here).  Warps 4
// and 5 finally read lanes 0..63 of the accumulator and store Y.
constexpr int SF_TOKENS = 64, SF_BK = 64, SF_SB = 4, SF_MAX_STAGES = 6;
constexpr int SF_X_BYTES = SF_TOKENS * SF_BK * 2;      // 8 KB: one tile
constexpr int SF_RING_BYTES = 200 * 1024;
constexpr int SF_SETS = 4;                             // compress warp sets (four warps each)
constexpr int SF_THREADS = 64 + SF_SETS * 128;
constexpr int SF_BAR_BYTES = 1024;                     // barriers, TMEM slot, abort flag
constexpr size_t SF_SMEM = 1024 + SF_RING_BYTES + 16384 /* A descriptor overhang */ + SF_BAR_BYTES + VELORA_MAX_DSUB * 4;

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* m, uint32_t bar, int c0, int c1, int c2)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(m)), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
        : "memory");
}

template <bool Z_BF16>
__global__ void __launch_bounds__(SF_THREADS, 1)
skinny_forward_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmX3,
                      const __grid_constant__ CUtensorMap tmW, int use3d,
                      __nv_bfloat16* __restrict__ Y, int64_t ldy, int N, int O, int D, int w_rows, int stages,
                      int* __restrict__ status, const FuseArgs fz)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (base - raw);
    constexpr int TAIL_OFF = SF_RING_BYTES + 16384;
    const int w_tile = (w_rows * 128 + 1023) & ~1023;
    const int stage_bytes = SF_SB * (SF_X_BYTES + w_tile);      // four X tiles, then four W tiles
    uint8_t* tail = smem + TAIL_OFF;
    const uint32_t bars = base + TAIL_OFF;
    const uint32_t full = bars, empty = bars + 8 * SF_MAX_STAGES, tfull = bars + 16 * SF_MAX_STAGES;
    // ready[set][s]: stage s holds landed tiles for compress set `set`.  Signalled by the MMA thread, which
    // sees every phase of full[s] in order; a set that only looked at full[s] for its own stages would skip
    // phases and could not tell them apart by parity.
    const uint32_t ready = tfull + 8;
    static_assert(8 * (2 * SF_MAX_STAGES + 1 + SF_SETS * SF_MAX_STAGES) + 16 <= SF_BAR_BYTES, "barrier area");
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tail + SF_BAR_BYTES - 16);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tail + SF_BAR_BYTES - 8);
    float* sv = reinterpret_cast<float*>(tail + SF_BAR_BYTES);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int t0 = blockIdx.x * SF_TOKENS;
    const int kblocks = (D + SF_BK - 1) / SF_BK;
    const int nsb = (kblocks + SF_SB - 1) / SF_SB;              // stages' worth of columns
    const int cw = fz.Dsub >= SF_BK ? fz.Dsub / SF_BK : 1;      // k-blocks per sub-token (a power of two)
    const int cwshift = 31 - __clz(cw);
    const uint32_t stage_tx = static_cast<uint32_t>(SF_SB * (SF_X_BYTES + w_rows * 128));
    // The set that compresses stage-load sb: sub-tokens longer than a stage stay with one set.
    auto set_of = [&](int sb) { return (cw > SF_SB ? (sb * SF_SB) >> cwshift : sb) & (SF_SETS - 1); };

    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) {
            mbar_init(full + 8 * s, 1);
            mbar_init(empty + 8 * s, 5);                         // the MMA commit + the four warps of a compress set
        }
        mbar_init(tfull, 1);
        for (int i = 0; i < SF_SETS * SF_MAX_STAGES; ++i) mbar_init(ready + 8 * i, 1);
        *abort_flag = 0;
        fence_mbar_init();
        prefetch_tensormap(&tmX);
        prefetch_tensormap(&tmX3);
        prefetch_tensormap(&tmW);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(tmem_slot), 64);
        tmem_relinquish();
    }
    for (int j = threadIdx.x; j < fz.Dsub; j += SF_THREADS) sv[j] = fz.v[j];
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    bool failed = false;
    if (warp == 0) {
        if (lane == 0) {
            int sb = 0;
            uint32_t s = 0, ph = 0;
            for (; sb < nsb; ++sb) {
                if (!mbar_wait(empty + 8 * s, ph ^ 1u, abort_flag)) { failed = true; break; }
                mbar_arrive_expect_tx(full + 8 * s, stage_tx);
                const uint32_t dst = base + s * stage_bytes;
                // Column chunks beyond D are zero-filled (and counted) like any other part of a box.
                if (use3d) {
                    tma_load_3d(dst, &tmX3, full + 8 * s, 0, t0, sb * SF_SB);
                } else {
#pragma unroll
                    for (int j = 0; j < SF_SB; ++j)
                        tma_load_2d(dst + j * SF_X_BYTES, &tmX, full + 8 * s, (sb * SF_SB + j) * SF_BK, t0);
                }
#pragma unroll
                for (int j = 0; j < SF_SB; ++j)
                    tma_load_2d(dst + SF_SB * SF_X_BYTES + j * w_tile, &tmW, full + 8 * s, (sb * SF_SB + j) * SF_BK, 0);
                if (++s == static_cast<uint32_t>(stages)) { s = 0; ph ^= 1u; }
            }
            if (failed) {
                *abort_flag = 1;
                const int back = sb < stages ? sb : stages;          // own copies still in flight
                for (int j = 1; j <= back; ++j) {
                    const int jt = sb - j;
                    const unsigned long long tb = globaltimer_ns();
                    while (!mbar_try_wait(full + 8 * (jt % stages), (jt / stages) & 1u))
                        if (globaltimer_ns() - tb > kWaitLimitNs) break;
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = umma_idesc_bf16(128, SF_TOKENS, false, false);
            uint32_t s = 0, ph = 0;
            for (int sb = 0; sb < nsb; ++sb) {
                if (!mbar_wait(full + 8 * s, ph, abort_flag)) { failed = true; break; }
                // Relaxed: a release in this thread would wait for the MMAs in flight.  The compress warps
                // take their acquire from full[s] itself.
                asm volatile("mbarrier.arrive.relaxed.cta.shared::cta.b64 _, [%0];"
                             ::"r"(ready + 8 * (set_of(sb) * SF_MAX_STAGES + s)) : "memory");
                tc_fence_after_sync();
                const uint32_t x0 = base + s * stage_bytes, w0 = x0 + SF_SB * SF_X_BYTES;
#pragma unroll
                for (int j = 0; j < SF_SB; ++j) {
                    if (sb * SF_SB + j >= kblocks) break;            // nothing but zero fill beyond D
#pragma unroll
                    for (int k = 0; k < SF_BK / 16; ++k)
                        umma_bf16(tmem_base, umma_smem_desc(w0 + j * w_tile + k * 32, 16, 1024),
                                  umma_smem_desc(x0 + j * SF_X_BYTES + k * 32, 16, 1024), idesc, (sb | j | k) != 0);
                }
                umma_commit(empty + 8 * s);
                if (++s == static_cast<uint32_t>(stages)) { s = 0; ph ^= 1u; }
            }
            if (!failed) umma_commit(tfull);
            else *abort_flag = 1;
        }
    } else {
        // ---- compress: warp cwp of a set takes tile rows 16 cwp .. 16 cwp + 15, four at a time, eight lanes per row
        const int cwp = (warp - 2) & 3, set = (warp - 2) >> 2;
        const int sub = lane >> 3, c = lane & 7;
        const int lanes_per_sub = fz.Dsub >= SF_BK ? 8 : fz.Dsub / 8;      // lanes that share a sub-token inside a row
        const int dshift = 31 - __clz(fz.Dsub);
        float acc[4] = {0.f, 0.f, 0.f, 0.f};                                // running sums of sub-tokens longer than a tile
        uint32_t s = 0, ph = 0, par = 0;                                    // par bit s: parity of ready[set][s]'s next phase
        for (int sb = 0; sb < nsb; ++sb) {
            if (set_of(sb) != set) {
                if (++s == static_cast<uint32_t>(stages)) { s = 0; ph ^= 1u; }
                continue;
            }
            if (!mbar_wait_warp(ready + 8 * (set * SF_MAX_STAGES + s), (par >> s) & 1u, abort_flag, 32)) { failed = true; break; }
            par ^= 1u << s;
            mbar_try_wait(full + 8 * s, ph);                     // complete by now: one probe acquires the tiles
            const uint32_t x0 = base + s * stage_bytes;
            float zval[SF_SB][4];
#pragma unroll
            for (int j = 0; j < SF_SB; ++j) {
                const int kb = sb * SF_SB + j;
                const int jv = (((kb & (cw - 1)) << 6) + c * 8) & (fz.Dsub - 1);   // this lane's chunk inside its sub-token
                const float4 va = *reinterpret_cast<const float4*>(sv + jv);
                const float4 vb = *reinterpret_cast<const float4*>(sv + jv + 4);
                // Four rows per lane, kept apart step by step (loads, products, shuffles) so that the
                // dependency chains overlap.
                uint4 d[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int r = 16 * cwp + 4 * i + sub;
                    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];"
                                 : "=r"(d[i].x), "=r"(d[i].y), "=r"(d[i].z), "=r"(d[i].w)
                                 : "r"(x0 + j * SF_X_BYTES + r * 128 + (static_cast<uint32_t>(c ^ (r & 7)) << 4)));
                }
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    float p0 = bf16_lo(d[i].x) * va.x, p1 = bf16_hi(d[i].x) * va.y;
                    p0 = fmaf(bf16_lo(d[i].y), va.z, p0); p1 = fmaf(bf16_hi(d[i].y), va.w, p1);
                    p0 = fmaf(bf16_lo(d[i].z), vb.x, p0); p1 = fmaf(bf16_hi(d[i].z), vb.y, p1);
                    p0 = fmaf(bf16_lo(d[i].w), vb.z, p0); p1 = fmaf(bf16_hi(d[i].w), vb.w, p1);
                    zval[j][i] = p0 + p1;
                }
                for (int off = lanes_per_sub >> 1; off >= 1; off >>= 1) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) zval[j][i] += __shfl_xor_sync(0xffffffffu, zval[j][i], off);
                }
                if (cw > 1) {
                    const bool last_of_sub = ((kb & (cw - 1)) == cw - 1) || kb >= kblocks - 1;
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        acc[i] += zval[j][i];
                        zval[j][i] = acc[i];
                        if (last_of_sub) acc[i] = 0.f;
                    }
                }
            }
            // Release the stage BEFORE the stores to Z: the arrival is a release, and a release issued behind
            // global stores waits until they have been performed.
            __syncwarp();                                        // every lane's reads of the tiles are done
            if (lane == 0) mbar_arrive(empty + 8 * s);
#pragma unroll
            for (int j = 0; j < SF_SB; ++j) {
                const int kb = sb * SF_SB + j;
                if (kb >= kblocks) break;
                const int m = cw == 1 ? (kb * SF_BK + c * 8) >> dshift : kb >> cwshift;
                const bool writer = cw == 1 ? (c & (lanes_per_sub - 1)) == 0
                                            : (c == 0 && (((kb & (cw - 1)) == cw - 1) || kb == kblocks - 1));
                if (writer && m < fz.M) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int row = t0 + 16 * cwp + 4 * i + sub;
                        if (row < N) {
                            if (Z_BF16) static_cast<__nv_bfloat16*>(fz.Z)[static_cast<int64_t>(row) * fz.ldz + m] = __float2bfloat16_rn(zval[j][i]);
                            else static_cast<float*>(fz.Z)[static_cast<int64_t>(row) * fz.ldz + m] = zval[j][i];
                        }
                    }
                }
            }
            if (++s == static_cast<uint32_t>(stages)) { s = 0; ph ^= 1u; }
        }
        if (failed) *abort_flag = 1;
        // ---- epilogue: warps 4 and 5 own TMEM lanes 0..31 and 32..63 (= output columns o)
        if (!failed && warp >= 4 && warp <= 5 && (warp - 4) * 32 < O) {
            if (!mbar_wait_warp(tfull, 0u, abort_flag, 64)) {
                failed = true;
                *abort_flag = 1;
            } else {
                tc_fence_after_sync();
                const int o = (warp - 4) * 32 + lane;
                const uint32_t taddr = tmem_base + (static_cast<uint32_t>((warp - 4) * 32) << 16);
#pragma unroll 1
                for (int cc = 0; cc < SF_TOKENS / 32; ++cc) {
                    uint32_t r[32];
                    tmem_ld_32x32(taddr + cc * 32, r);
                    tmem_ld_wait();
                    if (o < O) {
#pragma unroll
                        for (int i = 0; i < 32; ++i) {
                            const int t = t0 + cc * 32 + i;
                            if (t < N) Y[static_cast<int64_t>(t) * ldy + o] = __float2bfloat16_rn(__uint_as_float(r[i]));
                        }
                    }
                }
            }
        }
    }
    if (failed && status) atomicExch(status, VELORA_ERR_TIMEOUT);

    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    if (warp == 1) {
        __syncwarp();
        tmem_dealloc(tmem_base, 64);
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
    // One 32-token chunk per CTA where that gives at most 512 partials: the partial kernel is a single round
    // trip to memory plus a little arithmetic, so more, shorter CTAs finish sooner.
    (void)sm_count;
    int64_t tpc = ceil_div64(N, 512);
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
    // The token range is always cut into at most 512 slices, whatever the device, so the size is fixed.
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
    if (z_dtype == VELORA_FP8_E4M3)
        rc = dy_dtype == VELORA_BF16 ? launch_partial<__nv_bfloat16, e4m3_t>(p, dY, lddy, Z, ldz, n, o, partials, stream)
                                     : launch_partial<float, e4m3_t>(p, dY, lddy, Z, ldz, n, o, partials, stream);
    else if (dy_dtype == VELORA_BF16)
        rc = z_dtype == VELORA_BF16 ? launch_partial<__nv_bfloat16, __nv_bfloat16>(p, dY, lddy, Z, ldz, n, o, partials, stream)
                                    : launch_partial<__nv_bfloat16, float>(p, dY, lddy, Z, ldz, n, o, partials, stream);
    else
        rc = z_dtype == VELORA_BF16 ? launch_partial<float, __nv_bfloat16>(p, dY, lddy, Z, ldz, n, o, partials, stream)
                                    : launch_partial<float, float>(p, dY, lddy, Z, ldz, n, o, partials, stream);
    if (rc != VELORA_OK) return rc;
    const int total = o * p.M;
    const int grid = (total + 31) / 32;
    if (P_out) {
        wg_skinny_reduce_kernel<<<grid, SK_THREADS, 0, stream>>>(partials, p.parts, o, p.M, P_out, ldp_out, beta);
        return after_launch();
    }
    wg_skinny_reduce_kernel<<<grid, SK_THREADS, 0, stream>>>(partials, p.parts, o, p.M, P, p.M, 0);
    rc = after_launch();
    if (rc != VELORA_OK) return rc;
    return launch_expand_p(P, 1, 0, p.M, v, O, D, Dsub, dW, dw_dtype, lddw, beta, stream);
}

// Returns VELORA_ERR_UNSUPPORTED (nothing launched) unless the layer is adapter-shaped (O <= 64), bf16, with
// TMA-addressable rows and Dsub a power of two in 8 .. 1024.
int launch_linear_forward_skinny(const void* X, int64_t ldx, const void* W, int64_t ldw, const float* v,
                                 void* Y, int64_t ldy, void* Z, int z_dtype, int64_t ldz,
                                 int64_t N, int64_t D, int64_t O, int Dsub, int* status, cudaStream_t stream)
{
    const bool pow2 = Dsub >= 8 && Dsub <= VELORA_MAX_DSUB && (Dsub & (Dsub - 1)) == 0;
    if (!pow2 || O < 1 || O > 64 || N < 1 || N > (1 << 30) || D > (1 << 30)) return VELORA_ERR_UNSUPPORTED;
    if (z_dtype == VELORA_FP8_E4M3) return VELORA_ERR_UNSUPPORTED;     // 8-bit Z: product, then the compress kernel
    if (!tc_operand_ok(X, ldx) || !tc_operand_ok(W, ldw)) return VELORA_ERR_UNSUPPORTED;
    DeviceInfo di;
    int rc = device_info(&di);
    if (rc != VELORA_OK) return rc;
    if (static_cast<size_t>(di.smem_optin) < SF_SMEM) return VELORA_ERR_UNSUPPORTED;
    const int w_rows = static_cast<int>((O + 7) / 8 * 8);
    const int w_tile = (w_rows * 128 + 1023) & ~1023;
    int stages = SF_RING_BYTES / (SF_SB * (SF_X_BYTES + w_tile));
    if (stages > SF_MAX_STAGES) stages = SF_MAX_STAGES;
    CUtensorMap tx, tx3, tw;
    rc = make_tmap_bf16_2d(&tx, X, D, N, ldx, SF_BK, SF_TOKENS);
    if (rc != VELORA_OK) return rc;
    rc = make_tmap_bf16_2d(&tw, W, D, O, ldw, SF_BK, w_rows);
    if (rc != VELORA_OK) return rc;
    // One box for four 64-column tiles needs whole 64-column chunks; otherwise four two-dimensional boxes.
    int use3d = (D % SF_BK == 0 && make_tmap_bf16_chunks3d(&tx3, X, D, N, ldx, SF_TOKENS, SF_SB) == VELORA_OK) ? 1 : 0;
    if (!use3d) tx3 = tx;
    static DeviceOnce configured;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return VELORA_ERR_CUDA;
    if (!configured.get(dev)) {
        if (cudaFuncSetAttribute(skinny_forward_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(SF_SMEM)) != cudaSuccess ||
            cudaFuncSetAttribute(skinny_forward_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(SF_SMEM)) != cudaSuccess)
            return VELORA_ERR_CUDA;
        configured.set(dev);
    }
    FuseArgs fz{v, Z, ldz, Dsub, static_cast<int>(ceil_div64(D, Dsub))};
    const int grid = static_cast<int>(ceil_div64(N, SF_TOKENS));
    if (z_dtype == VELORA_BF16)
        skinny_forward_kernel<true><<<grid, SF_THREADS, SF_SMEM, stream>>>(
            tx, tx3, tw, use3d, static_cast<__nv_bfloat16*>(Y), ldy, static_cast<int>(N), static_cast<int>(O), static_cast<int>(D),
            w_rows, stages, status, fz);
    else
        skinny_forward_kernel<false><<<grid, SF_THREADS, SF_SMEM, stream>>>(
            tx, tx3, tw, use3d, static_cast<__nv_bfloat16*>(Y), ldy, static_cast<int>(N), static_cast<int>(O), static_cast<int>(D),
            w_rows, stages, status, fz);
    return after_launch();
}

}  // namespace velora
