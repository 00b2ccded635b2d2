// Dense products of Algorithm 1 (arxiv 2405.17991) with CTA pairs: C[Mdim, Ndim] = A * B, bf16 in,
// fp32 accumulation, 256 x 256 output tile per pair of CTAs (a cluster of two on neighbouring SMs).
//
// tcgen05.mma with cta_group::2 lets the two tensor cores of a pair work on one tile: each CTA keeps
// its 128 rows of A and only HALF of the B tile (128 of the 256 columns) in its own shared memory and
// the hardware reads the other half from the peer.  Per CTA and K step that is 32 KB of operands instead
// of 48 KB for the same 128 x 256 x 64 multiply-accumulates: a third less L2 -> shared-memory traffic
// and shared-memory read bandwidth, which is what limits the single-CTA kernel, and room for a
// six-stage ring.  No TMA multicast is used: each CTA loads its own halves.
//
// Roles per CTA (192 threads): warp 0 lane 0 TMA producer, warp 1 lane 0 MMA issuer (leader CTA only),
// warps 2..5 epilogue.  Barriers live at the same shared-memory offsets in both CTAs:
//   full[s]    leader's copy is used: the leader posts the bytes of both CTAs' loads, every load (of
//              either CTA) completes on it.
//   empty[s]   one per CTA; the leader's tcgen05.commit arrives on both (multicast commit).
//   tfull[a]   one per CTA, same multicast commit: accumulator a of the pair is complete.
//   tempty[a]  leader's copy, 8 arrivals: the four epilogue warps of each CTA.
// Every wait is bounded; both CTAs always reach the closing cluster barrier.
//
// FUSE = 1 / 2 / 3 (forward only, both operands K-major): four more warps per CTA compute Z = compress(X, v)
// (fp32 / bf16 / E4M3 storage) for the row block the CTA is multiplying, from lines of X that are in L2 for
// the GEMM anyway, so X crosses HBM once for both results.  The CTA pair working on n-tile j handles the
// sub-token groups g with g % tiles_n == j.  These warps read X with plain 16-byte loads and share nothing
// with the GEMM's pipeline: no stage, no barrier, no producer work (a second copy of the X tile fetched by the
// TMA producer into a buffer of their own cost 4-9 % of the product's time).
#include <cooperative_groups.h>

#include "gemm_fuse.cuh"
#include "gemm_store.cuh"
#include "gemm_tc.cuh"
#include "tc_common.cuh"

namespace velora {

using namespace tc;

namespace {

constexpr int P_BM = 128;                 // rows per CTA (256 per pair)
constexpr int P_BN = 256;                 // columns per pair; 128 of them staged by each CTA
constexpr int P_BK = 64;
constexpr int P_STAGES = 6;
constexpr int P_A_BYTES = P_BM * P_BK * 2;          // 16 KB
constexpr int P_B_BYTES = (P_BN / 2) * P_BK * 2;    // 16 KB: this CTA's half of B
constexpr int P_STAGE_BYTES = P_A_BYTES + P_B_BYTES;
constexpr int P_SLAB = 64 * P_BK * 2;               // 8 KB, one 64-wide MN-major slab
constexpr int P_THREADS = 192;
constexpr int P_TMEM_COLS = 512;
constexpr int P_FUSE_THREADS = P_THREADS + 192;      // + four compress warps (6, 7, 10, 11) and two idle ones (8, 9)
constexpr size_t P_SMEM = 1024 + static_cast<size_t>(P_STAGES) * P_STAGE_BYTES + 256;
constexpr size_t P_FUSE_SMEM = P_SMEM;

__device__ __forceinline__ uint32_t map_to_cta(uint32_t local_addr, uint32_t rank)
{
    uint32_t remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_addr), "r"(rank));
    return remote;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr)
{
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// Tile load of a CTA pair: data to this CTA's shared memory, completion bytes to a barrier given by its
// cluster address (the leader's).
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* m, uint32_t bar_cluster, int c0, int c1)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(m)), "r"(bar_cluster), "r"(c0), "r"(c1)
        : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t slot_smem, uint32_t cols)
{
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot_smem), "r"(cols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair()
{
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t cols)
{
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void umma_bf16_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, bool accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate ? 1u : 0u)
        : "memory");
}
// Arrives on the barrier at this shared-memory offset in BOTH CTAs of the pair once the MMAs issued so
// far have completed.
__device__ __forceinline__ void umma_commit_pair(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"(static_cast<uint16_t>(3)) : "memory");
}

struct PairTile {
    int m0, n0;
};
// Pair tiles (256 x 256) walked in bands of 4 m-tiles so that pairs running together share B in L2.
__device__ __forceinline__ PairTile pair_tile(int tile, int tiles_m, int tiles_n)
{
    constexpr int BAND = 4;
    const int per_band = BAND * tiles_n;
    const int band = tile / per_band;
    const int in_band = tile - band * per_band;
    const int band_rows = (tiles_m - band * BAND < BAND) ? tiles_m - band * BAND : BAND;
    const int tn = in_band / band_rows;
    const int tm = band * BAND + (in_band - tn * band_rows);
    return {tm * 2 * P_BM, tn * P_BN};
}

template <bool A_MN, bool B_MN, typename CT, int FUSE>
__global__ void __launch_bounds__(FUSE ? P_FUSE_THREADS : P_THREADS, 1)
gemm_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                 CT* __restrict__ C, int64_t ldc, int beta, int Mdim, int Ndim, int Kdim,
                 int tiles_m, int tiles_n, int* __restrict__ status, const FuseArgs fz)
{
    static_assert(FUSE == 0 || (!A_MN && !B_MN), "compress rides on the K-major forward GEMM only");
    namespace cg = cooperative_groups;
    cg::cluster_group cluster = cg::this_cluster();
    const uint32_t rank = cluster.block_rank();              // 0 = leader
    const int pair = blockIdx.x >> 1;
    const int num_pairs = gridDim.x >> 1;

    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (base - raw);
    uint8_t* tail = smem + P_STAGES * P_STAGE_BYTES;
    const uint32_t bars = base + P_STAGES * P_STAGE_BYTES;
    const uint32_t full = bars, empty = bars + 8 * P_STAGES;
    const uint32_t tfull = bars + 16 * P_STAGES, tempty = tfull + 16;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tail + 16 * P_STAGES + 48);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tail + 16 * P_STAGES + 56);
    volatile int* tiles_started = reinterpret_cast<volatile int*>(tail + 16 * P_STAGES + 60);   // producer's progress, read by the compress warps

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int num_tiles = tiles_m * tiles_n;
    const int kblocks = (Kdim + P_BK - 1) / P_BK;

    if (threadIdx.x == 0) {
        for (int s = 0; s < P_STAGES; ++s) {
            mbar_init(full + 8 * s, 1);                      // the leader's expect_tx arrival
            mbar_init(empty + 8 * s, 1);                     // the leader's commit
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(tfull + 8 * a, 1);
            mbar_init(tempty + 8 * a, 8);                    // four epilogue warps of each CTA
        }
        *abort_flag = 0;
        *tiles_started = 0;
        fence_mbar_init();
        prefetch_tensormap(&tmA);
        prefetch_tensormap(&tmB);
    }
    if (warp == 1) {
        tmem_alloc_pair(smem_u32(tmem_slot), P_TMEM_COLS);
        tmem_relinquish_pair();
    }
    tc_fence_before_sync();
    __syncthreads();
    cluster.sync();                                          // both CTAs' barriers exist before anyone signals them
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    bool failed = false;
    if (warp == 0) {
        // ------------------------------------------------ TMA producer: this CTA's rows of A, its half of B
        if (lane == 0) {
            uint32_t it = 0;
            int started = 0;
            for (int tile = pair; tile < num_tiles && !failed; tile += num_pairs) {
                if (FUSE) *tiles_started = ++started;          // the compress warps may take this tile's row block now
                const PairTile t0 = pair_tile(tile, tiles_m, tiles_n);
                const int m0 = t0.m0 + static_cast<int>(rank) * P_BM;
                const int n0 = t0.n0 + static_cast<int>(rank) * (P_BN / 2);
                for (int kb = 0; kb < kblocks; ++kb, ++it) {
                    const uint32_t s = it % P_STAGES, ph = (it / P_STAGES) & 1u;
                    if (!mbar_wait(empty + 8 * s, ph ^ 1u, abort_flag)) { failed = true; break; }
                    const uint32_t lead_full = map_to_cta(full + 8 * s, 0);
                    if (rank == 0) mbar_arrive_expect_tx(full + 8 * s, 2 * P_STAGE_BYTES);
                    const int k0 = kb * P_BK;
                    const uint32_t a_dst = base + s * P_STAGE_BYTES, b_dst = a_dst + P_A_BYTES;
                    if (A_MN) {
#pragma unroll
                        for (int i = 0; i < P_BM / 64; ++i)
                            tma_load_2d_pair(a_dst + i * P_SLAB, &tmA, lead_full, m0 + 64 * i, k0);
                    } else {
                        tma_load_2d_pair(a_dst, &tmA, lead_full, k0, m0);
                    }
                    if (B_MN) {
#pragma unroll
                        for (int i = 0; i < P_BN / 128; ++i)
                            tma_load_2d_pair(b_dst + i * P_SLAB, &tmB, lead_full, n0 + 64 * i, k0);
                    } else {
                        tma_load_2d_pair(b_dst, &tmB, lead_full, k0, n0);
                    }
                }
            }
            if (failed) {
                *abort_flag = 1;
                // Let the copies in flight land before shared memory is given up: the ring's copies complete
                // on the leader's barriers, which the leader watches (each phase needs both CTAs' bytes) while
                // the peer allows them 50 us.
                const unsigned long long t0 = globaltimer_ns();
                if (rank == 0) {
                    const uint32_t back = it < P_STAGES ? it : P_STAGES;
                    for (uint32_t j = 1; j <= back; ++j) {
                        const uint32_t jt = it - j;
                        while (!mbar_try_wait(full + 8 * (jt % P_STAGES), (jt / P_STAGES) & 1u))
                            if (globaltimer_ns() - t0 > kWaitLimitNs) break;
                    }
                } else {
                    while (globaltimer_ns() - t0 < 50000ull) __nanosleep(1000);
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer: the leader's lane 0 drives both tensor cores
        if (lane == 0 && rank == 0) {
            constexpr uint32_t idesc = umma_idesc_bf16(2 * P_BM, P_BN, A_MN, B_MN);
            uint32_t it = 0, t = 0;
            for (int tile = pair; tile < num_tiles && !failed; tile += num_pairs, ++t) {
                const uint32_t acc = t & 1u, aph = (t >> 1) & 1u;
                if (!mbar_wait(tempty + 8 * acc, aph ^ 1u, abort_flag)) { failed = true; break; }
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + acc * P_BN;
                for (int kb = 0; kb < kblocks; ++kb, ++it) {
                    const uint32_t s = it % P_STAGES, ph = (it / P_STAGES) & 1u;
                    if (!mbar_wait(full + 8 * s, ph, abort_flag)) { failed = true; break; }
                    tc_fence_after_sync();
                    const uint32_t a_addr = base + s * P_STAGE_BYTES, b_addr = a_addr + P_A_BYTES;
#pragma unroll
                    for (int j = 0; j < P_BK / 16; ++j) {
                        const uint64_t da = A_MN ? umma_smem_desc(a_addr + j * 2048, P_SLAB, 1024)
                                                 : umma_smem_desc(a_addr + j * 32, 16, 1024);
                        const uint64_t db = B_MN ? umma_smem_desc(b_addr + j * 2048, P_SLAB, 1024)
                                                 : umma_smem_desc(b_addr + j * 32, 16, 1024);
                        umma_bf16_pair(d_tmem, da, db, idesc, (kb | j) != 0);
                    }
                    umma_commit_pair(empty + 8 * s);          // both CTAs may refill the stage
                }
                if (failed) break;
                umma_commit_pair(tfull + 8 * acc);            // both CTAs may read their half of the accumulator
            }
            if (failed) *abort_flag = 1;
        }
    } else if (FUSE && (warp == 8 || warp == 9)) {
        // Idle on purpose.  A warp is served by the scheduler warp % 4; warps 8 and 9 would share schedulers 0
        // and 1 with the TMA producer and the MMA issuer, single threads on the kernel's critical path.  With
        // the compress on those two warps the product ran 5-6 % slower, on warps 10 and 11 it runs 1-2.5 % slower.
    } else if (FUSE && warp >= 6) {
        // ------------------------------------------------ compress (4 warps, 32 rows of the CTA's 128 each)
        const int cwi = warp < 8 ? warp - 6 : warp - 8;
        // For the row block of every tile this pair works on, these warps compress the column groups
        // g = tn, tn + tiles_n, ... (tn = the tile's n index), so that the tiles of a row block share the
        // work; they read X themselves and run beside the GEMM's pipeline without touching it.
        const int cpr = (fz.Dsub >> 3) < 8 ? 8 : (fz.Dsub >> 3);
        const int n_groups = (Kdim + 8 * cpr - 1) / (8 * cpr);
        auto walk = [&](auto vs) {
            vs.load(fz.v, fz.Dsub, lane);
            int ti = 0;
            for (int tile = pair; tile < num_tiles; tile += num_pairs, ++ti) {
                if (!wait_for_tile(tiles_started, ti, abort_flag)) { failed = true; break; }
                const PairTile t0 = pair_tile(tile, tiles_m, tiles_n);
                const int r0 = t0.m0 + static_cast<int>(rank) * P_BM + cwi * 32;
                if (r0 >= Mdim) continue;
                for (int g = t0.n0 / P_BN; g < n_groups; g += tiles_n)
                    compress_group_direct<FUSE>(fz, vs, r0, Mdim, Kdim, g, lane);
            }
        };
        if (fz.Dsub <= 256) walk(VSlice<1>{});
        else if (fz.Dsub == 512) walk(VSlice<2>{});
        else walk(VSlice<4>{});
    } else {
        // ------------------------------------------------ epilogue: this CTA's 128 rows of the pair tile
        const int quarter = warp & 3;
        const uint32_t lead_tempty0 = map_to_cta(tempty, 0);
        uint32_t t = 0;
        for (int tile = pair; tile < num_tiles && !failed; tile += num_pairs, ++t) {
            const PairTile t0 = pair_tile(tile, tiles_m, tiles_n);
            const uint32_t acc = t & 1u, aph = (t >> 1) & 1u;
            if (!mbar_wait_warp(tfull + 8 * acc, aph, abort_flag, 256)) { failed = true; break; }
            tc_fence_after_sync();
            const int row = t0.m0 + static_cast<int>(rank) * P_BM + quarter * 32 + lane;
            const uint32_t taddr = tmem_base + acc * P_BN + (static_cast<uint32_t>(quarter * 32) << 16);
            CT* crow = C + static_cast<int64_t>(row) * ldc + t0.n0;
#pragma unroll 1
            for (int c = 0; c < P_BN / 32; ++c) {
                uint32_t r[32];
                tmem_ld_32x32(taddr + c * 32, r);
                tmem_ld_wait();
                if (c == P_BN / 32 - 1) {                     // accumulator fully read: tell the leader
                    tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) mbar_arrive_cluster(lead_tempty0 + 8 * acc);
                }
                const int valid = Ndim - (t0.n0 + c * 32);
                if (row < Mdim && valid > 0) Store32<CT>::run(crow + c * 32, r, valid, beta);
            }
        }
        if (failed) *abort_flag = 1;
    }
    if (failed && status) atomicExch(status, VELORA_ERR_TIMEOUT);

    tc_fence_before_sync();
    __syncthreads();
    cluster.sync();                                          // nobody signals or reads a CTA that has left
    tc_fence_after_sync();
    if (warp == 1) {
        __syncwarp();
        tmem_dealloc_pair(tmem_base, P_TMEM_COLS);
    }
}

template <bool A_MN, bool B_MN, typename CT, int FUSE = 0>
int launch_pair(const CUtensorMap& ta, const CUtensorMap& tb, void* C, int64_t ldc, int beta,
                int Mdim, int Ndim, int Kdim, int* status, int sm_count, cudaStream_t stream,
                const FuseArgs fz = FuseArgs{})
{
    constexpr size_t smem_bytes = FUSE ? P_FUSE_SMEM : P_SMEM;
    static DeviceOnce configured;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return VELORA_ERR_CUDA;
    auto kern = gemm_pair_kernel<A_MN, B_MN, CT, FUSE>;
    if (!configured.get(dev)) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem_bytes)) != cudaSuccess)
            return VELORA_ERR_CUDA;
        configured.set(dev);
    }
    const int tiles_m = (Mdim + 2 * P_BM - 1) / (2 * P_BM), tiles_n = (Ndim + P_BN - 1) / P_BN;
    const int64_t tiles = static_cast<int64_t>(tiles_m) * tiles_n;
    int pairs = sm_count / 2;
    if (tiles < pairs) pairs = static_cast<int>(tiles);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(2 * pairs), 1, 1);
    cfg.blockDim = dim3(FUSE ? P_FUSE_THREADS : P_THREADS, 1, 1);
    cfg.dynamicSmemBytes = smem_bytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, kern, ta, tb, static_cast<CT*>(C), ldc, beta, Mdim, Ndim, Kdim, tiles_m, tiles_n, status, fz) !=
        cudaSuccess) {
        cudaGetLastError();
        return VELORA_ERR_CUDA;
    }
    return after_launch();
}

}  // namespace

int launch_gemm_tc_pair(int kind, const void* A, int64_t lda, const void* B, int64_t ldb,
                        void* C, int c_dtype, int64_t ldc, int beta,
                        int64_t Mdim, int64_t Ndim, int64_t Kdim, int in_dtype, int* status, cudaStream_t stream)
{
    if (in_dtype != VELORA_BF16) return VELORA_ERR_UNSUPPORTED;
    if (Mdim < 1 || Ndim < 1 || Kdim < 1) return VELORA_ERR_UNSUPPORTED;
    if (Mdim > (1 << 30) || Ndim > (1 << 30) || Kdim > (1 << 30)) return VELORA_ERR_UNSUPPORTED;
    if (!tc_operand_ok(A, lda) || !tc_operand_ok(B, ldb)) return VELORA_ERR_UNSUPPORTED;
    if (!aligned16(C) || (ldc * static_cast<int64_t>(dtype_size(c_dtype))) % 16) return VELORA_ERR_UNSUPPORTED;
    DeviceInfo di;
    int rc = device_info(&di);
    if (rc != VELORA_OK) return rc;
    if (static_cast<size_t>(di.smem_optin) < P_SMEM || di.sm_count < 2) return VELORA_ERR_UNSUPPORTED;

    const bool a_mn = (kind == GEMM_TN_MN_MN);
    const bool b_mn = (kind != GEMM_NT_K_K);
    CUtensorMap ta, tb;
    // K-major operand: [rows][K], box 64 (K) x 128 rows.  MN-major: [K][rows], box 64 x 64.
    rc = a_mn ? make_tmap_bf16_2d(&ta, A, Mdim, Kdim, lda, 64, P_BK) : make_tmap_bf16_2d(&ta, A, Kdim, Mdim, lda, P_BK, P_BM);
    if (rc != VELORA_OK) return rc;
    rc = b_mn ? make_tmap_bf16_2d(&tb, B, Ndim, Kdim, ldb, 64, P_BK) : make_tmap_bf16_2d(&tb, B, Kdim, Ndim, ldb, P_BK, P_BN / 2);
    if (rc != VELORA_OK) return rc;

    const int m = static_cast<int>(Mdim), n = static_cast<int>(Ndim), k = static_cast<int>(Kdim);
#define VELORA_PAIR_CASE(AMN, BMN)                                                                              \
    return c_dtype == VELORA_BF16                                                                               \
               ? launch_pair<AMN, BMN, __nv_bfloat16>(ta, tb, C, ldc, beta, m, n, k, status, di.sm_count, stream) \
               : launch_pair<AMN, BMN, float>(ta, tb, C, ldc, beta, m, n, k, status, di.sm_count, stream)
    if (!a_mn && !b_mn) { VELORA_PAIR_CASE(false, false); }
    if (!a_mn && b_mn) { VELORA_PAIR_CASE(false, true); }
    VELORA_PAIR_CASE(true, true);
#undef VELORA_PAIR_CASE
}

// Forward of the layer with compress fused in (see the kernel's header); returns VELORA_ERR_UNSUPPORTED
// without launching when the device cannot hold the kernel's shared memory.
int launch_linear_forward_tc_pair(const void* X, int64_t ldx, const void* W, int64_t ldw, const float* v,
                                  void* Y, int64_t ldy, void* Z, int z_dtype, int64_t ldz,
                                  int64_t N, int64_t D, int64_t O, int Dsub, int* status, cudaStream_t stream)
{
    DeviceInfo di;
    int rc = device_info(&di);
    if (rc != VELORA_OK) return rc;
    if (static_cast<size_t>(di.smem_optin) < P_FUSE_SMEM || di.sm_count < 2) return VELORA_ERR_UNSUPPORTED;
    CUtensorMap ta, tb;
    rc = make_tmap_bf16_2d(&ta, X, D, N, ldx, P_BK, P_BM);
    if (rc != VELORA_OK) return rc;
    rc = make_tmap_bf16_2d(&tb, W, D, O, ldw, P_BK, P_BN / 2);
    if (rc != VELORA_OK) return rc;
    FuseArgs fz{v, Z, ldz, Dsub, static_cast<int>((D + Dsub - 1) / Dsub), static_cast<const uint4*>(X), ldx / 8};
    const int m = static_cast<int>(N), n = static_cast<int>(O), k = static_cast<int>(D);
    if (z_dtype == VELORA_F32)
        return launch_pair<false, false, __nv_bfloat16, 1>(ta, tb, Y, ldy, 0, m, n, k, status, di.sm_count, stream, fz);
    if (z_dtype == VELORA_FP8_E4M3)
        return launch_pair<false, false, __nv_bfloat16, 3>(ta, tb, Y, ldy, 0, m, n, k, status, di.sm_count, stream, fz);
    return launch_pair<false, false, __nv_bfloat16, 2>(ta, tb, Y, ldy, 0, m, n, k, status, di.sm_count, stream, fz);
}

}  // namespace velora
