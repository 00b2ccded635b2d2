// Dense products of Algorithm 1 (arxiv 2405.17991) on the sm_100a tensor cores:
//   Y = X W^T (forward), dX = dY W (input gradient), dW = dY^T Xhat (explicit weight gradient).
//
// One persistent, warp-specialised kernel: C[Mdim, Ndim] = A * B with bf16 operands and fp32
// accumulation.  Output tile 128 x 256, K step 64.  Warp 0 feeds a 4-stage shared-memory ring with
// TMA tile loads (128-byte swizzle); warp 1 issues tcgen05.mma (M = 128, N = 256, K = 16) into one of
// two 256-column TMEM accumulators; warps 2..5 drain the other accumulator with tcgen05.ld, convert
// and store, so the epilogue of a tile overlaps the main loop of the next.  Either operand may be
// K-major (rows contiguous along K) or MN-major (rows contiguous along M or N): the latter is loaded
// as 64 x 64 boxes and consumed through an MN-major matrix descriptor, so no transpose pass exists.
// Ragged edges rely on TMA zero fill for loads and on predicated stores.
#include "gemm_fuse.cuh"
#include "gemm_store.cuh"
#include "gemm_tc.cuh"
#include "tc_common.cuh"

namespace velora {

using namespace tc;

namespace {

constexpr int BM = 128, BN = 256, BK = 64, STAGES = 4;
constexpr int A_BYTES = BM * BK * 2;              // 16 KB
constexpr int B_BYTES = BN * BK * 2;              // 32 KB
constexpr int SLAB_BYTES = 64 * BK * 2;           // one 64-wide MN-major slab: 64 k-rows x 128 bytes
constexpr int GEMM_THREADS = 192;
constexpr int TMEM_COLS = 512;
constexpr int FUSE_THREADS = GEMM_THREADS + 192;    // + four compress warps (6, 7, 10, 11) and two idle ones (8, 9)
constexpr size_t GEMM_SMEM = 1024 + static_cast<size_t>(STAGES) * (A_BYTES + B_BYTES) + 256;
constexpr size_t FUSE_SMEM = GEMM_SMEM;

struct TileCoord {
    int m0, n0;
};

// Tiles are walked in bands of 8 m-tiles so that CTAs running together share B tiles in L2.
__device__ __forceinline__ TileCoord tile_coord(int tile, int tiles_m, int tiles_n)
{
    constexpr int BAND = 8;
    const int per_band = BAND * tiles_n;
    const int band = tile / per_band;
    const int in_band = tile - band * per_band;
    const int band_rows = (tiles_m - band * BAND < BAND) ? tiles_m - band * BAND : BAND;
    const int tn = in_band / band_rows;
    const int tm = band * BAND + (in_band - tn * band_rows);
    return {tm * BM, tn * BN};
}

// FUSE = 0: plain GEMM.  FUSE = 1 / 2 / 3 (forward only, A = X K-major): Z = compress(X, v) (fp32 / bf16 /
// E4M3 storage) is computed by four extra warps for the row block the CTA is multiplying, from lines of X
// that are on their way through L2 for the GEMM anyway, so X crosses HBM once for both results.  The CTA
// working on n-tile j handles the sub-token groups g with g % tiles_n == j, so the work is spread over the
// CTAs that share a row block.  The compress warps read X with plain 16-byte loads and keep v in registers:
// they share no stage, no barrier and no shared-memory bandwidth with the GEMM's pipeline (gemm_fuse.cuh),
// and they sit on warps 6, 7, 10, 11 so that none of them shares a warp scheduler (warp % 4) with the TMA
// producer (warp 0) or the MMA issuer (warp 1).
template <bool A_MN, bool B_MN, typename CT, int FUSE>
__global__ void __launch_bounds__(FUSE ? FUSE_THREADS : GEMM_THREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
               CT* __restrict__ C, int64_t ldc, int beta, int Mdim, int Ndim, int Kdim,
               int tiles_m, int tiles_n, int* __restrict__ status, const FuseArgs fz)
{
    static_assert(FUSE == 0 || (!A_MN && !B_MN), "compress rides on the K-major forward GEMM only");
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;               // swizzled tiles need 1024-byte alignment
    uint8_t* smem = smem_raw + (base - raw);
    const uint32_t sA = base;
    const uint32_t sB = base + STAGES * A_BYTES;
    uint8_t* tail = smem + STAGES * (A_BYTES + B_BYTES);
    const uint32_t bars = base + STAGES * (A_BYTES + B_BYTES);
    const uint32_t full = bars, empty = bars + 8 * STAGES;
    const uint32_t tfull = bars + 16 * STAGES, tempty = tfull + 16;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tail + 16 * STAGES + 48);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tail + 16 * STAGES + 56);
    volatile int* tiles_started = reinterpret_cast<volatile int*>(tail + 16 * STAGES + 60);   // producer's progress, read by the compress warps

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int num_tiles = tiles_m * tiles_n;
    const int kblocks = (Kdim + BK - 1) / BK;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(full + 8 * s, 1);
            mbar_init(empty + 8 * s, 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(tfull + 8 * a, 1);
            mbar_init(tempty + 8 * a, 4);
        }
        *abort_flag = 0;
        *tiles_started = 0;
        fence_mbar_init();
        prefetch_tensormap(&tmA);
        prefetch_tensormap(&tmB);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(tmem_slot), TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    bool failed = false;
    if (warp == 0) {
        // ------------------------------------------------ TMA producer (one lane)
        if (lane == 0) {
            uint32_t it = 0;
            int started = 0;
            for (int tile = blockIdx.x; tile < num_tiles && !failed; tile += gridDim.x) {
                if (FUSE) *tiles_started = ++started;          // the compress warps may take this tile's row block now
                const TileCoord tc0 = tile_coord(tile, tiles_m, tiles_n);
                for (int kb = 0; kb < kblocks; ++kb, ++it) {
                    const uint32_t s = it % STAGES, ph = (it / STAGES) & 1u;
                    if (!mbar_wait(empty + 8 * s, ph ^ 1u, abort_flag)) { failed = true; break; }
                    mbar_arrive_expect_tx(full + 8 * s, A_BYTES + B_BYTES);
                    const int k0 = kb * BK;
                    if (A_MN) {
#pragma unroll
                        for (int i = 0; i < BM / 64; ++i)
                            tma_load_2d(sA + s * A_BYTES + i * SLAB_BYTES, &tmA, full + 8 * s, tc0.m0 + 64 * i, k0);
                    } else {
                        tma_load_2d(sA + s * A_BYTES, &tmA, full + 8 * s, k0, tc0.m0);
                    }
                    if (B_MN) {
#pragma unroll
                        for (int i = 0; i < BN / 64; ++i)
                            tma_load_2d(sB + s * B_BYTES + i * SLAB_BYTES, &tmB, full + 8 * s, tc0.n0 + 64 * i, k0);
                    } else {
                        tma_load_2d(sB + s * B_BYTES, &tmB, full + 8 * s, k0, tc0.n0);
                    }
                }
            }
            if (failed) {
                *abort_flag = 1;
                // Let this CTA's own copies in flight land before shared memory is given up.
                const uint32_t back = it < STAGES ? it : STAGES;
                for (uint32_t j = 1; j <= back; ++j) {
                    const uint32_t jt = it - j;
                    const unsigned long long t0 = globaltimer_ns();
                    while (!mbar_try_wait(full + 8 * (jt % STAGES), (jt / STAGES) & 1u))
                        if (globaltimer_ns() - t0 > kWaitLimitNs) break;
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer (one lane)
        if (lane == 0) {
            constexpr uint32_t idesc = umma_idesc_bf16(BM, BN, A_MN, B_MN);
            uint32_t it = 0, t = 0;
            for (int tile = blockIdx.x; tile < num_tiles && !failed; tile += gridDim.x, ++t) {
                const uint32_t acc = t & 1u, aph = (t >> 1) & 1u;
                if (!mbar_wait(tempty + 8 * acc, aph ^ 1u, abort_flag)) { failed = true; break; }
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + acc * BN;
                for (int kb = 0; kb < kblocks; ++kb, ++it) {
                    const uint32_t s = it % STAGES, ph = (it / STAGES) & 1u;
                    if (!mbar_wait(full + 8 * s, ph, abort_flag)) { failed = true; break; }
                    tc_fence_after_sync();
                    const uint32_t a_addr = sA + s * A_BYTES, b_addr = sB + s * B_BYTES;
#pragma unroll
                    for (int j = 0; j < BK / 16; ++j) {
                        // K-major: 16 elements of K = 32 bytes inside the swizzled 128-byte row.
                        // MN-major: 16 k-rows of 128 bytes; 64-wide slabs are BK*128 bytes apart.
                        const uint64_t da = A_MN ? umma_smem_desc(a_addr + j * 2048, SLAB_BYTES, 1024)
                                                 : umma_smem_desc(a_addr + j * 32, 16, 1024);
                        const uint64_t db = B_MN ? umma_smem_desc(b_addr + j * 2048, SLAB_BYTES, 1024)
                                                 : umma_smem_desc(b_addr + j * 32, 16, 1024);
                        umma_bf16(d_tmem, da, db, idesc, (kb | j) != 0);
                    }
                    umma_commit(empty + 8 * s);           // the stage is free once these MMAs have read it
                }
                if (failed) break;
                umma_commit(tfull + 8 * acc);             // the accumulator is complete
            }
            if (failed) *abort_flag = 1;
        }
    } else if (FUSE && (warp == 8 || warp == 9)) {
        // Idle on purpose: these two would share warp schedulers 0 and 1 with the producer and the MMA issuer.
    } else if (FUSE && warp >= 6) {
        // ------------------------------------------------ compress (4 warps, 32 rows of the tile's 128 each)
        const int cwi = warp < 8 ? warp - 6 : warp - 8;
        const int cpr = (fz.Dsub >> 3) < 8 ? 8 : (fz.Dsub >> 3);
        const int n_groups = (Kdim + 8 * cpr - 1) / (8 * cpr);
        auto walk = [&](auto vs) {
            vs.load(fz.v, fz.Dsub, lane);
            int ti = 0;
            for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x, ++ti) {
                if (!wait_for_tile(tiles_started, ti, abort_flag)) { failed = true; break; }
                const TileCoord tc0 = tile_coord(tile, tiles_m, tiles_n);
                const int r0 = tc0.m0 + cwi * 32;
                if (r0 >= Mdim) continue;
                for (int g = tc0.n0 / BN; g < n_groups; g += tiles_n)
                    compress_group_direct<FUSE>(fz, vs, r0, Mdim, Kdim, g, lane);
            }
        };
        if (fz.Dsub <= 256) walk(VSlice<1>{});
        else if (fz.Dsub == 512) walk(VSlice<2>{});
        else walk(VSlice<4>{});
    } else {
        // ------------------------------------------------ epilogue (4 warps, one TMEM lane quarter each)
        const int quarter = warp & 3;
        uint32_t t = 0;
        for (int tile = blockIdx.x; tile < num_tiles && !failed; tile += gridDim.x, ++t) {
            const TileCoord tc0 = tile_coord(tile, tiles_m, tiles_n);
            const uint32_t acc = t & 1u, aph = (t >> 1) & 1u;
            if (!mbar_wait_warp(tfull + 8 * acc, aph, abort_flag, 256)) { failed = true; break; }
            tc_fence_after_sync();
            const int row = tc0.m0 + quarter * 32 + lane;
            const uint32_t taddr = tmem_base + acc * BN + (static_cast<uint32_t>(quarter * 32) << 16);
            CT* crow = C + static_cast<int64_t>(row) * ldc + tc0.n0;
#pragma unroll 1
            for (int c = 0; c < BN / 32; ++c) {
                uint32_t r[32];
                tmem_ld_32x32(taddr + c * 32, r);
                tmem_ld_wait();
                if (c == BN / 32 - 1) {                   // accumulator fully read: hand it back
                    tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(tempty + 8 * acc);
                }
                const int valid = Ndim - (tc0.n0 + c * 32);
                if (row < Mdim && valid > 0) Store32<CT>::run(crow + c * 32, r, valid, beta);
            }
        }
        if (failed) *abort_flag = 1;
    }
    if (failed && status) atomicExch(status, VELORA_ERR_TIMEOUT);

    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    if (warp == 1) {
        __syncwarp();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

// ------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

template <bool A_MN, bool B_MN, typename CT, int FUSE = 0>
int launch_kernel(const CUtensorMap& ta, const CUtensorMap& tb, void* C, int64_t ldc, int beta,
                  int Mdim, int Ndim, int Kdim, int* status, cudaStream_t stream, const FuseArgs fz = FuseArgs{})
{
    static DeviceOnce configured;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return VELORA_ERR_CUDA;
    auto kern = gemm_tc_kernel<A_MN, B_MN, CT, FUSE>;
    if (!configured.get(dev)) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 static_cast<int>(FUSE ? FUSE_SMEM : GEMM_SMEM)) != cudaSuccess)
            return VELORA_ERR_CUDA;
        configured.set(dev);
    }
    DeviceInfo di;
    int rc = device_info(&di);
    if (rc != VELORA_OK) return rc;
    const int tiles_m = (Mdim + BM - 1) / BM, tiles_n = (Ndim + BN - 1) / BN;
    const int64_t tiles = static_cast<int64_t>(tiles_m) * tiles_n;
    const int grid = static_cast<int>(tiles < di.sm_count ? tiles : di.sm_count);
    kern<<<grid, FUSE ? FUSE_THREADS : GEMM_THREADS, FUSE ? FUSE_SMEM : GEMM_SMEM, stream>>>(
        ta, tb, static_cast<CT*>(C), ldc, beta, Mdim, Ndim, Kdim, tiles_m, tiles_n, status, fz);
    return after_launch();
}

}  // namespace

int make_tmap_bf16_2d(CUtensorMap* map, const void* base, int64_t inner, int64_t outer, int64_t ld_elems,
                      int box_inner, int box_outer, bool swizzle128)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return VELORA_ERR_CUDA;
    const cuuint64_t gdim[2] = {static_cast<cuuint64_t>(inner), static_cast<cuuint64_t>(outer)};
    const cuuint64_t gstride[1] = {static_cast<cuuint64_t>(ld_elems) * 2};
    const cuuint32_t box[2] = {static_cast<cuuint32_t>(box_inner), static_cast<cuuint32_t>(box_outer)};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), gdim, gstride, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? VELORA_OK : VELORA_ERR_CUDA;
}

int make_tmap_bf16_chunks3d(CUtensorMap* map, const void* base, int64_t inner, int64_t outer, int64_t ld_elems,
                            int box_rows, int box_chunks)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return VELORA_ERR_CUDA;
    if (inner % 64) return VELORA_ERR_UNSUPPORTED;
    const cuuint64_t gdim[3] = {64, static_cast<cuuint64_t>(outer), static_cast<cuuint64_t>(inner / 64)};
    const cuuint64_t gstride[2] = {static_cast<cuuint64_t>(ld_elems) * 2, 128};
    const cuuint32_t box[3] = {64, static_cast<cuuint32_t>(box_rows), static_cast<cuuint32_t>(box_chunks)};
    const cuuint32_t estr[3] = {1, 1, 1};
    const CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), gdim, gstride, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? VELORA_OK : VELORA_ERR_UNSUPPORTED;
}

bool gemm_pair_preferred(int64_t Mdim, int64_t Ndim)
{
    DeviceInfo di;
    if (device_info(&di) != VELORA_OK) return false;
    const int64_t pair_tiles = ((Mdim + 255) / 256) * ((Ndim + 255) / 256);
    return pair_tiles >= di.sm_count / 2;
}

bool tc_operand_ok(const void* p, int64_t ld_elems)
{
    return aligned16(p) && ld_elems % 8 == 0 && ld_elems * 2 < (static_cast<int64_t>(1) << 40);
}

int launch_gemm_tc(int kind, const void* A, int64_t lda, const void* B, int64_t ldb,
                   void* C, int c_dtype, int64_t ldc, int beta,
                   int64_t Mdim, int64_t Ndim, int64_t Kdim, int in_dtype, int* status, cudaStream_t stream)
{
    if (in_dtype != VELORA_BF16) return VELORA_ERR_UNSUPPORTED;
    if (Mdim < 1 || Ndim < 1 || Kdim < 1) return VELORA_ERR_UNSUPPORTED;
    if (Mdim > (1 << 30) || Ndim > (1 << 30) || Kdim > (1 << 30)) return VELORA_ERR_UNSUPPORTED;
    if (!tc_operand_ok(A, lda) || !tc_operand_ok(B, ldb)) return VELORA_ERR_UNSUPPORTED;
    if (!aligned16(C) || (ldc * static_cast<int64_t>(dtype_size(c_dtype))) % 16) return VELORA_ERR_UNSUPPORTED;
    if ((static_cast<int64_t>((Mdim + BM - 1) / BM) * ((Ndim + BN - 1) / BN)) > (1 << 30)) return VELORA_ERR_UNSUPPORTED;

    if (gemm_pair_preferred(Mdim, Ndim)) {
        const int prc = launch_gemm_tc_pair(kind, A, lda, B, ldb, C, c_dtype, ldc, beta, Mdim, Ndim, Kdim, in_dtype, status, stream);
        if (prc != VELORA_ERR_UNSUPPORTED) return prc;
    }
    const bool a_mn = (kind == GEMM_TN_MN_MN);
    const bool b_mn = (kind != GEMM_NT_K_K);
    CUtensorMap ta, tb;
    int rc;
    // K-major operand: [rows = M or N][K], box 64 (K) x tile rows.  MN-major: [K][M or N], box 64 x 64.
    rc = a_mn ? make_tmap_bf16_2d(&ta, A, Mdim, Kdim, lda, 64, BK) : make_tmap_bf16_2d(&ta, A, Kdim, Mdim, lda, BK, BM);
    if (rc != VELORA_OK) return rc;
    rc = b_mn ? make_tmap_bf16_2d(&tb, B, Ndim, Kdim, ldb, 64, BK) : make_tmap_bf16_2d(&tb, B, Kdim, Ndim, ldb, BK, BN);
    if (rc != VELORA_OK) return rc;

    const int m = static_cast<int>(Mdim), n = static_cast<int>(Ndim), k = static_cast<int>(Kdim);
#define VELORA_GEMM_CASE(AMN, BMN)                                                                        \
    return c_dtype == VELORA_BF16                                                                         \
               ? launch_kernel<AMN, BMN, __nv_bfloat16>(ta, tb, C, ldc, beta, m, n, k, status, stream)    \
               : launch_kernel<AMN, BMN, float>(ta, tb, C, ldc, beta, m, n, k, status, stream)
    if (!a_mn && !b_mn) { VELORA_GEMM_CASE(false, false); }
    if (!a_mn && b_mn) { VELORA_GEMM_CASE(false, true); }
    VELORA_GEMM_CASE(true, true);
#undef VELORA_GEMM_CASE
}

int launch_linear_forward_tc(const void* X, int64_t ldx, const void* W, int64_t ldw, const float* v,
                             void* Y, int64_t ldy, void* Z, int z_dtype, int64_t ldz,
                             int dtype, int64_t N, int64_t D, int64_t O, int Dsub, int* status, cudaStream_t stream)
{
    // Fused path: Dsub a power of two between 8 and 1024 (sub-token boundaries then fall on 16-byte
    // chunks of the 64-column X tiles); everything else runs the GEMM and the compress kernel in turn.
    if (dtype == VELORA_BF16 && O <= 64) {               // adapter-shaped: one pass over X for Y and Z
        const int src = launch_linear_forward_skinny(X, ldx, W, ldw, v, Y, ldy, Z, z_dtype, ldz, N, D, O, Dsub, status, stream);
        if (src != VELORA_ERR_UNSUPPORTED) return src;
    }
    const bool pow2 = Dsub >= 8 && Dsub <= VELORA_MAX_DSUB && (Dsub & (Dsub - 1)) == 0;
    const bool gemm_ok = dtype == VELORA_BF16 && N >= 1 && N < (1 << 30) && D < (1 << 30) && O < (1 << 30) &&
                         tc_operand_ok(X, ldx) && tc_operand_ok(W, ldw) && aligned16(Y) && ldy % 8 == 0;
    // One CTA compresses one k-block in tiles_n; with fewer than four n-tiles the compress warps would
    // hold the producer back, so narrow outputs take the two-kernel route as well.
    const bool wide = (O + BN - 1) / BN >= 4;
    if (pow2 && gemm_ok && wide) {
        if (gemm_pair_preferred(N, O)) {
            const int prc = launch_linear_forward_tc_pair(X, ldx, W, ldw, v, Y, ldy, Z, z_dtype, ldz, N, D, O, Dsub, status, stream);
            if (prc != VELORA_ERR_UNSUPPORTED) return prc;
        }
        CUtensorMap ta, tb;
        int rc = make_tmap_bf16_2d(&ta, X, D, N, ldx, BK, BM);
        if (rc != VELORA_OK) return rc;
        rc = make_tmap_bf16_2d(&tb, W, D, O, ldw, BK, BN);
        if (rc != VELORA_OK) return rc;
        FuseArgs fz{v, Z, ldz, Dsub, static_cast<int>(ceil_div64(D, Dsub)), static_cast<const uint4*>(X), ldx / 8};
        const int m = static_cast<int>(N), n = static_cast<int>(O), k = static_cast<int>(D);
        if (z_dtype == VELORA_F32)
            return launch_kernel<false, false, __nv_bfloat16, 1>(ta, tb, Y, ldy, 0, m, n, k, status, stream, fz);
        if (z_dtype == VELORA_FP8_E4M3)
            return launch_kernel<false, false, __nv_bfloat16, 3>(ta, tb, Y, ldy, 0, m, n, k, status, stream, fz);
        return launch_kernel<false, false, __nv_bfloat16, 2>(ta, tb, Y, ldy, 0, m, n, k, status, stream, fz);
    }
    int rc = launch_gemm_tc(GEMM_NT_K_K, X, ldx, W, ldw, Y, dtype, ldy, 0, N, O, D, dtype, status, stream);
    if (rc != VELORA_OK) return rc;
    return launch_compress(X, dtype, N, D, ldx, Dsub, v, Z, z_dtype, ldz, stream);
}

}  // namespace velora
