// The compress (Section 3.1, Eq. 1) that rides on the forward GEMM's X tiles: arguments and the
// per-k-block arithmetic shared by the single-CTA and the CTA-pair kernels.
#pragma once

#include "common.cuh"

namespace velora {

struct FuseArgs {
    const float* v;
    void* Z;
    int64_t ldz;
    int Dsub, M;
};

// Which k-blocks are compressed during the work on n-tile tn?  Those of the sub-token groups g = kb / cw
// (cw = k-blocks per sub-token, a power of two) with g % tiles_n == tn, so that the tiles of one row block
// share the work.  Walked incrementally: the TMA producer is a single thread on the kernel's critical
// path, where two integer divisions per k-block cost 10 % of the run time.
struct OwnedWalk {
    int cwmask, tiles_n, tn, gm;
    __device__ __forceinline__ OwnedWalk(int cw, int tiles_n_, int tn_) : cwmask(cw - 1), tiles_n(tiles_n_), tn(tn_), gm(0) {}
    __device__ __forceinline__ bool owned() const { return gm == tn; }
    __device__ __forceinline__ void step(int kb_next)          // call when moving on to k-block kb_next
    {
        if ((kb_next & cwmask) == 0 && ++gm == tiles_n) gm = 0;
    }
};

// One thread, one row of a 128-row x 64-column bf16 X tile that TMA wrote with the 128-byte swizzle at
// `tile` (shared-memory address, 1024-byte aligned).  Adds the row's 64 columns of k-block `kb` into the
// running inner product `acc` with v (copy in shared memory `sv`, Dsub a power of two >= 8) and stores
// Z[row, m] whenever a sub-token ends inside the block.  cw = k-blocks per sub-token (1 if Dsub <= 64).
// ZK selects the storage type of Z: 1 fp32, 2 bf16, 3 E4M3 (the values of the kernels' FUSE parameter).
template <int ZK>
__device__ __forceinline__ void compress_kblock(uint32_t tile, int trow, const float* sv, const FuseArgs& fz,
                                                int cw, int kb, int kblocks, int row, int Mdim, float& acc)
{
    constexpr int BK = 64;
    const int Dsub = fz.Dsub;
    const uint32_t rowaddr = tile + trow * 128;
    uint4 d[8];
#pragma unroll
    for (int c = 0; c < 8; ++c) {
        // Chunk c of row r sits at chunk position c ^ (r & 7): conflict-free 16-byte reads.
        const uint32_t a = rowaddr + (static_cast<uint32_t>(c ^ (trow & 7)) << 4);
        asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];"
                     : "=r"(d[c].x), "=r"(d[c].y), "=r"(d[c].z), "=r"(d[c].w) : "r"(a));
    }
    const int j0 = (kb % cw) * BK;                 // position of this k-block inside the sub-token
    if (kb % cw == 0) acc = 0.f;
#pragma unroll
    for (int c = 0; c < 8; ++c) {
        const int jv = (j0 + c * 8) & (Dsub - 1);
        const float4 va = *reinterpret_cast<const float4*>(sv + jv);
        const float4 vb = *reinterpret_cast<const float4*>(sv + jv + 4);
        if (Dsub < BK && jv == 0) acc = 0.f;       // a new sub-token starts inside the k-block
        float a0 = bf16_lo(d[c].x) * va.x, a1 = bf16_hi(d[c].x) * va.y;
        a0 = fmaf(bf16_lo(d[c].y), va.z, a0); a1 = fmaf(bf16_hi(d[c].y), va.w, a1);
        a0 = fmaf(bf16_lo(d[c].z), vb.x, a0); a1 = fmaf(bf16_hi(d[c].z), vb.y, a1);
        a0 = fmaf(bf16_lo(d[c].w), vb.z, a0); a1 = fmaf(bf16_hi(d[c].w), vb.w, a1);
        acc += a0 + a1;
        // The sub-token ends with this chunk, or the row does (ragged last sub-token: the columns beyond
        // D were zero-filled by TMA and no further k-block follows).
        if (jv + 8 == Dsub || (kb == kblocks - 1 && c == 7)) {
            const int m = (kb * BK + c * 8) / Dsub;
            if (row < Mdim && m < fz.M) {
                if (ZK == 2) static_cast<__nv_bfloat16*>(fz.Z)[static_cast<int64_t>(row) * fz.ldz + m] = __float2bfloat16_rn(acc);
                else if (ZK == 3) static_cast<e4m3_t*>(fz.Z)[static_cast<int64_t>(row) * fz.ldz + m] = float_to_e4m3(acc);
                else static_cast<float*>(fz.Z)[static_cast<int64_t>(row) * fz.ldz + m] = acc;
            }
        }
    }
}

}  // namespace velora
