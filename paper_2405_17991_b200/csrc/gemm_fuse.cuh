// The compress (Section 3.1, Eq. 1) that rides on the forward GEMM: arguments and the per-group
// arithmetic shared by the single-CTA and the CTA-pair kernels.
#pragma once

#include "common.cuh"

namespace velora {

struct FuseArgs {
    const float* v;
    void* Z;
    int64_t ldz;
    int Dsub, M;
    const uint4* X;           // the layer input once more, as 16-byte chunks (rows 16-byte aligned)
    int64_t ldx_chunks;
};

// The compress warps keep step with the GEMM: they take the row block of the CTA's ti-th tile only once the
// TMA producer has started on that tile (it publishes the number of tiles started in shared memory), so their
// loads of X meet the GEMM's in L2 instead of running a hundred microseconds ahead and sending X through HBM
// a second time.  A hint, not a barrier: nothing waits for the compress warps.  Bounded like every wait: gives
// up when another role has raised the abort flag or after a second.
__device__ __forceinline__ bool wait_for_tile(volatile int* tiles_started, int ti, volatile int* abort_flag)
{
    if (*tiles_started > ti) return true;
    unsigned long long t0;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t0));
    unsigned spins = 0;
    while (*tiles_started <= ti) {
        __nanosleep(200);
        if ((++spins & 15u) == 0u) {
            if (*abort_flag) return false;
            unsigned long long t;
            asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
            if (t - t0 > 1000000000ull) return false;
        }
    }
    return true;
}

template <int ZK> __device__ __forceinline__ void store_z(const FuseArgs& fz, int row, int m, float z)
{
    if (ZK == 2) static_cast<__nv_bfloat16*>(fz.Z)[static_cast<int64_t>(row) * fz.ldz + m] = __float2bfloat16_rn(z);
    else if (ZK == 3) static_cast<e4m3_t*>(fz.Z)[static_cast<int64_t>(row) * fz.ldz + m] = float_to_e4m3(z);
    else static_cast<float*>(fz.Z)[static_cast<int64_t>(row) * fz.ldz + m] = z;
}

// 16 bytes of X for the compress warps: read-only path, not kept in L1 (each line is used once here, and
// L1 shares its storage and bandwidth with the shared memory the tensor cores are reading).
__device__ __forceinline__ uint4 ld_x_chunk(const uint4* p)
{
    uint4 x;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(x.x), "=r"(x.y), "=r"(x.z), "=r"(x.w) : "l"(p));
    return x;
}

// The slice of v a lane of a compress warp works with: lane l always meets chunk (32 * part + l) % L of a
// sub-token of L = Dsub / 8 chunks, part = 0 .. CH - 1 (CH = L / 32 for L > 32, else 1).
template <int CH> struct VSlice {
    float v[CH][8];
    __device__ __forceinline__ void load(const float* vg, int Dsub, int lane)
    {
        const int L = Dsub >> 3;
#pragma unroll
        for (int i = 0; i < CH; ++i) {
            const int pos = (32 * i + lane) & (L - 1);
#pragma unroll
            for (int e = 0; e < 8; ++e) v[i][e] = __ldg(vg + 8 * pos + e);
        }
    }
};

// The compress of one "group" of a row block by ONE warp, read straight from global memory (the lines are
// in L2 around the time the GEMM's own loads of the same row block run, so X still crosses HBM once):
// rows [r0, r0 + 32) of X, columns [8 * cpr * g, 8 * cpr * (g + 1)), cpr = max(Dsub / 8, 8) 16-byte chunks
// per row, i.e. one whole sub-token per row (Dsub >= 64) or the 64 / Dsub sub-tokens of a 64-column block.
// A load instruction covers 32 consecutive chunks of the warp's 32 x cpr chunk rectangle in row-major
// order; eight instructions are issued before the first is used.  L = Dsub / 8 chunks form a sub-token:
// lps = min(L, 32) adjacent lanes hold (a part of) it, for L > 32 the CH = L / 32 consecutive instructions
// complete it.  fp32 products and sums, xor-shuffle reduction, one lane stores Z[row, m].  Columns at or
// beyond D count as zeros (ragged last sub-token), rows at or beyond N are skipped.  No shared memory and
// no barrier (v sits in registers): the warps that do this never touch the GEMM's pipeline, and in
// particular not the shared-memory bandwidth the tensor cores live on.
template <int ZK, int CH>
__device__ __forceinline__ void compress_group_direct(const FuseArgs& fz, const VSlice<CH>& vs, int r0, int N, int D, int g, int lane)
{
    const int L = fz.Dsub >> 3;                         // a power of two, 1 .. 128 (host)
    const int lps = L < 32 ? L : 32;
    const int cpr = L < 8 ? 8 : L;
    const int cshift = 31 - __clz(cpr), lshift = 31 - __clz(L);
    const int d8 = D >> 3, tail = D & 7;
    const int c_base = g * cpr;                         // first chunk of the group in a row
    const int subs_per_row = cpr >> lshift;             // sub-tokens of one row inside the group (1 if Dsub >= 64)
    for (int i0 = 0; i0 < cpr; i0 += 8) {               // cpr instructions cover the warp's 32 rows
        uint4 d[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int flat = 32 * (i0 + u) + lane;
            const int row = r0 + (flat >> cshift), c = c_base + (flat & (cpr - 1));
            uint4 x = make_uint4(0u, 0u, 0u, 0u);
            if (row < N && (c < d8 || (c == d8 && tail))) {
                x = ld_x_chunk(fz.X + static_cast<int64_t>(row) * fz.ldx_chunks + c);
                if (c == d8) {                          // the chunk straddles D: zero the columns beyond it
                    uint32_t w[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        if (2 * k >= tail) w[k] = 0u;
                        else if (2 * k + 1 >= tail) w[k] &= 0x0000ffffu;
                    }
                    x = make_uint4(w[0], w[1], w[2], w[3]);
                }
            }
            d[u] = x;
        }
        float part = 0.f;
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int pi = u & (CH - 1);                // which 32-chunk part of the sub-token (i0 is a multiple of 8)
            const float (&v)[8] = vs.v[pi];
            float a0 = bf16_lo(d[u].x) * v[0], a1 = bf16_hi(d[u].x) * v[1];
            a0 = fmaf(bf16_lo(d[u].y), v[2], a0); a1 = fmaf(bf16_hi(d[u].y), v[3], a1);
            a0 = fmaf(bf16_lo(d[u].z), v[4], a0); a1 = fmaf(bf16_hi(d[u].z), v[5], a1);
            a0 = fmaf(bf16_lo(d[u].w), v[6], a0); a1 = fmaf(bf16_hi(d[u].w), v[7], a1);
            part = (pi == 0) ? a0 + a1 : part + (a0 + a1);
            if (pi == CH - 1) {
                float k = part;
                for (int off = lps >> 1; off >= 1; off >>= 1) k += __shfl_xor_sync(0xffffffffu, k, off);
                const int flat = 32 * (i0 + u) + lane;
                const int row = r0 + (flat >> cshift);
                const int m = g * subs_per_row + ((flat & (cpr - 1)) >> lshift);
                if ((lane & (lps - 1)) == 0 && row < N && m < fz.M) store_z<ZK>(fz, row, m, k);
            }
        }
    }
}

}  // namespace velora
