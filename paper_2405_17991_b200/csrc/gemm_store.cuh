// Epilogue stores of the tensor-core GEMMs: 32 consecutive fp32 accumulator values of one output row,
// converted to the output type, optionally added to what is already there (beta = 1).
#pragma once

#include "common.cuh"

namespace velora {

// 32 bytes in one store instruction (sm_100 has 256-bit global stores).  A thread of the epilogue owns a
// contiguous piece of ONE output row, so 16-byte stores touch every 32-byte sector twice, from two
// instructions, and L2 counts two sector writes: on a product that is all epilogue (tiny K) ncu showed
// 4.19 M sector writes for 2.10 M sectors of output and the L2 at 65 % of its throughput.
__device__ __forceinline__ void st_global_32B(void* p, const uint4& a, const uint4& b)
{
    asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                 ::"l"(p), "r"(a.x), "r"(a.y), "r"(a.z), "r"(a.w), "r"(b.x), "r"(b.y), "r"(b.z), "r"(b.w) : "memory");
}

template <typename CT> struct Store32;
template <> struct Store32<__nv_bfloat16> {
    // 32 consecutive outputs of one row.
    static __device__ __forceinline__ void run(__nv_bfloat16* p, const uint32_t (&r)[32], int valid, int beta)
    {
        if (valid >= 32) {
            uint4* q = reinterpret_cast<uint4*>(p);
            uint4 o[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                float f[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) f[e] = __uint_as_float(r[8 * i + e]);
                if (beta) {
                    const uint4 old = q[i];
                    f[0] += bf16_lo(old.x); f[1] += bf16_hi(old.x);
                    f[2] += bf16_lo(old.y); f[3] += bf16_hi(old.y);
                    f[4] += bf16_lo(old.z); f[5] += bf16_hi(old.z);
                    f[6] += bf16_lo(old.w); f[7] += bf16_hi(old.w);
                }
                o[i].x = pack_bf16x2(f[0], f[1]);
                o[i].y = pack_bf16x2(f[2], f[3]);
                o[i].z = pack_bf16x2(f[4], f[5]);
                o[i].w = pack_bf16x2(f[6], f[7]);
            }
            if ((reinterpret_cast<uintptr_t>(p) & 31u) == 0) {
                st_global_32B(q, o[0], o[1]);
                st_global_32B(q + 2, o[2], o[3]);
            } else {
#pragma unroll
                for (int i = 0; i < 4; ++i) q[i] = o[i];
            }
        } else {
#pragma unroll
            for (int e = 0; e < 32; ++e)
                if (e < valid) {
                    float f = __uint_as_float(r[e]);
                    if (beta) f += __bfloat162float(p[e]);
                    p[e] = __float2bfloat16_rn(f);
                }
        }
    }
};
template <> struct Store32<float> {
    static __device__ __forceinline__ void run(float* p, const uint32_t (&r)[32], int valid, int beta)
    {
        if (valid >= 32) {
            float4* q = reinterpret_cast<float4*>(p);
            float4 o[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                o[i] = make_float4(__uint_as_float(r[4 * i]), __uint_as_float(r[4 * i + 1]),
                                   __uint_as_float(r[4 * i + 2]), __uint_as_float(r[4 * i + 3]));
                if (beta) {
                    const float4 old = q[i];
                    o[i].x += old.x; o[i].y += old.y; o[i].z += old.z; o[i].w += old.w;
                }
            }
            if ((reinterpret_cast<uintptr_t>(p) & 31u) == 0) {
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    st_global_32B(q + 2 * i, *reinterpret_cast<const uint4*>(&o[2 * i]), *reinterpret_cast<const uint4*>(&o[2 * i + 1]));
            } else {
#pragma unroll
                for (int i = 0; i < 8; ++i) q[i] = o[i];
            }
        } else {
#pragma unroll
            for (int e = 0; e < 32; ++e)
                if (e < valid) {
                    float f = __uint_as_float(r[e]);
                    if (beta) f += p[e];
                    p[e] = f;
                }
        }
    }
};

}  // namespace velora
