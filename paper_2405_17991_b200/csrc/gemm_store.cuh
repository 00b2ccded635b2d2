// Epilogue stores of the tensor-core GEMMs: 32 consecutive fp32 accumulator values of one output row,
// converted to the output type, optionally added to what is already there (beta = 1).
#pragma once

#include "common.cuh"

namespace velora {

template <typename CT> struct Store32;
template <> struct Store32<__nv_bfloat16> {
    // 32 consecutive outputs of one row.
    static __device__ __forceinline__ void run(__nv_bfloat16* p, const uint32_t (&r)[32], int valid, int beta)
    {
        if (valid >= 32) {
            uint4* q = reinterpret_cast<uint4*>(p);
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
                uint4 o;
                o.x = pack_bf16x2(f[0], f[1]);
                o.y = pack_bf16x2(f[2], f[3]);
                o.z = pack_bf16x2(f[4], f[5]);
                o.w = pack_bf16x2(f[6], f[7]);
                q[i] = o;
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
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                float4 o = make_float4(__uint_as_float(r[4 * i]), __uint_as_float(r[4 * i + 1]),
                                       __uint_as_float(r[4 * i + 2]), __uint_as_float(r[4 * i + 3]));
                if (beta) {
                    const float4 old = q[i];
                    o.x += old.x; o.y += old.y; o.z += old.z; o.w += old.w;
                }
                q[i] = o;
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
