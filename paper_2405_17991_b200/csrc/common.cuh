// Shared declarations of the VeLoRA CUDA library (sm_100a).
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "velora.h"

namespace velora {

constexpr int kStreamThreads = 256;       // CTA size of the streaming kernels
constexpr int kStreamCtasPerSm = 8;       // resident CTAs per SM they are sized for
constexpr int kInitVMaxCtas = 1184;       // rows of the init_v partial-sum scratch (148 SMs x 8)
constexpr size_t kStatusBytes = 256;      // status word + padding at the head of a workspace

struct DeviceInfo {
    int sm_count;
    int smem_optin;
};
// Attributes of the current device (cached per device ordinal).
int device_info(DeviceInfo* out);

// Call right after every kernel launch: counts it and turns a launch error into a status.
int after_launch();

// "Done once per device" flags for host-side set-up that is harmless to repeat (a kernel attribute set to
// the same value, an address looked up again): atomics keep the first calls of two host threads from being
// a data race; nothing worse than a repeated set-up can happen.
struct DeviceOnce {
    std::atomic<bool> done[64];
    bool get(int dev) const { return done[dev].load(std::memory_order_acquire); }
    void set(int dev) { done[dev].store(true, std::memory_order_release); }
};

inline int64_t ceil_div64(int64_t a, int64_t b) { return (a + b - 1) / b; }
// Programmatic dependent launch.  A kernel launched with pdl_attribute() may become resident while the
// kernel before it in the stream is still running; it must call pdl_wait() before it touches anything
// that kernel writes (the wait returns once that kernel has completed and its writes are visible).
// pdl_trigger() in a kernel lets the NEXT kernel in the stream, if launched this way, start early.
// Used between the Z conversion and the weight-gradient kernel; tried on the dense products as well,
// where hiding the launch latency of a 200-500 us kernel made no measurable difference.
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
#endif
inline cudaLaunchAttribute pdl_attribute()
{
    cudaLaunchAttribute a{};
    a.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    a.val.programmaticStreamSerializationAllowed = 1;
    return a;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline size_t dtype_size(int dt) { return dt == VELORA_BF16 ? 2 : (dt == VELORA_FP8_E4M3 ? 1 : 4); }
inline bool valid_dtype(int dt) { return dt == VELORA_F32 || dt == VELORA_BF16; }                 // X, W, dY, Y, dX, dW
inline bool valid_z_dtype(int dt) { return valid_dtype(dt) || dt == VELORA_FP8_E4M3; }              // stored Z

// ---- streaming kernels (stream_kernels.cu) ----
// sum_only != 0: v receives the un-normalised sub-token sum s and nothing is synchronised.
int launch_init_v(const void* X, int x_dtype, int64_t N, int64_t D, int64_t ldx, int Dsub,
                  float* v, void* ws, size_t ws_bytes, cudaStream_t stream, int sum_only = 0);
// v = s / ||s|| (fp64 inside), degenerate flag read back (synchronises).
int launch_normalize_v(const float* s, int Dsub, float* v, void* ws, size_t ws_bytes, cudaStream_t stream);
// ---- adapter-shaped layers (skinny.cu) ----
size_t weight_grad_skinny_workspace_bytes(int64_t N, int64_t D, int64_t O, int Dsub);
int launch_weight_grad_skinny(const void* dY, int dy_dtype, int64_t N, int64_t O, int64_t lddy,
                              const void* Z, int z_dtype, int64_t ldz, const float* v, int64_t D, int Dsub,
                              void* dW, int dw_dtype, int64_t lddw, int beta,
                              void* ws, size_t ws_bytes, cudaStream_t stream, float* P_out, int64_t ldp_out);
size_t init_v_workspace_bytes(int Dsub);
// Scale of the 8-bit Z store from a batch: zscale = headroom * max|compress(X, v)| / 448 (1 if that maximum is
// zero or not finite), v_store = v / zscale, v_load = v * zscale.  Asynchronous.
size_t z8_calibrate_workspace_bytes(int64_t N, int64_t D, int Dsub);
int launch_z8_calibrate(const void* X, int x_dtype, int64_t N, int64_t D, int64_t ldx, int Dsub, const float* v,
                        float headroom, float* zscale, float* v_store, float* v_load,
                        void* ws, size_t ws_bytes, cudaStream_t stream);
size_t update_v_workspace_bytes(int Dsub);
int launch_update_v(const void* X, int x_dtype, int64_t N, int64_t D, int64_t ldx, int Dsub, float rho,
                    float* a, float* v, void* ws, size_t ws_bytes, cudaStream_t stream);
int launch_compress(const void* X, int x_dtype, int64_t N, int64_t D, int64_t ldx, int Dsub,
                    const float* v, void* Z, int z_dtype, int64_t ldz, cudaStream_t stream);
int launch_reconstruct(const void* Z, int z_dtype, int64_t ldz, int64_t N, int64_t D, int Dsub,
                       const float* v, void* Xhat, int x_dtype, int64_t ldxhat, cudaStream_t stream);

// ---- GEMMs ----
// C[m, n] = sum_k A(m, k) * B(n, k) with element strides; fp32 accumulation on CUDA cores.
// Serves the all-fp32 case and shapes the tensor-core path does not take.
int launch_gemm_simt(const void* A, int a_dtype, int64_t a_sm, int64_t a_sk,
                     const void* B, int b_dtype, int64_t b_sn, int64_t b_sk,
                     void* C, int c_dtype, int64_t ldc, int beta,
                     int64_t Mdim, int64_t Ndim, int64_t Kdim, cudaStream_t stream);

// dW[o, m*Dsub + j] = beta*dW + (sum over `splits` partial P[s][o][m], fp32) * v[j].
int launch_expand_p(const float* P, int splits, int64_t split_stride, int64_t ldp, const float* v,
                    int64_t O, int64_t D, int Dsub, void* dW, int dw_dtype, int64_t lddw, int beta,
                    cudaStream_t stream);

// Vector form of "row of scalars times v": out[r, m*Dsub + j] = beta*out + (sum_s S[s][r][m]) * v[j] for bf16 or
// fp32 S (one split: reconstruct; several: the factored weight gradient).  VELORA_ERR_UNSUPPORTED if the shape
// needs the element-wise kernels.  (expand_kernels.cu)
int launch_expand_rows_vec(const void* S, int s_dtype, int splits, int64_t split_stride, int64_t lds, const float* v,
                           int64_t R, int64_t D, int Dsub, void* out, int out_dtype, int64_t ldo, int beta,
                           cudaStream_t stream);

__device__ __forceinline__ float bf16_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t u) { return __uint_as_float(u & 0xffff0000u); }
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi)
{
    __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&h);
}

// One byte of the 8-bit floating-point format E4M3 (4 exponent bits, bias 7; 3 mantissa bits; no infinities,
// largest finite value 448): a storage type for Z only.  Conversions are the hardware's: round to nearest
// even, saturating at +-448.
struct e4m3_t {
    unsigned char bits;
};
#ifdef __CUDACC__
__device__ __forceinline__ e4m3_t float_to_e4m3(float x)
{
    unsigned short pair;                                  // the first source lands in the upper byte, the second in the lower
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(pair) : "f"(0.f), "f"(x));
    e4m3_t r;
    r.bits = static_cast<unsigned char>(pair & 0xffu);
    return r;
}
__device__ __forceinline__ float e4m3_to_float(e4m3_t q)
{
    unsigned int halves;                                  // the lower byte becomes the lower half-precision value
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(halves) : "h"(static_cast<unsigned short>(q.bits)));
    return __half2float(__ushort_as_half(static_cast<unsigned short>(halves & 0xffffu)));
}
#endif

template <typename T> struct Elem;
template <> struct Elem<float> {
    static __device__ __forceinline__ float load(const float* p) { return *p; }
    static __device__ __forceinline__ void store(float* p, float x) { *p = x; }
};
template <> struct Elem<__nv_bfloat16> {
    static __device__ __forceinline__ float load(const __nv_bfloat16* p) { return __bfloat162float(*p); }
    static __device__ __forceinline__ void store(__nv_bfloat16* p, float x) { *p = __float2bfloat16_rn(x); }
};
template <> struct Elem<e4m3_t> {
    static __device__ __forceinline__ float load(const e4m3_t* p) { return e4m3_to_float(*p); }
    static __device__ __forceinline__ void store(e4m3_t* p, float x) { *p = float_to_e4m3(x); }
};

}  // namespace velora
