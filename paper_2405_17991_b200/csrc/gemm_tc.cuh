// Tensor-core (tcgen05 / TMA / TMEM) kernels of the VeLoRA path.
#pragma once

#include <cuda.h>

#include "common.cuh"

namespace velora {

// Operand layouts of the three dense products of Algorithm 1 (C is row-major [Mdim, Ndim]).
enum GemmKind {
    GEMM_NT_K_K = 0,    // Y  = X  W^T : A[Mdim, K] rows contiguous in K, B[Ndim, K] rows contiguous in K
    GEMM_NN_K_MN = 1,   // dX = dY W   : A[Mdim, K] contiguous in K,      B[K, Ndim] contiguous in Ndim
    GEMM_TN_MN_MN = 2   // dW = dY^T Xh: A[K, Mdim] contiguous in Mdim,   B[K, Ndim] contiguous in Ndim
};

// `status` (may be NULL) is a device word that a kernel sets to VELORA_ERR_TIMEOUT if one of its bounded
// waits expires; nothing ever clears it but velora_workspace_init.
// Returns VELORA_ERR_UNSUPPORTED (nothing launched) when the operands do not meet the tensor-core
// path's requirements (bf16 data, 16-byte aligned rows); the caller then uses the CUDA-core GEMM.
int launch_gemm_tc(int kind, const void* A, int64_t lda, const void* B, int64_t ldb,
                   void* C, int c_dtype, int64_t ldc, int beta,
                   int64_t Mdim, int64_t Ndim, int64_t Kdim, int in_dtype, int* status, cudaStream_t stream);

// The same product with CTA pairs (tcgen05 cta_group::2, 256 x 256 tile per pair).  (gemm_tc2.cu)
int launch_gemm_tc_pair(int kind, const void* A, int64_t lda, const void* B, int64_t ldb,
                        void* C, int c_dtype, int64_t ldc, int beta,
                        int64_t Mdim, int64_t Ndim, int64_t Kdim, int in_dtype, int* status, cudaStream_t stream);

int launch_linear_forward_tc_pair(const void* X, int64_t ldx, const void* W, int64_t ldw, const float* v,
                                  void* Y, int64_t ldy, void* Z, int z_dtype, int64_t ldz,
                                  int64_t N, int64_t D, int64_t O, int Dsub, int* status, cudaStream_t stream);
// Adapter-shaped layers (O <= 64): Y and Z in one pass over X.  (skinny.cu)
int launch_linear_forward_skinny(const void* X, int64_t ldx, const void* W, int64_t ldw, const float* v,
                                 void* Y, int64_t ldy, void* Z, int z_dtype, int64_t ldz,
                                 int64_t N, int64_t D, int64_t O, int Dsub, int* status, cudaStream_t stream);
// True when a product with this output shape fills the device with 256 x 256 pair tiles.
bool gemm_pair_preferred(int64_t Mdim, int64_t Ndim);

// Tensor map of a row-major bf16 matrix: `inner` contiguous elements per row, `outer` rows, row pitch
// ld_elems; 128-byte swizzle (or none), zero fill outside the matrix.  (gemm_tc.cu)
int make_tmap_bf16_2d(CUtensorMap* map, const void* base, int64_t inner, int64_t outer, int64_t ld_elems,
                      int box_inner, int box_outer, bool swizzle128 = true);
bool tc_operand_ok(const void* p, int64_t ld_elems);
// The same matrix seen as [64 elements][outer rows][inner / 64 column chunks] (inner a multiple of 64): a box of
// box_rows rows x box_chunks chunks lands in shared memory as box_chunks tiles of box_rows x 128 bytes, each
// swizzled like a two-dimensional 64-column box, from box_chunks * 128 contiguous bytes of every row.
// VELORA_ERR_UNSUPPORTED if the driver does not take the description.
int make_tmap_bf16_chunks3d(CUtensorMap* map, const void* base, int64_t inner, int64_t outer, int64_t ld_elems,
                            int box_rows, int box_chunks);

// Y = X W^T with compress(X, v) computed from the same staged X tiles.
int launch_linear_forward_tc(const void* X, int64_t ldx, const void* W, int64_t ldw, const float* v,
                             void* Y, int64_t ldy, void* Z, int z_dtype, int64_t ldz,
                             int dtype, int64_t N, int64_t D, int64_t O, int Dsub, int* status, cudaStream_t stream);

// Row-streaming kernels (stream_rows.cu): bf16 X with 16-byte aligned rows, Dsub = 8 * 2^k up to 1024.
// Return VELORA_ERR_UNSUPPORTED (nothing launched) when the shape does not fit them.
int launch_compress_rows(const void* X, int64_t N, int64_t D, int64_t ldx, int Dsub, const float* v,
                         void* Z, int z_dtype, int64_t ldz, cudaStream_t stream);
int launch_init_v_partials_rows(const void* X, int64_t N, int64_t D, int64_t ldx, int Dsub,
                                float* partials, int max_partials, int* num_partials, cudaStream_t stream);

// One tiny CTA whose bounded waits run out (limit_ns for the first, the abort flag for the second); raises
// `status` (may be NULL) and the per-device error word like a real kernel would.  observed[4]: device ints.
int launch_wait_timeout_selftest(int* status, unsigned long long limit_ns, int* observed, cudaStream_t stream);

// Reads (synchronising `stream`) and clears the device word in which the streaming kernels record an
// expired wait: VELORA_OK or VELORA_ERR_TIMEOUT.
int read_and_clear_stream_error(cudaStream_t stream);

// Factored weight gradient: P = dY^T Z on tensor cores (split over tokens), dW = P (x) v.
size_t weight_grad_tc_workspace_bytes(int64_t N, int64_t D, int64_t O, int Dsub);
// With P_out != NULL only the factor is produced: P_out[O, M] = beta * P_out + dY^T Z (fp32), dW untouched.
int launch_weight_grad_tc(const void* dY, int dy_dtype, int64_t N, int64_t O, int64_t lddy,
                          const void* Z, int z_dtype, int64_t ldz, const float* v, int64_t D, int Dsub,
                          void* dW, int dw_dtype, int64_t lddw, int beta,
                          void* ws, size_t ws_bytes, int* status, cudaStream_t stream,
                          float* P_out = nullptr, int64_t ldp_out = 0);

}  // namespace velora
