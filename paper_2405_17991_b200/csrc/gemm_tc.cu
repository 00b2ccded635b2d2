#include "gemm_tc.cuh"

namespace velora {

int launch_gemm_tc(int, const void*, int64_t, const void*, int64_t, void*, int, int64_t, int,
                   int64_t, int64_t, int64_t, int, cudaStream_t)
{
    return VELORA_ERR_UNSUPPORTED;
}

int launch_linear_forward_tc(const void*, int64_t, const void*, int64_t, const float*, void*, int64_t, void*, int,
                             int64_t, int, int64_t, int64_t, int64_t, int, cudaStream_t)
{
    return VELORA_ERR_UNSUPPORTED;
}

size_t weight_grad_tc_workspace_bytes(int64_t, int64_t, int64_t, int) { return 0; }

int launch_weight_grad_tc(const void*, int, int64_t, int64_t, int64_t, const void*, int, int64_t, const float*,
                          int64_t, int, void*, int, int64_t, int, void*, size_t, cudaStream_t)
{
    return VELORA_ERR_UNSUPPORTED;
}

}  // namespace velora
