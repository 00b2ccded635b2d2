// The per-device error word of the entry points that take no workspace, and the self-test of the bounded
// waits that all tensor-core pipelines of this library share (tc_common.cuh).
#include "gemm_tc.cuh"
#include "tc_common.cuh"

namespace velora {

using namespace tc;

namespace {
__device__ int g_stream_error = 0;
}  // namespace

// Self-test of the give-up path that every pipeline in this library shares.  One CTA, no copies in flight,
// no tensor memory held: warp 0's elected lane waits (mbar_wait, the production routine) on a barrier on
// which nobody ever arrives, with the caller's short limit; warp 1 waits as a whole warp (mbar_wait_warp,
// with back-off) on a second such barrier with the ordinary one-second limit and must be released early by
// the abort flag that warp 0 raises.  Both then record the failure the way the real kernels do: the
// workspace's status word and the per-device error word.
__global__ void __launch_bounds__(64) wait_timeout_selftest_kernel(int* status, unsigned long long limit_ns, int* observed)
{
    __shared__ __align__(8) unsigned long long bars[2];
    __shared__ int abort_word;
    volatile int* abort_flag = &abort_word;
    const uint32_t bar0 = smem_u32(&bars[0]), bar1 = smem_u32(&bars[1]);
    if (threadIdx.x == 0) {
        mbar_init(bar0, 1);
        mbar_init(bar1, 1);
        *abort_flag = 0;
        fence_mbar_init();
    }
    __syncthreads();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    bool failed = false;
    if (warp == 0) {
        if (lane == 0) {
            const unsigned long long t0 = globaltimer_ns();
            if (!mbar_wait(bar0, 0u, abort_flag, 0, limit_ns)) {
                failed = true;
                *abort_flag = 1;
            }
            observed[0] = failed ? 1 : 0;
            observed[1] = static_cast<int>((globaltimer_ns() - t0) / 1000ull);      // microseconds waited
        }
    } else {
        const unsigned long long t0 = globaltimer_ns();
        if (!mbar_wait_warp(bar1, 0u, abort_flag, 256)) failed = true;
        if (lane == 0) {
            observed[2] = failed ? 1 : 0;
            observed[3] = static_cast<int>((globaltimer_ns() - t0) / 1000ull);
        }
    }
    if (failed && (threadIdx.x & 31) == 0) {
        if (status) atomicExch(status, VELORA_ERR_TIMEOUT);
        atomicExch(&g_stream_error, VELORA_ERR_TIMEOUT);
    }
}

int launch_wait_timeout_selftest(int* status, unsigned long long limit_ns, int* observed, cudaStream_t stream)
{
    wait_timeout_selftest_kernel<<<1, 64, 0, stream>>>(status, limit_ns, observed);
    return after_launch();
}

int read_and_clear_stream_error(cudaStream_t stream)
{
    int word = 0;
    if (cudaMemcpyFromSymbolAsync(&word, g_stream_error, sizeof(int), 0, cudaMemcpyDeviceToHost, stream) != cudaSuccess)
        return VELORA_ERR_CUDA;
    if (cudaStreamSynchronize(stream) != cudaSuccess) return VELORA_ERR_CUDA;
    if (word != 0) {
        const int zero = 0;
        if (cudaMemcpyToSymbolAsync(g_stream_error, &zero, sizeof(int), 0, cudaMemcpyHostToDevice, stream) != cudaSuccess)
            return VELORA_ERR_CUDA;
        cudaStreamSynchronize(stream);
        return VELORA_ERR_TIMEOUT;
    }
    return VELORA_OK;
}

}  // namespace velora
