// Two small entry points that exist so that parts of the library which no operator call can
// single out are still observable from outside:
//   - forge_activation_f32 applies the GEMM epilogue's activation function element-wise in fp32
//     (bf16 outputs of the fused linear cannot tell tanh-GELU from erf-GELU: the two differ by at
//     most 4.7e-4);
//   - forge_debug_wait_timeout runs the bounded wait that every kernel uses on a barrier that
//     nothing completes, so that the give-up path (status word, FORGE_ERR_TIMEOUT from
//     forge_check_status) can be exercised without starving a real kernel.
#include "activations.cuh"
#include "forge_common.cuh"
#include "sm100_ptx.cuh"

namespace forge {
namespace {

template <int ACT, bool EXACT>
__global__ void activation_kernel(const float* __restrict__ x, float* __restrict__ y, size_t n) {
    pdl_launch_dependents();
    pdl_wait();
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) y[i] = activate<ACT, EXACT>(x[i]);
}

template <bool EXACT>
int launch_activation(const float* x, float* y, size_t n, int act, cudaStream_t s) {
    const int block = 256;
    const size_t want = (n + block - 1) / block;
    const int grid = (int)(want < 4096 ? want : 4096);
    switch (act) {
        case FORGE_ACT_GELU_TANH: FORGE_CUDA_TRY(launch_pdl(activation_kernel<FORGE_ACT_GELU_TANH, EXACT>, dim3(grid), dim3(block), 0, s, x, y, n)); break;
        case FORGE_ACT_GELU_ERF: FORGE_CUDA_TRY(launch_pdl(activation_kernel<FORGE_ACT_GELU_ERF, EXACT>, dim3(grid), dim3(block), 0, s, x, y, n)); break;
        case FORGE_ACT_RELU: FORGE_CUDA_TRY(launch_pdl(activation_kernel<FORGE_ACT_RELU, EXACT>, dim3(grid), dim3(block), 0, s, x, y, n)); break;
        case FORGE_ACT_SILU: FORGE_CUDA_TRY(launch_pdl(activation_kernel<FORGE_ACT_SILU, EXACT>, dim3(grid), dim3(block), 0, s, x, y, n)); break;
        default: FORGE_CUDA_TRY(launch_pdl(activation_kernel<FORGE_ACT_NONE, EXACT>, dim3(grid), dim3(block), 0, s, x, y, n)); break;
    }
    return finish_launch(1);
}

// One warp waits, with the library's bounded wait, for a barrier phase that no one completes.
__global__ void wait_timeout_kernel(long long budget_clocks, int* status) {
    __shared__ uint64_t bar;
    pdl_launch_dependents();
    pdl_wait();
    if (threadIdx.x == 0) {
        ptx::mbar_init(&bar, 1);
        ptx::fence_mbar_init();
    }
    __syncwarp();
    // phase 0 of a freshly initialised barrier with one pending arrival never completes
    if (!ptx::warp_wait(&bar, 0, budget_clocks)) {
        if (threadIdx.x == 0) atomicExch(status, 1);
    }
}

}  // namespace
}  // namespace forge

extern "C" int forge_activation_f32(const float* x, float* y, size_t n, int act, int exact, void* stream) {
    using namespace forge;
    if (!x || !y || n == 0) return FORGE_ERR_INVALID_ARG;
    if (act < FORGE_ACT_GELU_TANH || act > FORGE_ACT_NONE) return FORGE_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(x) & 3u) || (reinterpret_cast<uintptr_t>(y) & 3u)) return FORGE_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    return exact ? launch_activation<true>(x, y, n, act, s) : launch_activation<false>(x, y, n, act, s);
}

extern "C" int forge_debug_wait_timeout(long long budget_clocks, void* stream) {
    using namespace forge;
    // the probe is meant to give up quickly: at most about a tenth of a second of SM clocks
    if (budget_clocks < 0 || budget_clocks > 200000000LL) return FORGE_ERR_INVALID_ARG;
    int* status = device_status_word();
    if (!status) return FORGE_ERR_CUDA;
    FORGE_CUDA_TRY(launch_pdl(wait_timeout_kernel, dim3(1), dim3(32), 0, static_cast<cudaStream_t>(stream),
                              budget_clocks, status));
    return finish_launch(1);
}
