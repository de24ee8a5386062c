// Shared host-side plumbing of the library: status bookkeeping, launch counting,
// argument checks.  Nothing here computes anything of the operators.
#pragma once

#include <cuda_runtime.h>
#include <cstddef>
#include <cstdint>

#include "../../include/forge.h"

namespace forge {

// Per-thread record of the last failing CUDA call (returned by forge_last_cuda_error()).
void set_last_cuda_error(cudaError_t e);
// Counts a kernel launch (returned by forge_launch_count()).
void count_launch(int n = 1);
// Device-side status word, set by kernels whose bounded waits expire.
int* device_status_word();   // device address of the current device's word, resolved once per device

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Checks a launch: returns FORGE_OK or records the error and returns FORGE_ERR_CUDA.
inline int finish_launch(int nkernels) {
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { set_last_cuda_error(e); return FORGE_ERR_CUDA; }
    count_launch(nkernels);
    return FORGE_OK;
}

// Number of SMs of the current device (looked up once per device).
int sm_count();

// Launches `kernel` with programmatic stream serialisation: its CTAs may become resident while the
// previous kernel in the stream is still running (once that kernel has let its dependents go, or has
// finished), so launch latency and the kernel's own set-up overlap the predecessor's tail.  Every kernel
// of this library calls pdl_wait() before its first access to global memory, which blocks until the
// predecessor has completed and its writes are visible; a predecessor that never lets go behaves as
// with an ordinary launch.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem_bytes, cudaStream_t s,
                              Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem_bytes;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

#ifdef __CUDACC__
// Device side of launch_pdl(): let the next kernel in the stream become resident / wait for the previous one.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
#endif

// Opts a kernel in to `bytes` of dynamic shared memory once per device and call site (the attribute
// call costs microseconds, which matters for the latency-bound shapes).
#define FORGE_SET_SMEM_ONCE(kernel, bytes)                                                          \
    do {                                                                                            \
        static bool done__[64] = {};                                                                \
        int dev__ = 0;                                                                              \
        FORGE_CUDA_TRY(cudaGetDevice(&dev__));                                                      \
        if (dev__ < 0 || dev__ >= 64 || !done__[dev__]) {                                           \
            FORGE_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, \
                                                (int)(bytes)));                                     \
            if (dev__ >= 0 && dev__ < 64) done__[dev__] = true;                                     \
        }                                                                                           \
    } while (0)

#define FORGE_CUDA_TRY(expr)                                         \
    do {                                                             \
        cudaError_t e__ = (expr);                                    \
        if (e__ != cudaSuccess) {                                    \
            ::forge::set_last_cuda_error(e__);                       \
            return FORGE_ERR_CUDA;                                   \
        }                                                            \
    } while (0)

// Common validation of the attention entry points' scalar arguments and pointers.
inline int check_attn_args(const void* q, const void* k, const void* v, const void* out,
                           int B, int Hq, int Hkv, int Sq, int Skv, int D,
                           int mask_kind, const int32_t* lens, bool any_head_dim = false, int max_head_dim = 128) {
    if (!q || !k || !v || !out) return FORGE_ERR_INVALID_ARG;
    if (B <= 0 || Hq <= 0 || Hkv <= 0 || Sq <= 0 || Skv <= 0 || D <= 0) return FORGE_ERR_INVALID_ARG;
    if (Hq % Hkv != 0) return FORGE_ERR_INVALID_ARG;
    if (mask_kind < 0 || mask_kind > 3) return FORGE_ERR_INVALID_ARG;
    if ((mask_kind & FORGE_MASK_PADDING) && !lens) return FORGE_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out)) return FORGE_ERR_INVALID_ARG;
    if (lens && (reinterpret_cast<uintptr_t>(lens) & 3u)) return FORGE_ERR_INVALID_ARG;
    // any_head_dim: every multiple of 8 (16-byte rows) up to max_head_dim; otherwise the two sizes with their own kernels
    if (any_head_dim ? (D > max_head_dim || (D % 8) != 0) : (D != 64 && D != 128)) return FORGE_ERR_UNSUPPORTED;
    return FORGE_OK;
}

}  // namespace forge
