// The fused linear on CTA pairs (linear_pair.cu): entry points for the dispatcher in linear_gelu.cu.
#pragma once

#include <cuda_runtime.h>

namespace forge {

// True when the pair kernel (256 x 256 tiles on pairs of SMs) is expected to beat the one-CTA kernel
// (128 x 192 tiles) for an M x N output on a GPU with `sms` SMs.
bool linear_pair_pays(int M, int N, int sms);

// act(x W + b) + residual on CTA pairs; arguments as forge_linear_act (f16: fp16 instead of bf16 tensors).
int linear_pair(bool f16, const void* x, const void* w, const void* b, const void* residual, void* y, int M, int N,
                int K, int act, int w_layout, cudaStream_t s);

// silu(x Wg) * (x Wu) on CTA pairs (bf16); arguments as forge_linear_swiglu.  Pays whenever M > 128.
int linear_pair_swiglu(const void* x, const void* w_gate, const void* w_up, void* y, int M, int N, int K, int w_layout,
                       cudaStream_t s);

}  // namespace forge
