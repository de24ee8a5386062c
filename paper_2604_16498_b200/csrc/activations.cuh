// Epilogue activations of the operator-fusion patterns (Section 4.3 "Pass 5": linear+gelu, linear+relu,
// linear+silu, mm+add; Eq. 11).  One definition serves the GEMM epilogues and the element-wise entry
// point forge_activation_f32, so what that entry point shows is what the epilogues compute.
//
// EXACT = false is what the kernels use: one special-function-unit instruction per element
// (tanh.approx, relative error 2^-11 of tanh, i.e. up to 5e-4 absolute on the sigmoid factor), because
// the epilogue of a fused linear with a short K is bound by that unit: with exponential and reciprocal
// (two instructions) the 8192 x 3072 x 768 case spends more time in the epilogue than in the MMAs.  The
// absolute error this leaves on the activation, below 2.5e-4 |z|, is far inside the rounding of 16-bit outputs.
// EXACT = true uses the accurate library routines and exists to check the formulas themselves against a
// reference at 1e-6.
#pragma once

#include <cuda_runtime.h>

#include "../../include/forge.h"

namespace forge {

__device__ __forceinline__ float tanh_approx(float x) {
    float t;
    asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(x));
    return t;
}

// 1 / (1 + exp(-x)) = 0.5 + 0.5 tanh(x / 2)
template <bool EXACT>
__device__ __forceinline__ float sigmoid_f32(float x) {
    if constexpr (EXACT) return 1.0f / (1.0f + expf(-x));
    else return fmaf(0.5f, tanh_approx(0.5f * x), 0.5f);
}

// gelu_tanh(z) = 0.5 z (1 + tanh(u)),  u = sqrt(2/pi) (z + 0.044715 z^3)
template <bool EXACT>
__device__ __forceinline__ float gelu_tanh_f32(float z) {
    const float u = 0.7978845608028654f * z * fmaf(0.044715f * z, z, 1.0f);
    const float hz = 0.5f * z;
    return fmaf(hz, EXACT ? tanhf(u) : tanh_approx(u), hz);
}

template <int ACT, bool EXACT = false>
__device__ __forceinline__ float activate(float z) {
    if constexpr (ACT == FORGE_ACT_GELU_TANH) return gelu_tanh_f32<EXACT>(z);
    if constexpr (ACT == FORGE_ACT_GELU_ERF) return 0.5f * z * (1.0f + erff(z * 0.70710678118654752f));
    if constexpr (ACT == FORGE_ACT_RELU) return fmaxf(z, 0.f);
    if constexpr (ACT == FORGE_ACT_SILU) return z * sigmoid_f32<EXACT>(z);
    return z;
}

}  // namespace forge
