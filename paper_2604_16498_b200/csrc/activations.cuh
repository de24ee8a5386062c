// Epilogue activations of the operator-fusion patterns (Section 4.3 "Pass 5": linear+gelu, linear+relu,
// linear+silu, mm+add; Eq. 11).  One definition serves the GEMM epilogues and the element-wise entry
// point forge_activation_f32, so what that entry point shows is what the epilogues compute.
//
// EXACT = false is what the kernels use: exponentials and reciprocals on the special-function unit
// (ex2.approx, rcp.approx: about 2 ulp each).  EXACT = true uses the accurate library routines and
// exists to check the formulas themselves against a reference at 1e-6.
#pragma once

#include <cuda_runtime.h>

#include "../../include/forge.h"

namespace forge {

// 1 / (1 + 2^(-x * log2(e))) = 1 / (1 + exp(-x))
template <bool EXACT>
__device__ __forceinline__ float sigmoid_f32(float x) {
    if constexpr (EXACT) {
        return 1.0f / (1.0f + expf(-x));
    } else {
        float e, r;
        asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(-1.4426950408889634f * x));
        asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(1.0f + e));
        return r;
    }
}

// gelu_tanh(z) = 0.5 z (1 + tanh(u)),  u = sqrt(2/pi) (z + 0.044715 z^3).
// 0.5 (1 + tanh(u)) = 1 / (1 + exp(-2u)), and in that form the negative tail (where 1 + tanh(u)
// cancels) keeps its relative accuracy: the hardware tanh approximation has an absolute error near 5e-4
// on a factor that is itself only a few 1e-3 there.
template <bool EXACT>
__device__ __forceinline__ float gelu_tanh_f32(float z) {
    const float u = 0.7978845608028654f * z * fmaf(0.044715f * z, z, 1.0f);
    if constexpr (EXACT) {
        const float hz = 0.5f * z;
        return fmaf(hz, tanhf(u), hz);
    } else {
        return z * sigmoid_f32<false>(2.0f * u);
    }
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
