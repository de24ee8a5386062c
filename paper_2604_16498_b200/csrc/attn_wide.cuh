// Fused attention for head sizes above 128 (attn_wide.cu): entry point for the dispatchers in attn_bf16.cu.
#pragma once

#include <cuda_runtime.h>
#include <cstdint>

namespace forge {

// softmax(scale q k^T + mask) v for 128 < head_dim <= 256 (a multiple of 8), bf16 (f16 = false) or fp16 tensors.
// strides[0..3]: element strides {batch, head, row} of q, k, v, out.  Other arguments as forge_attn_fused.
int attn_wide(bool f16, const void* q, const void* k, const void* v, void* out, int B, int Hq, int Hkv, int Sq, int Skv,
              int head_dim, int mask_kind, const int32_t* lens, float scale, const long long (*strides)[3], cudaStream_t s);

}  // namespace forge
