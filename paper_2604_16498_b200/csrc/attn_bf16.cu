// placeholder replaced below
#include "forge_common.cuh"
extern "C" int forge_attn_fused(const void* q, const void* k, const void* v, void* out,
                                int B, int Hq, int Hkv, int Sq, int Skv, int D,
                                int mask_kind, const int32_t* lens, float scale, void* stream) {
    return FORGE_ERR_UNSUPPORTED;
}
