// Split-KV decode attention and its combine step: Eq. 9 for a single query row per head
// over the first lens[b] rows of a KV cache.  The cached sequence is cut into num_splits
// ranges; each range yields a partial (running max m, running sum l, unnormalised output)
// and the combine step merges the partials:
//     M = max_s m_s,   L = sum_s 2^(m_s - M) l_s,   out = sum_s 2^(m_s - M) O_s / L
// (scores are kept in log2 units: they are pre-multiplied by scale * log2(e)).
//
// The kernel is bound by streaming K and V from HBM: every lane issues 128-bit loads that
// cover whole 128-byte lines, K and V loads of a group of keys are issued together, and the
// G = Hq / Hkv query heads that share a KV head are processed by the same CTA so that each
// cached row is read exactly once.
#include <cuda_bf16.h>

#include <mutex>

#include "forge_common.cuh"

namespace forge {
namespace {

constexpr int kWarps = 4;
constexpr int kThreads = kWarps * 32;
constexpr int kU = 4;  // 128-bit loads in flight per lane and per tensor

__device__ __forceinline__ uint4 ld_stream(const void* p) {
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
                 : "l"(p));
    return r;
}
// bf16 pair packed in 32 bits -> two floats (exact widening)
__device__ __forceinline__ float bf_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }
__device__ __forceinline__ void unpack8(const uint4& r, float (&f)[8]) {
    f[0] = bf_lo(r.x); f[1] = bf_hi(r.x); f[2] = bf_lo(r.y); f[3] = bf_hi(r.y);
    f[4] = bf_lo(r.z); f[5] = bf_hi(r.z); f[6] = bf_lo(r.w); f[7] = bf_hi(r.w);
}

// grid = (num_splits, Hkv, B)
template <int D, int G>
__global__ void __launch_bounds__(kThreads)
decode_split_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ kc,
                    const __nv_bfloat16* __restrict__ vc, const int32_t* __restrict__ lens,
                    float* __restrict__ ws_o, float* __restrict__ ws_ml,
                    int Hq, int Hkv, int Smax, int num_splits, float scale_log2) {
    constexpr int LPK = D / 8;     // lanes that share one cached row (16 bytes each)
    constexpr int KPL = 32 / LPK;  // rows covered by one warp-wide load
    constexpr int KPI = KPL * kU;  // rows per warp iteration

    const int split = blockIdx.x, kvh = blockIdx.y, b = blockIdx.z;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int sub = lane / LPK;    // which of the KPL rows of a load this lane reads
    const int chunk = lane % LPK;  // which 8 dims of the row

    const int len = min(max(lens[b], 0), Smax);
    const int per = (len + num_splits - 1) / num_splits;
    const int s0 = split * per;
    const int s1 = min(s0 + per, len);

    __shared__ float sm_m[kWarps][G];
    __shared__ float sm_l[kWarps][G];
    __shared__ __align__(16) float sm_acc[kWarps][G][D];

    // query rows of the G heads, pre-scaled; each lane keeps its 8 dims
    float qf[G][8];
#pragma unroll
    for (int g = 0; g < G; ++g) {
        const uint4 raw = *reinterpret_cast<const uint4*>(q + ((size_t)b * Hq + kvh * G + g) * D + chunk * 8);
        unpack8(raw, qf[g]);
#pragma unroll
        for (int i = 0; i < 8; ++i) qf[g][i] *= scale_log2;
    }

    float m_run[G], l_run[G], acc[G][8];
#pragma unroll
    for (int g = 0; g < G; ++g) {
        m_run[g] = -INFINITY;
        l_run[g] = 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[g][i] = 0.f;
    }

    const __nv_bfloat16* kbase = kc + ((size_t)b * Hkv + kvh) * (size_t)Smax * D + chunk * 8;
    const __nv_bfloat16* vbase = vc + ((size_t)b * Hkv + kvh) * (size_t)Smax * D + chunk * 8;

    for (int j0 = s0 + warp * KPI; j0 < s1; j0 += kWarps * KPI) {
        uint4 kr[kU], vr[kU];
#pragma unroll
        for (int u = 0; u < kU; ++u) {
            const int j = j0 + u * KPL + sub;
            if (j < s1) {
                kr[u] = ld_stream(kbase + (size_t)j * D);
                vr[u] = ld_stream(vbase + (size_t)j * D);
            } else {
                kr[u] = make_uint4(0, 0, 0, 0);
                vr[u] = make_uint4(0, 0, 0, 0);
            }
        }
        float s[kU][G];
#pragma unroll
        for (int u = 0; u < kU; ++u) {
            float kf[8];
            unpack8(kr[u], kf);
#pragma unroll
            for (int g = 0; g < G; ++g) {
                float d = 0.f;
#pragma unroll
                for (int i = 0; i < 8; ++i) d = fmaf(qf[g][i], kf[i], d);
                s[u][g] = d;
            }
        }
        // sum the partial dot products over the LPK lanes of a row (all of them get the total)
#pragma unroll
        for (int o = 1; o < LPK; o <<= 1)
#pragma unroll
            for (int u = 0; u < kU; ++u)
#pragma unroll
                for (int g = 0; g < G; ++g) s[u][g] += __shfl_xor_sync(0xffffffffu, s[u][g], o);

        float alpha[G], m_ref[G];
#pragma unroll
        for (int g = 0; g < G; ++g) {
            float mt = -INFINITY;
#pragma unroll
            for (int u = 0; u < kU; ++u) {
                const bool ok = (j0 + u * KPL + sub) < s1;
                s[u][g] = ok ? s[u][g] : -INFINITY;
                mt = fmaxf(mt, s[u][g]);
            }
#pragma unroll
            for (int o = LPK; o < 32; o <<= 1) mt = fmaxf(mt, __shfl_xor_sync(0xffffffffu, mt, o));
            const float m_new = fmaxf(m_run[g], mt);
            m_ref[g] = (m_new == -INFINITY) ? 0.f : m_new;
            alpha[g] = exp2f(m_run[g] - m_ref[g]);
            m_run[g] = m_new;
        }
#pragma unroll
        for (int g = 0; g < G; ++g) {
            l_run[g] *= alpha[g];
#pragma unroll
            for (int i = 0; i < 8; ++i) acc[g][i] *= alpha[g];
        }
#pragma unroll
        for (int u = 0; u < kU; ++u) {
            float vf[8];
            unpack8(vr[u], vf);
#pragma unroll
            for (int g = 0; g < G; ++g) {
                const float p = exp2f(s[u][g] - m_ref[g]);  // masked row: exactly 0
                l_run[g] += p;
#pragma unroll
                for (int i = 0; i < 8; ++i) acc[g][i] = fmaf(p, vf[i], acc[g][i]);
            }
        }
    }

    // merge the KPL row-groups of the warp (they share m_run), then the warps via shared memory
#pragma unroll
    for (int o = LPK; o < 32; o <<= 1) {
#pragma unroll
        for (int g = 0; g < G; ++g) {
            l_run[g] += __shfl_xor_sync(0xffffffffu, l_run[g], o);
#pragma unroll
            for (int i = 0; i < 8; ++i) acc[g][i] += __shfl_xor_sync(0xffffffffu, acc[g][i], o);
        }
    }
    if (sub == 0) {
#pragma unroll
        for (int g = 0; g < G; ++g) {
            if (chunk == 0) { sm_m[warp][g] = m_run[g]; sm_l[warp][g] = l_run[g]; }
#pragma unroll
            for (int i = 0; i < 8; ++i) sm_acc[warp][g][chunk * 8 + i] = acc[g][i];
        }
    }
    __syncthreads();
    for (int idx = tid; idx < G * D; idx += kThreads) {
        const int g = idx / D, d = idx % D;
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) M = fmaxf(M, sm_m[w][g]);
        const float Mref = (M == -INFINITY) ? 0.f : M;
        float L = 0.f, O = 0.f;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) {
            const float wgt = exp2f(sm_m[w][g] - Mref);
            L = fmaf(wgt, sm_l[w][g], L);
            O = fmaf(wgt, sm_acc[w][g][d], O);
        }
        const size_t slot = ((size_t)b * Hq + kvh * G + g) * num_splits + split;
        ws_o[slot * D + d] = O;
        if (d == 0) { ws_ml[slot * 2] = M; ws_ml[slot * 2 + 1] = L; }
    }
}

// grid = B * Hq, block = D threads: merges the num_splits partials of one (batch, head).
template <int D>
__global__ void __launch_bounds__(D)
decode_combine_kernel(const float* __restrict__ ws_o, const float* __restrict__ ws_ml,
                      __nv_bfloat16* __restrict__ out, int num_splits) {
    const size_t bh = blockIdx.x;
    const int d = threadIdx.x;
    const float* ml = ws_ml + bh * num_splits * 2;
    float M = -INFINITY;
    for (int s = 0; s < num_splits; ++s) M = fmaxf(M, ml[2 * s]);
    float L = 0.f, O = 0.f;
    if (M != -INFINITY) {
        for (int s = 0; s < num_splits; ++s) {
            const float ms = ml[2 * s];
            if (ms == -INFINITY) continue;  // empty split: its output slot was never written
            const float wgt = exp2f(ms - M);
            L = fmaf(wgt, ml[2 * s + 1], L);
            O = fmaf(wgt, ws_o[(bh * num_splits + s) * D + d], O);
        }
    }
    out[bh * D + d] = __float2bfloat16_rn(L > 0.f ? O / L : 0.f);
}

template <int D, int G>
void launch_split(const void* q, const void* kc, const void* vc, const int32_t* lens, float* ws_o, float* ws_ml,
                  int B, int Hq, int Hkv, int Smax, int num_splits, float scale_log2, cudaStream_t s) {
    decode_split_kernel<D, G><<<dim3(num_splits, Hkv, B), kThreads, 0, s>>>(
        static_cast<const __nv_bfloat16*>(q), static_cast<const __nv_bfloat16*>(kc),
        static_cast<const __nv_bfloat16*>(vc), lens, ws_o, ws_ml, Hq, Hkv, Smax, num_splits, scale_log2);
}

template <int D>
int dispatch_g(int G, const void* q, const void* kc, const void* vc, const int32_t* lens, float* ws_o,
               float* ws_ml, int B, int Hq, int Hkv, int Smax, int num_splits, float scale_log2, cudaStream_t s) {
    switch (G) {
        case 1: launch_split<D, 1>(q, kc, vc, lens, ws_o, ws_ml, B, Hq, Hkv, Smax, num_splits, scale_log2, s); break;
        case 2: launch_split<D, 2>(q, kc, vc, lens, ws_o, ws_ml, B, Hq, Hkv, Smax, num_splits, scale_log2, s); break;
        case 4: launch_split<D, 4>(q, kc, vc, lens, ws_o, ws_ml, B, Hq, Hkv, Smax, num_splits, scale_log2, s); break;
        case 8: launch_split<D, 8>(q, kc, vc, lens, ws_o, ws_ml, B, Hq, Hkv, Smax, num_splits, scale_log2, s); break;
        default: return FORGE_ERR_UNSUPPORTED;
    }
    return FORGE_OK;
}

}  // namespace
}  // namespace forge

extern "C" size_t forge_attn_decode_workspace_bytes(int B, int Hq, int D, int num_splits) {
    if (B <= 0 || Hq <= 0 || D <= 0 || num_splits <= 0) return 0;
    const size_t slots = (size_t)B * Hq * num_splits;
    return (slots * (size_t)(D + 2) * sizeof(float) + 15) & ~(size_t)15;
}

extern "C" int forge_attn_decode_splitkv(const void* q, const void* k_cache, const void* v_cache, void* out,
                                         int B, int Hq, int Hkv, int Smax, int D,
                                         const int32_t* lens, int num_splits, float scale,
                                         void* workspace, size_t workspace_bytes, void* stream) {
    using namespace forge;
    if (!lens) return FORGE_ERR_INVALID_ARG;
    int st = check_attn_args(q, k_cache, v_cache, out, B, Hq, Hkv, 1, Smax, D, FORGE_MASK_PADDING, lens);
    if (st != FORGE_OK) return st;
    if (num_splits < 1) return FORGE_ERR_INVALID_ARG;
    if (num_splits > 64 || Hkv > 65535 || B > 65535) return FORGE_ERR_UNSUPPORTED;
    if (!workspace || !aligned16(workspace)) return FORGE_ERR_INVALID_ARG;
    if (workspace_bytes < forge_attn_decode_workspace_bytes(B, Hq, D, num_splits)) return FORGE_ERR_WORKSPACE;

    const size_t slots = (size_t)B * Hq * num_splits;
    float* ws_o = static_cast<float*>(workspace);
    float* ws_ml = ws_o + slots * D;
    const float scale_log2 = scale * 1.4426950408889634f;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int G = Hq / Hkv;
    st = (D == 64) ? dispatch_g<64>(G, q, k_cache, v_cache, lens, ws_o, ws_ml, B, Hq, Hkv, Smax, num_splits, scale_log2, s)
                   : dispatch_g<128>(G, q, k_cache, v_cache, lens, ws_o, ws_ml, B, Hq, Hkv, Smax, num_splits, scale_log2, s);
    if (st != FORGE_OK) return st;
    st = finish_launch(1);
    if (st != FORGE_OK) return st;
    if (D == 64)
        decode_combine_kernel<64><<<B * Hq, 64, 0, s>>>(ws_o, ws_ml, static_cast<__nv_bfloat16*>(out), num_splits);
    else
        decode_combine_kernel<128><<<B * Hq, 128, 0, s>>>(ws_o, ws_ml, static_cast<__nv_bfloat16*>(out), num_splits);
    return finish_launch(1);
}

// ---------------------------------------------------------------------------------------------
// Decode without a caller workspace.
//
// Some callers cannot hand over scratch memory because they cannot allocate any: a serving loop
// whose device-memory plan is frozen after start-up, a plugin living inside a host runtime that
// owns the allocator, or code on a latency path where cudaMalloc's implicit device synchronisation
// is not acceptable.  For them the split partials live in a fixed array that is part of the
// library's device image.  Every GPU that loads the library carries this array until the process
// exits, whether or not the entry point is ever called.
namespace forge {
namespace {

static __device__ __align__(256) unsigned char g_decode_static_scratch[FORGE_DECODE_STATIC_SCRATCH_BYTES];

// In host code the array's name is only a handle for the runtime, not a device address; the address
// has to be asked for, once per device, with that device current.
void* static_scratch_for_current_device() {
    constexpr int kMaxDevices = 64;
    static void* cache[kMaxDevices] = {nullptr};
    static std::mutex mu;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        set_last_cuda_error(cudaErrorInvalidDevice);
        return nullptr;
    }
    std::lock_guard<std::mutex> lock(mu);
    if (!cache[dev]) {
        void* ptr = nullptr;
        const cudaError_t e = cudaGetSymbolAddress(&ptr, g_decode_static_scratch);
        if (e != cudaSuccess || !ptr) {
            set_last_cuda_error(e != cudaSuccess ? e : cudaErrorInvalidSymbol);
            return nullptr;
        }
        cache[dev] = ptr;
    }
    return cache[dev];
}

}  // namespace
}  // namespace forge

extern "C" int forge_attn_decode_splitkv_static(const void* q, const void* k_cache, const void* v_cache, void* out,
                                                int B, int Hq, int Hkv, int Smax, int D,
                                                const int32_t* lens, int num_splits, float scale, void* stream) {
    using namespace forge;
    if (B <= 0 || Hq <= 0 || D <= 0 || num_splits <= 0) return FORGE_ERR_INVALID_ARG;
    // the partials of this problem, B * Hq * num_splits * (D + 2) * 4 bytes, must fit the fixed array
    const size_t need = forge_attn_decode_workspace_bytes(B, Hq, D, num_splits);
    if (need > (size_t)FORGE_DECODE_STATIC_SCRATCH_BYTES) return FORGE_ERR_WORKSPACE;
    if (!q || !k_cache || !v_cache || !out || !lens) return FORGE_ERR_INVALID_ARG;
    void* scratch = static_scratch_for_current_device();
    if (!scratch) return FORGE_ERR_CUDA;
    return forge_attn_decode_splitkv(q, k_cache, v_cache, out, B, Hq, Hkv, Smax, D, lens, num_splits, scale,
                                     scratch, (size_t)FORGE_DECODE_STATIC_SCRATCH_BYTES, stream);
}
