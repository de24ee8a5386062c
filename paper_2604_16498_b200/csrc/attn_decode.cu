// Split-KV decode attention and its combine step: Eq. 9 for a single query row per head
// over the first lens[b] rows of a KV cache.  The cached sequence is cut into num_splits
// ranges; each range yields a partial (running max m, running sum l, unnormalised output)
// and the combine step merges the partials:
//     M = max_s m_s,   L = sum_s 2^(m_s - M) l_s,   out = sum_s 2^(m_s - M) O_s / L
// (scores are kept in log2 units: they are pre-multiplied by scale * log2(e)).
//
// The kernel is bound by streaming K and V from HBM: every lane issues 128-bit loads straight
// into MMA fragments (no shared-memory staging), K and V loads of a block of rows are issued
// together, and the G = Hq / Hkv query heads that share a KV head are processed by the same CTA
// so that each cached row is read exactly once.  The dot products run on warp-level tensor-core
// MMAs (m16n8k16) only because fp32 FMAs with shuffle reductions were bound by instruction issue.
#include <cuda_bf16.h>

#include <mutex>

#include "forge_common.cuh"

namespace forge {
namespace {

constexpr int kWarps = 4;
constexpr int kThreads = kWarps * 32;
constexpr int kBlockKeys = 16;  // cached rows per warp iteration

__device__ __forceinline__ uint4 ld_stream(const void* p) {
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
                 : "l"(p));
    return r;
}

// D(16x8, fp32) += A(16x16, bf16, row) * B(16x8, bf16, col).  Lane = (g = lane / 4, c = lane % 4):
//   A: a0 = (row g, k 2c..2c+1)  a1 = (row g+8, k 2c..)  a2 = (row g, k 2c+8..)  a3 = (row g+8, k 2c+8..)
//   B: b0 = (k 2c..2c+1, col g)  b1 = (k 2c+8.., col g)
//   D: d0 = (row g, col 2c)  d1 = (row g, col 2c+1)  d2 = (row g+8, col 2c)  d3 = (row g+8, col 2c+1)
__device__ __forceinline__ void mma16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, "
                 "{%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// grid = (num_splits, Hkv, B).  Each warp walks its share of the split in blocks of 16 cached rows:
//   S[head, key]  = Q K^T   as m16n8k16 with A = Q (rows = the G heads, padded with zero rows) and
//                   B = K rows straight from global memory (the contraction runs over the head
//                   dimension in whatever order the 16-byte loads deliver it, the same for Q and K);
//   online softmax on the accumulator fragment (lane (g, c) owns head g, keys 2c, 2c+1 of each 8);
//   O^T[dim, head] += V^T P^T  with A = pairs of V rows interleaved with byte permutes and B = the
//                   probabilities exactly where the first MMA left them.
// The arithmetic is a few instructions per cached row, so the kernel is bound by the HBM stream.
template <int D, int G>
__global__ void __launch_bounds__(kThreads)
decode_split_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ kc,
                    const __nv_bfloat16* __restrict__ vc, const int32_t* __restrict__ lens,
                    float* __restrict__ ws_o, float* __restrict__ ws_ml,
                    int Hq, int Hkv, int Smax, int num_splits, float scale_log2) {
    constexpr int NKB = D / 32;  // 32-dim blocks of the head dimension (two k16 MMAs each)
    constexpr int NHB = D / 64;  // 64-dim blocks of the output (four 16-dim MMAs each)

    const int split = blockIdx.x, kvh = blockIdx.y, b = blockIdx.z;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g = lane >> 2, c = lane & 3;

    const int len = min(max(lens[b], 0), Smax);
    const int per = (len + num_splits - 1) / num_splits;
    const int s0 = split * per;
    const int s1 = min(s0 + per, len);

    __shared__ float sm_m[kWarps][G];
    __shared__ float sm_l[kWarps][G];
    __shared__ __align__(16) float sm_acc[kWarps][G][D];

    // Q fragment: head g (zero rows for g >= G), 8 dims at c*8 of every 32-dim block
    uint32_t qr[NKB][4];
#pragma unroll
    for (int kb = 0; kb < NKB; ++kb) {
        uint4 raw = make_uint4(0, 0, 0, 0);
        if (g < G) raw = *reinterpret_cast<const uint4*>(q + ((size_t)b * Hq + kvh * G + g) * D + kb * 32 + c * 8);
        qr[kb][0] = raw.x; qr[kb][1] = raw.y; qr[kb][2] = raw.z; qr[kb][3] = raw.w;
    }

    float m_run = -INFINITY, l_run = 0.f;  // of head g (lanes with g >= G carry dummies)
    float acc[NHB][4][4];                  // O^T fragments: [64-dim block][16-dim MMA][d0..d3]
#pragma unroll
    for (int hb = 0; hb < NHB; ++hb)
#pragma unroll
        for (int t = 0; t < 4; ++t)
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[hb][t][i] = 0.f;

    const __nv_bfloat16* kbase = kc + ((size_t)b * Hkv + kvh) * (size_t)Smax * D;
    const __nv_bfloat16* vbase = vc + ((size_t)b * Hkv + kvh) * (size_t)Smax * D;

    for (int j0 = s0 + warp * kBlockKeys; j0 < s1; j0 += kWarps * kBlockKeys) {
        // K: rows j0 + u*8 + g, 16 bytes at dims kb*32 + c*8.  V: rows j0 + {2c, 2c+1, 2c+8, 2c+9},
        // 16 bytes at dims hb*64 + g*8.  Rows at or beyond s1 are not read (zeros).
        uint4 kr[2][NKB], vr[4][NHB];
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            const int j = j0 + u * 8 + g;
#pragma unroll
            for (int kb = 0; kb < NKB; ++kb)
                kr[u][kb] = (j < s1) ? ld_stream(kbase + (size_t)j * D + kb * 32 + c * 8) : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            const int j = j0 + 2 * c + (r & 1) + (r >> 1) * 8;
#pragma unroll
            for (int hb = 0; hb < NHB; ++hb)
                vr[r][hb] = (j < s1) ? ld_stream(vbase + (size_t)j * D + hb * 64 + g * 8) : make_uint4(0, 0, 0, 0);
        }

        // scores: s[u][0..1] = head g, keys j0 + u*8 + 2c + {0, 1}  (s[u][2..3] belong to zero rows)
        float s[2][4];
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            s[u][0] = s[u][1] = s[u][2] = s[u][3] = 0.f;
#pragma unroll
            for (int kb = 0; kb < NKB; ++kb) {
                mma16816(s[u], qr[kb][0], 0u, qr[kb][1], 0u, kr[u][kb].x, kr[u][kb].y);
                mma16816(s[u], qr[kb][2], 0u, qr[kb][3], 0u, kr[u][kb].z, kr[u][kb].w);
            }
        }
        float mt = -INFINITY;
#pragma unroll
        for (int u = 0; u < 2; ++u)
#pragma unroll
            for (int i = 0; i < 2; ++i) {
                const bool ok = (j0 + u * 8 + 2 * c + i) < s1;
                s[u][i] = ok ? s[u][i] * scale_log2 : -INFINITY;
                mt = fmaxf(mt, s[u][i]);
            }
        mt = fmaxf(mt, __shfl_xor_sync(0xffffffffu, mt, 1));
        mt = fmaxf(mt, __shfl_xor_sync(0xffffffffu, mt, 2));
        const float m_new = fmaxf(m_run, mt);
        const float m_ref = (m_new == -INFINITY) ? 0.f : m_new;
        float alpha = exp2f(m_run - m_ref);  // 0 on the first block (m_run = -inf)
        m_run = m_new;
        float p[2][2];
#pragma unroll
        for (int u = 0; u < 2; ++u)
#pragma unroll
            for (int i = 0; i < 2; ++i) p[u][i] = exp2f(s[u][i] - m_ref);  // masked key: exactly 0
        if (g >= G) { alpha = 1.f; p[0][0] = p[0][1] = p[1][0] = p[1][1] = 0.f; }
        l_run = l_run * alpha + (p[0][0] + p[0][1]) + (p[1][0] + p[1][1]);

        // rescale the accumulators: this lane holds output columns (heads) 2c and 2c+1
        const float a_even = __shfl_sync(0xffffffffu, alpha, (2 * c) * 4);
        const float a_odd = __shfl_sync(0xffffffffu, alpha, (2 * c + 1) * 4);
        if (__any_sync(0xffffffffu, alpha != 1.f)) {
#pragma unroll
            for (int hb = 0; hb < NHB; ++hb)
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    acc[hb][t][0] *= a_even; acc[hb][t][1] *= a_odd;
                    acc[hb][t][2] *= a_even; acc[hb][t][3] *= a_odd;
                }
        }

        // P^T as the B operand: k-slots (2c, 2c+1) = keys 2c, 2c+1; k-slots (2c+8, 2c+9) = keys 2c+8, 2c+9
        const uint32_t pb0 = pack_bf16x2(p[0][0], p[0][1]);
        const uint32_t pb1 = pack_bf16x2(p[1][0], p[1][1]);
#pragma unroll
        for (int hb = 0; hb < NHB; ++hb) {
            // interleave two V rows: word w of a row holds dims 2w, 2w+1 -> (row_a[d], row_b[d]) pairs
            const uint32_t va[4] = {vr[0][hb].x, vr[0][hb].y, vr[0][hb].z, vr[0][hb].w};
            const uint32_t vb[4] = {vr[1][hb].x, vr[1][hb].y, vr[1][hb].z, vr[1][hb].w};
            const uint32_t vc_[4] = {vr[2][hb].x, vr[2][hb].y, vr[2][hb].z, vr[2][hb].w};
            const uint32_t vd[4] = {vr[3][hb].x, vr[3][hb].y, vr[3][hb].z, vr[3][hb].w};
            uint32_t ab[8], cd[8];
#pragma unroll
            for (int w = 0; w < 4; ++w) {
                ab[2 * w] = __byte_perm(va[w], vb[w], 0x5410);
                ab[2 * w + 1] = __byte_perm(va[w], vb[w], 0x7632);
                cd[2 * w] = __byte_perm(vc_[w], vd[w], 0x5410);
                cd[2 * w + 1] = __byte_perm(vc_[w], vd[w], 0x7632);
            }
            // MMA t: row g = dim hb*64 + g*8 + t, row g+8 = dim hb*64 + g*8 + 4 + t
#pragma unroll
            for (int t = 0; t < 4; ++t) mma16816(acc[hb][t], ab[t], ab[4 + t], cd[t], cd[4 + t], pb0, pb1);
        }
    }

    // the 4 lanes of a head hold partial sums over their own keys
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
    if (g < G && c == 0) { sm_m[warp][g] = m_run; sm_l[warp][g] = l_run; }
#pragma unroll
    for (int hb = 0; hb < NHB; ++hb)
#pragma unroll
        for (int t = 0; t < 4; ++t) {
            const int d0 = hb * 64 + g * 8 + t;
            if (2 * c < G) { sm_acc[warp][2 * c][d0] = acc[hb][t][0]; sm_acc[warp][2 * c][d0 + 4] = acc[hb][t][2]; }
            if (2 * c + 1 < G) { sm_acc[warp][2 * c + 1][d0] = acc[hb][t][1]; sm_acc[warp][2 * c + 1][d0 + 4] = acc[hb][t][3]; }
        }
    __syncthreads();
    for (int idx = tid; idx < G * D; idx += kThreads) {
        const int hg = idx / D, d = idx % D;
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) M = fmaxf(M, sm_m[w][hg]);
        const float Mref = (M == -INFINITY) ? 0.f : M;
        float L = 0.f, O = 0.f;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) {
            const float wgt = exp2f(sm_m[w][hg] - Mref);
            L = fmaf(wgt, sm_l[w][hg], L);
            O = fmaf(wgt, sm_acc[w][hg][d], O);
        }
        const size_t slot = ((size_t)b * Hq + kvh * G + hg) * num_splits + split;
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
