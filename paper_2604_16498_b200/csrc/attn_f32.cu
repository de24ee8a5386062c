// Fused attention with fp32 tensors (Eq. 8 / Eq. 9): one kernel computes scores,
// mask, online softmax and the product with V; scores and probabilities stay on chip.
// Plain fp32 FMA arithmetic (no tensor cores) so that the result stays within 1e-4 of
// an fp64 evaluation.  The benchmark shape for this entry point (12 heads x 128 x 128 x 64)
// is latency-bound: small CTAs, many of them, two KV tiles at most per CTA.
//
// CTA = 128 threads = one (batch, head, 16-query-row tile).  Per KV tile of 64 keys:
//   scores : thread t -> row t/8, keys (t%8) + 8*jj   (K rows padded by 4 floats: conflict-free float4 reads)
//   softmax: running max / sum per row, reduced over the 8 threads of a row with shuffles
//   P.V    : thread t -> row t/8, output dims (t%8)*4 + 32*dd  (float4 columns of V: conflict-free)
#include "forge_common.cuh"

namespace forge {
namespace {

constexpr int kBM = 16;      // query rows per CTA
constexpr int kBN = 64;      // keys per tile
constexpr int kThreads = 128;
constexpr int kPad = 4;      // floats of padding per shared-memory row

template <int D>
__global__ void __launch_bounds__(kThreads)
attn_f32_kernel(const float* __restrict__ q, const float* __restrict__ k, const float* __restrict__ v,
                float* __restrict__ out, int Hq, int Hkv, int Sq, int Skv, int mask_kind,
                const int32_t* __restrict__ lens, float scale_log2) {
    constexpr int LD = D + kPad;
    constexpr int DV = D / 32;  // float4 groups of output per thread
    extern __shared__ __align__(16) float smem_f32[];
    float* sQ = smem_f32;
    float* sK = sQ + kBM * LD;
    float* sV = sK + kBN * LD;
    float* sP = sV + kBN * LD;

    pdl_launch_dependents();  // the next kernel may move in; nothing global is touched before the previous one is done
    pdl_wait();
    const int tid = threadIdx.x;
    const int q0 = blockIdx.x * kBM;
    const int h = blockIdx.y;
    const int b = blockIdx.z;
    const int kvh = h / (Hq / Hkv);

    int kvlen = Skv;
    if (mask_kind & FORGE_MASK_PADDING) kvlen = min(max(lens[b], 0), Skv);
    const int causal_off = Skv - Sq;
    // keys this CTA can see at all: the last row of the tile sees the most
    int kv_end = kvlen;
    if (mask_kind & FORGE_MASK_CAUSAL) kv_end = min(kv_end, min(q0 + kBM, Sq) + causal_off);
    kv_end = max(kv_end, 0);

    const float* qb = q + ((size_t)(b * Hq + h) * Sq + q0) * D;
    const float* kb = k + (size_t)(b * Hkv + kvh) * Skv * D;
    const float* vb = v + (size_t)(b * Hkv + kvh) * Skv * D;

    // Q tile -> shared memory, pre-multiplied by scale * log2(e) so that exp2 can be used.
    for (int idx = tid; idx < kBM * (D / 4); idx += kThreads) {
        const int r = idx / (D / 4), c = idx % (D / 4);
        float4 val = make_float4(0.f, 0.f, 0.f, 0.f);
        if (q0 + r < Sq) val = reinterpret_cast<const float4*>(qb + (size_t)r * D)[c];
        val.x *= scale_log2; val.y *= scale_log2; val.z *= scale_log2; val.w *= scale_log2;
        reinterpret_cast<float4*>(sQ + r * LD)[c] = val;
    }

    const int row = tid >> 3;   // 0..15
    const int sub = tid & 7;    // 0..7
    const int qi = q0 + row;    // global query index of this thread's row
    float m_run = -INFINITY, l_run = 0.f;
    float4 acc[DV];
#pragma unroll
    for (int i = 0; i < DV; ++i) acc[i] = make_float4(0.f, 0.f, 0.f, 0.f);

    for (int j0 = 0; j0 < kv_end; j0 += kBN) {
        __syncthreads();  // previous tile fully consumed (and sQ written, first time round)
        for (int idx = tid; idx < kBN * (D / 4); idx += kThreads) {
            const int r = idx / (D / 4), c = idx % (D / 4);
            float4 kk = make_float4(0.f, 0.f, 0.f, 0.f), vv = kk;
            if (j0 + r < kv_end) {
                kk = reinterpret_cast<const float4*>(kb + (size_t)(j0 + r) * D)[c];
                vv = reinterpret_cast<const float4*>(vb + (size_t)(j0 + r) * D)[c];
            }
            reinterpret_cast<float4*>(sK + r * LD)[c] = kk;
            reinterpret_cast<float4*>(sV + r * LD)[c] = vv;
        }
        __syncthreads();

        // scores for (row, keys sub + 8*jj)
        float s[kBN / 8];
#pragma unroll
        for (int jj = 0; jj < kBN / 8; ++jj) s[jj] = 0.f;
#pragma unroll 2
        for (int c = 0; c < D / 4; ++c) {
            const float4 qv = reinterpret_cast<const float4*>(sQ + row * LD)[c];
#pragma unroll
            for (int jj = 0; jj < kBN / 8; ++jj) {
                const float4 kv4 = reinterpret_cast<const float4*>(sK + (sub + 8 * jj) * LD)[c];
                s[jj] = fmaf(qv.x, kv4.x, s[jj]);
                s[jj] = fmaf(qv.y, kv4.y, s[jj]);
                s[jj] = fmaf(qv.z, kv4.z, s[jj]);
                s[jj] = fmaf(qv.w, kv4.w, s[jj]);
            }
        }
        // mask + tile max
        float m_tile = -INFINITY;
#pragma unroll
        for (int jj = 0; jj < kBN / 8; ++jj) {
            const int j = j0 + sub + 8 * jj;
            bool ok = j < kvlen;
            if (mask_kind & FORGE_MASK_CAUSAL) ok = ok && (j <= qi + causal_off);
            s[jj] = ok ? s[jj] : -INFINITY;
            m_tile = fmaxf(m_tile, s[jj]);
        }
#pragma unroll
        for (int o = 1; o < 8; o <<= 1) m_tile = fmaxf(m_tile, __shfl_xor_sync(0xffffffffu, m_tile, o));
        const float m_new = fmaxf(m_run, m_tile);
        // a row that has seen no key yet keeps m = -inf; use 0 as the reference to avoid inf - inf
        const float m_ref = (m_new == -INFINITY) ? 0.f : m_new;
        const float alpha = exp2f(m_run - m_ref);  // 0 when m_run = -inf
        float l_tile = 0.f;
#pragma unroll
        for (int jj = 0; jj < kBN / 8; ++jj) {
            const float p = exp2f(s[jj] - m_ref);  // masked: exp2(-inf) = 0 exactly
            l_tile += p;
            sP[row * (kBN + kPad) + sub + 8 * jj] = p;
        }
#pragma unroll
        for (int o = 1; o < 8; o <<= 1) l_tile += __shfl_xor_sync(0xffffffffu, l_tile, o);
        l_run = l_run * alpha + l_tile;
        m_run = m_new;
#pragma unroll
        for (int i = 0; i < DV; ++i) {
            acc[i].x *= alpha; acc[i].y *= alpha; acc[i].z *= alpha; acc[i].w *= alpha;
        }
        __syncwarp();  // the 8 threads of a row live in one warp: sP row is complete

        // out[row, dims] += P[row, :] . V[:, dims]
#pragma unroll 4
        for (int j = 0; j < kBN; ++j) {
            const float p = sP[row * (kBN + kPad) + j];
#pragma unroll
            for (int i = 0; i < DV; ++i) {
                const float4 vv = reinterpret_cast<const float4*>(sV + j * LD)[sub + 8 * i];
                acc[i].x = fmaf(p, vv.x, acc[i].x);
                acc[i].y = fmaf(p, vv.y, acc[i].y);
                acc[i].z = fmaf(p, vv.z, acc[i].z);
                acc[i].w = fmaf(p, vv.w, acc[i].w);
            }
        }
    }

    if (qi < Sq) {
        const float inv = l_run > 0.f ? 1.f / l_run : 0.f;  // no visible key -> zeros
        float* orow = out + ((size_t)(b * Hq + h) * Sq + qi) * D;
#pragma unroll
        for (int i = 0; i < DV; ++i) {
            float4 o = acc[i];
            o.x *= inv; o.y *= inv; o.z *= inv; o.w *= inv;
            reinterpret_cast<float4*>(orow)[sub + 8 * i] = o;
        }
    }
}

}  // namespace
}  // namespace forge

extern "C" int forge_attn_fused_f32(const void* q, const void* k, const void* v, void* out,
                                    int B, int Hq, int Hkv, int Sq, int Skv, int D,
                                    int mask_kind, const int32_t* lens, float scale, void* stream) {
    using namespace forge;
    int st = check_attn_args(q, k, v, out, B, Hq, Hkv, Sq, Skv, D, mask_kind, lens);
    if (st != FORGE_OK) return st;
    if (Hq > 65535 || B > 65535) return FORGE_ERR_UNSUPPORTED;
    const dim3 grid((Sq + kBM - 1) / kBM, Hq, B);
    const float scale_log2 = scale * 1.4426950408889634f;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const float* qf = static_cast<const float*>(q);
    const float* kf = static_cast<const float*>(k);
    const float* vf = static_cast<const float*>(v);
    float* of = static_cast<float*>(out);
    const size_t smem = sizeof(float) * ((size_t)(kBM + 2 * kBN) * (D + kPad) + kBM * (kBN + kPad));
    if (D == 64) {
        FORGE_CUDA_TRY(launch_pdl(attn_f32_kernel<64>, grid, dim3(kThreads), smem, s, qf, kf, vf, of, Hq, Hkv, Sq, Skv,
                                  mask_kind, lens, scale_log2));
    } else {
        static bool attr_set = false;  // opt in to > 48 KB of dynamic shared memory once
        if (!attr_set) {
            FORGE_CUDA_TRY(cudaFuncSetAttribute(attn_f32_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                (int)smem));
            attr_set = true;
        }
        FORGE_CUDA_TRY(launch_pdl(attn_f32_kernel<128>, grid, dim3(kThreads), smem, s, qf, kf, vf, of, Hq, Hkv, Sq, Skv,
                                  mask_kind, lens, scale_log2));
    }
    return finish_launch(1);
}
