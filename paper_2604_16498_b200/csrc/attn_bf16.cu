// Fused attention, bf16 in / fp32 accumulate / bf16 out (Eq. 8 / Eq. 9): scores, mask, online
// softmax and the product with V in one kernel; S and P never reach global memory.
//
// One CTA = one (batch, query head, 128-query-row tile).  Warp roles:
//   warp 0    : TMA producer: Q tile once, then K and V tiles (128 keys) through 2-stage rings
//   warp 1    : tcgen05.mma issuer (one elected lane), owns the TMEM allocation
//   warps 2-5 : softmax / rescale / epilogue; thread = one query row (TMEM lane), so row
//               maxima and sums need no cross-thread reduction
// Tensor memory: S (128 x 128 fp32) double-buffered in columns [0,256), O (128 x D fp32) at 256.
// Per KV tile j:   S_j = Q K_j^T  ->  softmax warps read S_j, update the running max m and sum l,
// write P_j (bf16) to shared memory  ->  O += P_j V_j.  S_{j+1} is issued before P_j is waited
// for, so the tensor core computes the next scores while the softmax of the current tile runs.
// O is rescaled in TMEM only when a row's maximum grows by more than 2^8 (the stale maximum is
// kept otherwise; the final division by l uses the same reference, so the result is unchanged).
//
// Q and K are K-major operands, V [keys, D] is the MN-major B operand of P V, P is written in the
// K-major 128-byte-swizzled layout the MMA expects.
#include <cuda_bf16.h>

#include "forge_common.cuh"
#include "sm100_ptx.cuh"
#include "tmap.cuh"

namespace forge {
namespace {

using namespace ptx;

constexpr int kBM = 128;          // query rows per CTA
constexpr int kBN = 128;          // keys per tile
constexpr int kThreads = 192;
constexpr int kSoftmaxThreads = 128;
constexpr int kKVStages = 2;
constexpr int kTmemCols = 512;
constexpr int kColS = 0;          // S buffers at columns 0 and 128
constexpr int kColO = 256;
constexpr float kRescaleThreshold = 8.0f;  // log2 units

template <int D>
struct AttnSmem {
    static constexpr int kChunkBytes = 128 * 128;            // 128 rows x 64 bf16 (one swizzle span wide)
    static constexpr int kTileBytes = (D / 64) * kChunkBytes;  // Q, K or V tile
    static constexpr int kPBytes = 2 * kChunkBytes;          // 128 x 128 bf16
    static constexpr int kQOff = 0;
    static constexpr int kKOff = kQOff + kTileBytes;
    static constexpr int kVOff = kKOff + kKVStages * kTileBytes;
    static constexpr int kPOff = kVOff + kKVStages * kTileBytes;
    static constexpr int kBarOff = kPOff + kPBytes;
    static constexpr int kNumBars = 1 + 4 * kKVStages + 2 + 2;  // q_full, k/v full+empty, s_full[2], p_ready, pv_done
    static constexpr int kTotal = kBarOff + kNumBars * 8 + 16;
    static constexpr int kAlloc = kTotal + 1024;
};

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

struct AttnParams {
    __nv_bfloat16* out;
    const int32_t* lens;
    int Hq, Hkv, Sq, Skv;
    int mask_kind;
    float scale_log2;
    int* status;
};

template <int D>
__global__ void __launch_bounds__(kThreads, 1)
attn_bf16_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
                 const __grid_constant__ CUtensorMap tmap_v, const AttnParams p) {
    using L = AttnSmem<D>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* sQ = smem + L::kQOff;
    uint8_t* sK = smem + L::kKOff;
    uint8_t* sV = smem + L::kVOff;
    uint8_t* sP = smem + L::kPOff;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::kBarOff);
    uint64_t* q_full = bars;
    uint64_t* k_full = bars + 1;
    uint64_t* k_empty = k_full + kKVStages;
    uint64_t* v_full = k_empty + kKVStages;
    uint64_t* v_empty = v_full + kKVStages;
    uint64_t* s_full = v_empty + kKVStages;  // [2]
    uint64_t* p_ready = s_full + 2;
    uint64_t* pv_done = p_ready + 1;
    uint32_t* tmem_base_slot = reinterpret_cast<uint32_t*>(pv_done + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int num_q_tiles = (p.Sq + kBM - 1) / kBM;
    const int q_tile = num_q_tiles - 1 - blockIdx.x;  // longest (causal) tiles first
    const int h = blockIdx.y, b = blockIdx.z;
    const int kvh = h / (p.Hq / p.Hkv);
    const int q0 = q_tile * kBM;
    const int causal_off = p.Skv - p.Sq;
    const bool causal = (p.mask_kind & FORGE_MASK_CAUSAL) != 0;

    int kvlen = p.Skv;
    if (p.mask_kind & FORGE_MASK_PADDING) kvlen = min(max(p.lens[b], 0), p.Skv);
    int kv_end = kvlen;  // keys visible to at least one row of this tile
    if (causal) kv_end = min(kv_end, min(q0 + kBM, p.Sq) + causal_off);
    kv_end = max(kv_end, 0);
    const int n_tiles = (kv_end + kBN - 1) / kBN;

    if (threadIdx.x == 0) {
        mbar_init(q_full, 1);
        for (int i = 0; i < kKVStages; ++i) {
            mbar_init(&k_full[i], 1); mbar_init(&k_empty[i], 1);
            mbar_init(&v_full[i], 1); mbar_init(&v_empty[i], 1);
        }
        mbar_init(&s_full[0], 1); mbar_init(&s_full[1], 1);
        mbar_init(p_ready, kSoftmaxThreads);
        mbar_init(pv_done, 1);
        fence_mbar_init();
        prefetch_tmap(&tmap_q); prefetch_tmap(&tmap_k); prefetch_tmap(&tmap_v);
    }
    if (warp == 1) {
        tmem_alloc(tmem_base_slot, kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_base_slot;
    bool failed = false;

    if (warp == 0) {
        if (n_tiles > 0 && elect_one()) {
            mbar_expect_tx(q_full, L::kTileBytes);
#pragma unroll
            for (int c = 0; c < D / 64; ++c) tma_load_3d(sQ + c * L::kChunkBytes, &tmap_q, q_full, c * 64, q0, b * p.Hq + h);
            for (int j = 0; j < n_tiles; ++j) {
                const int st = j % kKVStages;
                const uint32_t ph = (j / kKVStages) & 1;
                if (!mbar_wait(&k_empty[st], ph ^ 1)) { failed = true; break; }
                mbar_expect_tx(&k_full[st], L::kTileBytes);
#pragma unroll
                for (int c = 0; c < D / 64; ++c)
                    tma_load_3d(sK + st * L::kTileBytes + c * L::kChunkBytes, &tmap_k, &k_full[st], c * 64, j * kBN,
                                b * p.Hkv + kvh);
                if (!mbar_wait(&v_empty[st], ph ^ 1)) { failed = true; break; }
                mbar_expect_tx(&v_full[st], L::kTileBytes);
#pragma unroll
                for (int c = 0; c < D / 64; ++c)
                    tma_load_3d(sV + st * L::kTileBytes + c * L::kChunkBytes, &tmap_v, &v_full[st], c * 64, j * kBN,
                                b * p.Hkv + kvh);
            }
        }
    } else if (warp == 1) {
        if (n_tiles > 0 && elect_one()) {
            constexpr uint32_t idesc_s = make_idesc_bf16(kBM, kBN, false, false);
            constexpr uint32_t idesc_o = make_idesc_bf16(kBM, D, false, true);
            const uint32_t q_addr = smem_u32(sQ), k_addr = smem_u32(sK), v_addr = smem_u32(sV), p_addr = smem_u32(sP);

            auto issue_qk = [&](int j) -> bool {
                const int st = j % kKVStages;
                if (!mbar_wait(&k_full[st], (j / kKVStages) & 1)) return false;
                tc_fence_after_sync();
                const uint32_t kb = k_addr + st * L::kTileBytes;
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                    const uint32_t off = (kk / 4) * L::kChunkBytes + (kk % 4) * 32;
                    mma_ss(tmem_base + kColS + (j & 1) * kBN, make_smem_desc(q_addr + off, 16, 1024),
                           make_smem_desc(kb + off, 16, 1024), idesc_s, kk != 0);
                }
                mma_commit(&k_empty[st]);
                mma_commit(&s_full[j & 1]);
                return true;
            };

            if (!mbar_wait(q_full, 0)) failed = true;
            if (!failed && !issue_qk(0)) failed = true;
            for (int j = 0; j < n_tiles && !failed; ++j) {
                if (j + 1 < n_tiles && !issue_qk(j + 1)) { failed = true; break; }
                const int st = j % kKVStages;
                if (!mbar_wait(p_ready, j & 1)) { failed = true; break; }
                if (!mbar_wait(&v_full[st], (j / kKVStages) & 1)) { failed = true; break; }
                tc_fence_after_sync();
                const uint32_t vb = v_addr + st * L::kTileBytes;
#pragma unroll
                for (int kk = 0; kk < kBN / 16; ++kk) {
                    // P: K-major, 16 keys = 32 bytes along the swizzled row, 64-key chunks 16 KB apart.
                    // V: MN-major, 16 keys = two 1024-byte groups; 64-wide chunks of D are 16 KB apart.
                    mma_ss(tmem_base + kColO,
                           make_smem_desc(p_addr + (kk / 4) * L::kChunkBytes + (kk % 4) * 32, 16, 1024),
                           make_smem_desc(vb + kk * 2048, L::kChunkBytes, 1024), idesc_o, (j | kk) != 0);
                }
                mma_commit(&v_empty[st]);
                mma_commit(pv_done);
            }
        }
    } else {
        const int quarter = warp & 3;
        const int row = quarter * 32 + lane;
        const int qi = q0 + row;
        const uint32_t lane_base = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
        const float sl2 = p.scale_log2;
        __nv_bfloat16* orow = p.out + ((size_t)(b * p.Hq + h) * p.Sq + qi) * D;

        if (n_tiles == 0) {
            if (qi < p.Sq) {
#pragma unroll
                for (int c = 0; c < D / 8; ++c) reinterpret_cast<uint4*>(orow)[c] = make_uint4(0, 0, 0, 0);
            }
        } else {
            float m_run = -INFINITY;  // running maximum of the raw scores (reference of the exponentials)
            float l_run = 0.f;
            const int row_limit = causal ? qi + causal_off : 0x7fffffff;  // last visible key of this row
            for (int j = 0; j < n_tiles; ++j) {
                if (!warp_wait(&s_full[j & 1], (j >> 1) & 1)) { failed = true; break; }
                tc_fence_after_sync();
                float s[kBN];
#pragma unroll
                for (int c = 0; c < kBN / 32; ++c) {
                    uint32_t r[32];
                    tmem_ld_x32(lane_base + kColS + (j & 1) * kBN + c * 32, r);
#pragma unroll
                    for (int i = 0; i < 32; ++i) s[c * 32 + i] = __uint_as_float(r[i]);
                }
                tmem_ld_wait();

                const int j0 = j * kBN;
                const bool need_mask = (j0 + kBN > kvlen) || (causal && (j0 + kBN - 1 > q0 + causal_off));
                if (need_mask) {
                    const int lim = min(kvlen - 1, row_limit) - j0;  // last visible column of this tile
#pragma unroll
                    for (int i = 0; i < kBN; ++i) s[i] = (i <= lim) ? s[i] : -INFINITY;
                }
                float m_tile = s[0];
#pragma unroll
                for (int i = 1; i < kBN; ++i) m_tile = fmaxf(m_tile, s[i]);

                // Keep the old reference unless this tile's maximum exceeds it by more than the
                // threshold (in log2 units of the scaled scores); then every later exponent is <= 8.
                float alpha = 1.f;
                bool grow = (m_tile - m_run) * sl2 > kRescaleThreshold || m_run == -INFINITY;
                if (m_tile == -INFINITY) grow = false;
                if (grow) {
                    // first visible keys of this row: nothing accumulated yet, nothing to rescale
                    alpha = (m_run == -INFINITY) ? 1.f : ex2((m_run - m_tile) * sl2);
                    m_run = m_tile;
                }
                const float m_ref = (m_run == -INFINITY) ? 0.f : m_run;
                const float neg_m = -m_ref * sl2;
                float l_tile = 0.f;
                uint32_t packed[kBN / 2];
#pragma unroll
                for (int i = 0; i < kBN / 2; ++i) {
                    // masked: s = -inf.  With sl2 > 0 the fma gives -inf and ex2 gives exactly 0.
                    float p0 = ex2(fmaf(s[2 * i], sl2, neg_m));
                    float p1 = ex2(fmaf(s[2 * i + 1], sl2, neg_m));
                    if (need_mask) {  // also covers sl2 == 0, where -inf * 0 would be NaN
                        p0 = (s[2 * i] == -INFINITY) ? 0.f : p0;
                        p1 = (s[2 * i + 1] == -INFINITY) ? 0.f : p1;
                    }
                    l_tile += p0 + p1;
                    packed[i] = pack_bf16(p0, p1);
                }
                l_run = l_run * alpha + l_tile;

                // P buffer and O are free once the previous P V has completed.
                if (j > 0) {
                    if (!warp_wait(pv_done, (j - 1) & 1)) { failed = true; break; }
                    tc_fence_after_sync();
                    if (__any_sync(0xffffffffu, alpha != 1.f)) {
#pragma unroll
                        for (int c = 0; c < D / 32; ++c) {
                            uint32_t r[32];
                            tmem_ld_x32(lane_base + kColO + c * 32, r);
                            tmem_ld_wait();
#pragma unroll
                            for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * alpha);
                            tmem_st_x32(lane_base + kColO + c * 32, r);
                        }
                        tmem_st_wait();
                    }
                }
                // P[row, 0..127] as bf16 into the K-major swizzled layout: 16-byte chunk c of the row
                // goes to chunk (c % 8) ^ (row % 8) of its 128-byte line; keys 64..127 sit 16 KB further.
#pragma unroll
                for (int c = 0; c < 16; ++c) {
                    uint8_t* dst = sP + (c / 8) * L::kChunkBytes + row * 128 + (((c % 8) ^ (row & 7)) << 4);
                    *reinterpret_cast<uint4*>(dst) =
                        make_uint4(packed[4 * c], packed[4 * c + 1], packed[4 * c + 2], packed[4 * c + 3]);
                }
                fence_proxy_async_smem();
                tc_fence_before_sync();
                mbar_arrive(p_ready);
            }

            if (!failed && !warp_wait(pv_done, (n_tiles - 1) & 1)) failed = true;
            if (!failed) {
                tc_fence_after_sync();
                const float inv = l_run > 0.f ? 1.f / l_run : 0.f;  // no visible key: zeros
#pragma unroll
                for (int c = 0; c < D / 32; ++c) {
                    uint32_t r[32];
                    tmem_ld_x32(lane_base + kColO + c * 32, r);
                    tmem_ld_wait();
                    if (qi < p.Sq) {
#pragma unroll
                        for (int v4 = 0; v4 < 4; ++v4) {
                            uint32_t w[4];
#pragma unroll
                            for (int i = 0; i < 4; ++i)
                                w[i] = pack_bf16(__uint_as_float(r[v4 * 8 + 2 * i]) * inv,
                                                 __uint_as_float(r[v4 * 8 + 2 * i + 1]) * inv);
                            reinterpret_cast<uint4*>(orow + c * 32)[v4] = make_uint4(w[0], w[1], w[2], w[3]);
                        }
                    }
                }
            }
        }
    }

    if (failed) {
        atomicExch(p.status, 1);
        for (int i = 0; i < 2000; ++i) __nanosleep(1000);  // let copies and MMAs in flight land
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

template <int D>
int launch_attn(const void* q, const void* k, const void* v, void* out, int B, int Hq, int Hkv, int Sq, int Skv,
                int mask_kind, const int32_t* lens, float scale, cudaStream_t s) {
    using L = AttnSmem<D>;
    CUtensorMap tq, tk, tv;
    const uint32_t box[3] = {64, 128, 1};
    {
        const uint64_t dims[3] = {(uint64_t)D, (uint64_t)Sq, (uint64_t)B * Hq};
        const uint64_t strides[2] = {(uint64_t)D * 2, (uint64_t)Sq * D * 2};
        if (!encode_tmap_bf16_sw128(&tq, q, 3, dims, strides, box)) return FORGE_ERR_CUDA;
    }
    {
        const uint64_t dims[3] = {(uint64_t)D, (uint64_t)Skv, (uint64_t)B * Hkv};
        const uint64_t strides[2] = {(uint64_t)D * 2, (uint64_t)Skv * D * 2};
        if (!encode_tmap_bf16_sw128(&tk, k, 3, dims, strides, box)) return FORGE_ERR_CUDA;
        if (!encode_tmap_bf16_sw128(&tv, v, 3, dims, strides, box)) return FORGE_ERR_CUDA;
    }
    AttnParams p;
    p.out = static_cast<__nv_bfloat16*>(out);
    p.lens = lens;
    p.Hq = Hq; p.Hkv = Hkv; p.Sq = Sq; p.Skv = Skv;
    p.mask_kind = mask_kind;
    p.scale_log2 = scale * 1.4426950408889634f;
    p.status = device_status_word();
    if (!p.status) return FORGE_ERR_CUDA;
    auto kernel = attn_bf16_kernel<D>;
    FORGE_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, L::kAlloc));
    const dim3 grid((Sq + kBM - 1) / kBM, Hq, B);
    kernel<<<grid, kThreads, L::kAlloc, s>>>(tq, tk, tv, p);
    return finish_launch(1);
}

}  // namespace
}  // namespace forge

extern "C" int forge_attn_fused(const void* q, const void* k, const void* v, void* out,
                                int B, int Hq, int Hkv, int Sq, int Skv, int D,
                                int mask_kind, const int32_t* lens, float scale, void* stream) {
    using namespace forge;
    int st = check_attn_args(q, k, v, out, B, Hq, Hkv, Sq, Skv, D, mask_kind, lens);
    if (st != FORGE_OK) return st;
    if (Hq > 65535 || B > 65535) return FORGE_ERR_UNSUPPORTED;
    if (!(scale >= 0.f)) return FORGE_ERR_UNSUPPORTED;  // the running maximum is taken on unscaled scores
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    return D == 64 ? launch_attn<64>(q, k, v, out, B, Hq, Hkv, Sq, Skv, mask_kind, lens, scale, s)
                   : launch_attn<128>(q, k, v, out, B, Hq, Hkv, Sq, Skv, mask_kind, lens, scale, s);
}
