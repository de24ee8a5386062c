// Fused attention for head sizes above 128, up to 256 (Eq. 8 / Eq. 9, the same operator as attn_bf16.cu).
// The two-tiles-per-CTA layout of that kernel does not fit here: two 256-column O accumulators fill the
// tensor memory and two 128 x 256 Q tiles most of the shared memory.  This kernel runs ONE 128-row query tile
// per work item:
//   tensor memory   S(even steps) at column 0, S(odd steps) at 64 (64 fp32 columns each), O at 128 (256 columns);
//                   P (16-bit, two per column) overwrites the first 32 columns of its S and is the A operand of P V
//   shared memory   Q 64 KB (four 64-column chunks of 128 rows x 128 B, 128-byte swizzle), two 32 KB stages of
//                   64 keys for K and two for V; the output is staged in Q's place before its TMA stores
//   warps 0-3       softmax, rescale and epilogue: thread = query row = TMEM lane
//   warp 4          TMA producer        warp 5   tcgen05.mma issuer (one elected lane), owns the TMEM allocation
// Per 64-key step g the issuer issues  O += P(g) V(g)  and then  S(g + 2) = Q K(g + 2)^T,  so the scores of the
// step after next are computed while the softmax threads work on the next one.  O is rescaled in tensor memory
// only when a row's maximum grows by more than 2^8 (the stale maximum is kept otherwise; the final division by
// l uses the same reference).  Head sizes that are not 256 (multiples of 8) cost time, not memory: the TMA unit
// zero-fills the missing columns on load and clips them on store.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "attn_wide.cuh"
#include "forge_common.cuh"
#include "sm100_ptx.cuh"
#include "tmap.cuh"

namespace forge {
namespace {

using namespace ptx;

constexpr int kD = 256;           // the kernel's head dimension
constexpr int kBM = 128;          // query rows per tile
constexpr int kStep = 64;         // keys per step and per K/V stage
constexpr int kStages = 2;
constexpr int kThreads = 192;
constexpr int kTmemCols = 512;
constexpr int kColS = 0;          // S of step g at kColS + (g & 1) * 64
constexpr int kColO = 128;
constexpr float kRescaleThreshold = 8.0f;  // log2 units

struct WideSmem {
    static constexpr int kChunkBytes = kBM * 128;               // Q: 128 rows x 64 elements
    static constexpr int kQBytes = (kD / 64) * kChunkBytes;     // 64 KB
    static constexpr int kKVChunkBytes = kStep * 128;           // K, V: 64 keys x 64 elements
    static constexpr int kKVBytes = (kD / 64) * kKVChunkBytes;  // 32 KB
    static constexpr int kQOff = 0;
    static constexpr int kKOff = kQOff + kQBytes;
    static constexpr int kVOff = kKOff + kStages * kKVBytes;
    static constexpr int kBarOff = kVOff + kStages * kKVBytes;
    // q_full, q_empty, k_full[2], k_empty[2], v_full[2], v_empty[2], s_full[2], p_ready[2], pv_done[2], o_free
    static constexpr int kNumBars = 2 + 4 * kStages + 7;
    static constexpr int kTotal = kBarOff + kNumBars * 8 + 16;
    static constexpr int kAlloc = kTotal + 1024;
};

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
template <bool F16>
__device__ __forceinline__ uint32_t pack16(float lo, float hi) {
    if constexpr (F16) {
        __half2 v = __floats2half2_rn(lo, hi);
        return *reinterpret_cast<uint32_t*>(&v);
    } else {
        __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
        return *reinterpret_cast<uint32_t*>(&v);
    }
}

struct WideParams {
    uint16_t* out;
    long long o_sb, o_sh, o_ss;  // element strides of out between batch entries, heads and rows
    const int32_t* lens;
    int B, Hq, Hkv, Sq, Skv, head_dim, mask_kind;
    float scale_log2;  // > 0
    int* status;
};

struct WideItem {
    int b, h, kvh, q0, kvlen, nsteps;  // nsteps: 64-key steps visible to at least one row of the tile (0: no work)
};

template <bool F16>
__global__ void __launch_bounds__(kThreads, 1)
attn_wide_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
                 const __grid_constant__ CUtensorMap tmap_v, const __grid_constant__ CUtensorMap tmap_o,
                 const WideParams p) {
    using L = WideSmem;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* sQ = smem + L::kQOff;
    uint8_t* sK = smem + L::kKOff;
    uint8_t* sV = smem + L::kVOff;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::kBarOff);
    uint64_t* q_full = bars;
    uint64_t* q_empty = bars + 1;            // the last scores of the item are done AND the epilogue has left Q's place
    uint64_t* k_full = bars + 2;
    uint64_t* k_empty = k_full + kStages;
    uint64_t* v_full = k_empty + kStages;
    uint64_t* v_empty = v_full + kStages;
    uint64_t* s_full = v_empty + kStages;    // [2] by step parity
    uint64_t* p_ready = s_full + 2;          // [2]
    uint64_t* pv_done = p_ready + 2;         // [2] one completion per P V product of that parity
    uint64_t* o_free = pv_done + 2;          // the epilogue has read O
    uint32_t* tmem_base_slot = reinterpret_cast<uint32_t*>(o_free + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = p.Hq / p.Hkv;
    const int num_q_tiles = (p.Sq + kBM - 1) / kBM;
    const int heads = p.B * p.Hq;
    const int num_items = num_q_tiles * heads;
    const int causal_off = p.Skv - p.Sq;
    const bool causal = (p.mask_kind & FORGE_MASK_CAUSAL) != 0;
    const bool padding = (p.mask_kind & FORGE_MASK_PADDING) != 0;

    // Items longest first (the last query tile of every head, then the one before, ...); CTA c takes item c of
    // every round of gridDim.x items, in alternating direction from round to round.
    auto item_of_round = [&](int r) {
        const int c = (r & 1) ? (int)gridDim.x - 1 - (int)blockIdx.x : (int)blockIdx.x;
        return r * (int)gridDim.x + c;
    };
    auto decode = [&](int i) {
        WideItem it;
        const int qstep = num_q_tiles - 1 - i / heads;
        const int bh = i % heads;
        it.b = bh / p.Hq;
        it.h = bh - it.b * p.Hq;
        it.kvh = it.h / G;
        it.q0 = qstep * kBM;
        it.kvlen = p.Skv;
        if (padding) it.kvlen = min(max(p.lens[it.b], 0), p.Skv);
        int kv_end = it.kvlen;
        if (causal) kv_end = min(kv_end, min(it.q0 + kBM, p.Sq) + causal_off);
        kv_end = max(kv_end, 0);
        it.nsteps = (kv_end + kStep - 1) / kStep;
        return it;
    };

    if (threadIdx.x == 0) {
        mbar_init(q_full, 1);
        mbar_init(q_empty, 1 + 4);  // the issuer's commit after the last scores + the four epilogue warps
        for (int i = 0; i < kStages; ++i) {
            mbar_init(&k_full[i], 1); mbar_init(&k_empty[i], 1);
            mbar_init(&v_full[i], 1); mbar_init(&v_empty[i], 1);
        }
        for (int i = 0; i < 2; ++i) { mbar_init(&s_full[i], 1); mbar_init(&p_ready[i], 4); mbar_init(&pv_done[i], 1); }
        mbar_init(o_free, 4);
        fence_mbar_init();
        prefetch_tmap(&tmap_q); prefetch_tmap(&tmap_k); prefetch_tmap(&tmap_v); prefetch_tmap(&tmap_o);
    }
    if (warp == 5) {
        tmem_alloc(tmem_base_slot, kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_base_slot;
    bool failed = false;
    pdl_launch_dependents();
    pdl_wait();

    if (warp == 4) {
        // ------------------------------------------------------------------ TMA producer
        if (elect_one()) {
            int kvn = 0;      // K/V stages loaded so far (ring position), across items
            int q_loads = 0;  // Q tiles loaded so far
            for (int r = 0; !failed; ++r) {
                const int i = item_of_round(r);
                if (i >= num_items) break;
                const WideItem it = decode(i);
                if (it.nsteps == 0) continue;
                if (!mbar_wait(q_empty, (q_loads & 1) ^ 1)) { failed = true; break; }
                ++q_loads;
                mbar_expect_tx(q_full, L::kQBytes);
#pragma unroll
                for (int c = 0; c < kD / 64; ++c)  // rows beyond Sq and columns beyond head_dim are zero-filled
                    tma_load_4d(sQ + c * L::kChunkBytes, &tmap_q, q_full, c * 64, it.q0, it.h, it.b);
                for (int j = 0; j < it.nsteps && !failed; ++j, ++kvn) {
                    const int st = kvn % kStages;
                    const uint32_t ph = (kvn / kStages) & 1;
                    if (!mbar_wait(&k_empty[st], ph ^ 1)) { failed = true; break; }
                    mbar_expect_tx(&k_full[st], L::kKVBytes);
#pragma unroll
                    for (int c = 0; c < kD / 64; ++c)
                        tma_load_4d(sK + st * L::kKVBytes + c * L::kKVChunkBytes, &tmap_k, &k_full[st], c * 64, j * kStep, it.kvh, it.b);
                    if (!mbar_wait(&v_empty[st], ph ^ 1)) { failed = true; break; }
                    mbar_expect_tx(&v_full[st], L::kKVBytes);
#pragma unroll
                    for (int c = 0; c < kD / 64; ++c)
                        tma_load_4d(sV + st * L::kKVBytes + c * L::kKVChunkBytes, &tmap_v, &v_full[st], c * 64, j * kStep, it.kvh, it.b);
                }
            }
        }
    } else if (warp == 5) {
        // ------------------------------------------------------------------ MMA issuer
        if (elect_one()) {
            constexpr uint32_t idesc_s = F16 ? make_idesc_f16(kBM, kStep, false, false) : make_idesc_bf16(kBM, kStep, false, false);
            constexpr uint32_t idesc_o = F16 ? make_idesc_f16(kBM, kD, false, true) : make_idesc_bf16(kBM, kD, false, true);
            const uint32_t q_addr = smem_u32(sQ), k_addr = smem_u32(sK), v_addr = smem_u32(sV);
            const uint32_t o_tmem = tmem_base + kColO;
            const uint64_t qd = make_smem_desc(q_addr, 16, 1024);
            int kvbase = 0;   // ring position of the item's first K/V stage
            int items = 0;    // items with work so far (phases of q_full, o_free)
            int steps[2] = {0, 0};  // steps issued so far per parity (phases of p_ready)
            for (int r = 0; !failed; ++r) {
                const int i = item_of_round(r);
                if (i >= num_items) break;
                const WideItem it = decode(i);
                const int n = it.nsteps;
                if (n == 0) continue;
                // S(g) = Q K(g)^T into S[g & 1]
                auto issue_qk = [&](int g) -> bool {
                    const int pos = kvbase + g, st = pos % kStages;
                    if (!mbar_wait(&k_full[st], (pos / kStages) & 1)) return false;
                    tc_fence_after_sync();
                    const uint64_t kd = make_smem_desc(k_addr + st * L::kKVBytes, 16, 1024);
#pragma unroll
                    for (int kk = 0; kk < kD / 16; ++kk) {
                        const uint32_t qoff = ((kk / 4) * L::kChunkBytes + (kk % 4) * 32) >> 4;
                        const uint32_t koff = ((kk / 4) * L::kKVChunkBytes + (kk % 4) * 32) >> 4;
                        mma_ss(tmem_base + kColS + (g & 1) * kStep, qd + qoff, kd + koff, idesc_s, kk != 0);
                    }
                    mma_commit(&s_full[g & 1]);
                    mma_commit(&k_empty[st]);
                    if (g == n - 1) mma_commit(q_empty);  // the item's last scores: Q is no longer read
                    return true;
                };
                if (!mbar_wait(q_full, items & 1)) { failed = true; break; }
                if (!issue_qk(0) || (n > 1 && !issue_qk(1))) { failed = true; break; }
                for (int g = 0; g < n; ++g) {
                    const int hh = g & 1, pos = kvbase + g, st = pos % kStages;
                    if (!mbar_wait(&v_full[st], (pos / kStages) & 1)) { failed = true; break; }
                    if (!mbar_wait(&p_ready[hh], steps[hh] & 1)) { failed = true; break; }
                    ++steps[hh];
                    // the first product of an item overwrites O: the previous item's epilogue must have read it
                    if (g == 0 && !mbar_wait(o_free, (items & 1) ^ 1)) { failed = true; break; }
                    tc_fence_after_sync();
                    // P: 16 keys = 8 columns of packed 16-bit pairs.  V: MN-major, 16 keys = two 1024-byte groups
                    // (2048 bytes per step); the 64-wide chunks of D are 8 KB apart.
                    const uint64_t vd = make_smem_desc(v_addr + st * L::kKVBytes, L::kKVChunkBytes, 1024);
                    const uint32_t p_tmem = tmem_base + kColS + hh * kStep;
#pragma unroll
                    for (int kk = 0; kk < kStep / 16; ++kk)
                        mma_ts(o_tmem, p_tmem + kk * 8, vd + kk * (2048 >> 4), idesc_o, (g | kk) != 0);
                    mma_commit(&pv_done[hh]);
                    mma_commit(&v_empty[st]);
                    if (g + 2 < n && !issue_qk(g + 2)) { failed = true; break; }
                }
                if (failed) break;
                kvbase += n;
                ++items;
            }
        }
    } else {
        // ------------------------------------------------------------------ softmax / rescale / epilogue
        const int row = warp * 32 + lane;
        const uint32_t lane_base = tmem_base + (static_cast<uint32_t>(warp * 32) << 16);
        const float sl2 = p.scale_log2;
        int steps[2] = {0, 0};  // steps done so far per parity (phases of s_full, pv_done)
        int kvbase = 0;
        for (int r = 0; !failed; ++r) {
            const int i = item_of_round(r);
            if (i >= num_items) break;
            const WideItem it = decode(i);
            const int qi = it.q0 + row;
            const int n = it.nsteps;
            if (n == 0) {  // no visible key for any row of this tile: zeros, with plain stores
                if (qi < p.Sq) {
                    uint16_t* orow = p.out + it.b * p.o_sb + it.h * p.o_sh + qi * p.o_ss;
                    for (int c = 0; c < p.head_dim / 8; ++c) reinterpret_cast<uint4*>(orow)[c] = make_uint4(0, 0, 0, 0);
                }
                continue;
            }
            float m_run = -INFINITY, l_run = 0.f;
            const int row_limit = min(it.kvlen - 1, causal ? qi + causal_off : 0x7fffffff);  // last visible key of this row
#pragma unroll 1
            for (int g = 0; g < n; ++g) {
                const int hh = g & 1;
                const uint32_t col_h = kColS + hh * kStep;
                if (!warp_wait(&s_full[hh], steps[hh] & 1)) { failed = true; break; }
                tc_fence_after_sync();
                float s[kStep];
#pragma unroll
                for (int c = 0; c < kStep / 32; ++c) {
                    uint32_t rr[32];
                    tmem_ld_x32(lane_base + col_h + c * 32, rr);
#pragma unroll
                    for (int k = 0; k < 32; ++k) s[c * 32 + k] = __uint_as_float(rr[k]);
                }
                tmem_ld_wait();
                const int key0 = g * kStep;
                const int lim = row_limit - key0;  // last visible column of this step
                if (lim < kStep - 1) {
#pragma unroll
                    for (int k = 0; k < kStep; ++k) s[k] = (k <= lim) ? s[k] : -INFINITY;
                }
                float m_tile = s[0];
#pragma unroll
                for (int k = 1; k < kStep; ++k) m_tile = fmaxf(m_tile, s[k]);
                // keep the old reference unless this step's maximum exceeds it by more than the threshold
                float alpha = 1.f;
                bool grow = (m_tile - m_run) * sl2 > kRescaleThreshold || m_run == -INFINITY;
                if (m_tile == -INFINITY) grow = false;
                if (grow) {
                    alpha = (m_run == -INFINITY) ? 1.f : ex2((m_run - m_tile) * sl2);
                    m_run = m_tile;
                }
                if (g > 0 && __any_sync(0xffffffffu, alpha != 1.f)) {
                    // O must hold every product issued so far and none may be in flight: the barrier above covers the
                    // products up to g - 2, the product of step g - 1 has its own
                    if (!warp_wait(&pv_done[hh ^ 1], (steps[hh ^ 1] - 1) & 1)) { failed = true; break; }
                    tc_fence_after_sync();
#pragma unroll 1
                    for (int c = 0; c < kD / 32; ++c) {
                        uint32_t rr[32];
                        tmem_ld_x32(lane_base + kColO + c * 32, rr);
                        tmem_ld_wait();
#pragma unroll
                        for (int k = 0; k < 32; ++k) rr[k] = __float_as_uint(__uint_as_float(rr[k]) * alpha);
                        tmem_st_x32(lane_base + kColO + c * 32, rr);
                    }
                }
                ++steps[hh];
                const float m_ref = (m_run == -INFINITY) ? 0.f : m_run;
                const float neg_m = -m_ref * sl2;
                float l_tile = 0.f;
                uint32_t packed[32];
#pragma unroll
                for (int k = 0; k < 32; ++k) {
                    const float p0 = ex2(fmaf(s[2 * k], sl2, neg_m)), p1 = ex2(fmaf(s[2 * k + 1], sl2, neg_m));  // masked: 0
                    l_tile += p0 + p1;
                    packed[k] = pack16<F16>(p0, p1);
                }
                tmem_st_x32(lane_base + col_h, packed);
                l_run = l_run * alpha + l_tile;
                // V rows at and beyond lens[b] hold the caller's padding (possibly NaN): zero them before the product
                if (padding && key0 + kStep > it.kvlen && it.kvlen < p.Skv) {
                    const int pos = kvbase + g, st = pos % kStages;
                    if (!warp_wait(&v_full[st], (pos / kStages) & 1)) { failed = true; break; }
                    const int first = max(it.kvlen - key0, 0);
                    const int per_chunk = (kStep - first) * 8;  // 16-byte pieces to clear per 64-column chunk
                    uint8_t* vt = sV + st * L::kKVBytes;
                    for (int t = warp * 32 + lane; t < (kD / 64) * per_chunk; t += 128) {
                        const int c = t / per_chunk, rem = t - c * per_chunk;
                        *reinterpret_cast<uint4*>(vt + c * L::kKVChunkBytes + (first + (rem >> 3)) * 128 + ((rem & 7) << 4)) =
                            make_uint4(0, 0, 0, 0);
                    }
                    fence_proxy_async_smem();
                }
                tmem_st_wait();
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(&p_ready[hh]);
            }
            if (failed) break;
            // the last product of either parity
            if (steps[0] > 0 && !warp_wait(&pv_done[0], (steps[0] - 1) & 1)) { failed = true; break; }
            if (steps[1] > 0 && !warp_wait(&pv_done[1], (steps[1] - 1) & 1)) { failed = true; break; }
            tc_fence_after_sync();
            // O / l as 16-bit values into Q's place (all scores of the item are done), 32 columns at a time
            const float inv = l_run > 0.f ? 1.f / l_run : 0.f;
#pragma unroll 1
            for (int c32 = 0; c32 < kD / 32; ++c32) {
                uint32_t cur[32];
                tmem_ld_x32(lane_base + kColO + c32 * 32, cur);
                tmem_ld_wait();
                uint8_t* line = sQ + (c32 >> 1) * L::kChunkBytes + row * 128;
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    uint32_t w[4];
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        w[k] = pack16<F16>(__uint_as_float(cur[c * 8 + 2 * k]) * inv, __uint_as_float(cur[c * 8 + 2 * k + 1]) * inv);
                    *reinterpret_cast<uint4*>(line + ((((c32 & 1) * 4 + c) ^ (row & 7)) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
                }
            }
            tc_fence_before_sync();
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(o_free);  // O may be overwritten by the next item's first product
                const int row0 = it.q0 + warp * 32;
                if (row0 < p.Sq) {
#pragma unroll
                    for (int cb = 0; cb < kD / 64; ++cb)
                        if (cb * 64 < p.head_dim) tma_store_4d(&tmap_o, sQ + cb * L::kChunkBytes + warp * 32 * 128, cb * 64, row0, it.h, it.b);
                    tma_store_commit();
                    tma_store_wait_read<0>();  // the stores have read the staging rows: Q's place is free again
                }
                mbar_arrive(q_empty);
            }
            kvbase += n;
        }
        if (lane == 0) tma_store_wait_all<0>();
    }

    if (failed) {
        atomicExch(p.status, 1);
        for (int i = 0; i < 2000; ++i) __nanosleep(1000);  // let copies and MMAs in flight land
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 5) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

template <bool F16>
int launch_wide(const void* q, const void* k, const void* v, void* out, int B, int Hq, int Hkv, int Sq, int Skv,
                int head_dim, int mask_kind, const int32_t* lens, float scale, const long long (*st)[3], cudaStream_t s) {
    using L = WideSmem;
    auto encode = [&](CUtensorMap* m, const void* base, int H, int S, const long long* str, uint32_t box_rows) {
        const uint32_t box[4] = {64, box_rows, 1, 1};
        const uint64_t dims[4] = {(uint64_t)head_dim, (uint64_t)S, (uint64_t)H, (uint64_t)B};
        const uint64_t strides[3] = {(uint64_t)str[2] * 2, (uint64_t)str[1] * 2, (uint64_t)str[0] * 2};
        return encode_tmap_bf16_sw128(m, base, 4, dims, strides, box);
    };
    CUtensorMap tq, tk, tv, to;
    if (!encode(&tq, q, Hq, Sq, st[0], kBM)) return FORGE_ERR_CUDA;
    if (!encode(&tk, k, Hkv, Skv, st[1], kStep)) return FORGE_ERR_CUDA;
    if (!encode(&tv, v, Hkv, Skv, st[2], kStep)) return FORGE_ERR_CUDA;
    if (!encode(&to, out, Hq, Sq, st[3], 32)) return FORGE_ERR_CUDA;
    WideParams p;
    p.out = static_cast<uint16_t*>(out);
    p.o_sb = st[3][0]; p.o_sh = st[3][1]; p.o_ss = st[3][2];
    p.lens = lens;
    p.B = B; p.Hq = Hq; p.Hkv = Hkv; p.Sq = Sq; p.Skv = Skv; p.head_dim = head_dim; p.mask_kind = mask_kind;
    p.scale_log2 = scale * 1.4426950408889634f;
    // scale = 0 (uniform weights): any positive multiplier whose products with the scores flush to zero
    if (!(p.scale_log2 > 0.f)) p.scale_log2 = 1.17549435e-38f;
    p.status = device_status_word();
    if (!p.status) return FORGE_ERR_CUDA;
    auto kernel = attn_wide_kernel<F16>;
    FORGE_SET_SMEM_ONCE(kernel, L::kAlloc);
    const int sms = sm_count();
    if (sms <= 0) return FORGE_ERR_CUDA;
    const long long items = (long long)B * Hq * ((Sq + kBM - 1) / kBM);
    const int grid = items < sms ? (int)items : sms;
    FORGE_CUDA_TRY(launch_pdl(kernel, dim3(grid), dim3(kThreads), L::kAlloc, s, tq, tk, tv, to, p));
    return finish_launch(1);
}

}  // namespace

int attn_wide(bool f16, const void* q, const void* k, const void* v, void* out, int B, int Hq, int Hkv, int Sq, int Skv,
              int head_dim, int mask_kind, const int32_t* lens, float scale, const long long (*strides)[3], cudaStream_t s) {
    return f16 ? launch_wide<true>(q, k, v, out, B, Hq, Hkv, Sq, Skv, head_dim, mask_kind, lens, scale, strides, s)
               : launch_wide<false>(q, k, v, out, B, Hq, Hkv, Sq, Skv, head_dim, mask_kind, lens, scale, strides, s);
}

}  // namespace forge
