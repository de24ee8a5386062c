// Fused attention, bf16 in / fp32 accumulate / bf16 out (Eq. 8 / Eq. 9): scores, mask, online
// softmax and the product with V in one kernel; S and P never reach global memory.
//
// One work item = two 128-row query tiles that share K and V (see the item decoding below).  The two tiles run in ping-pong so
// that the tensor core works on one tile while the softmax of the other is computed.  Warp roles:
//   warps 0-3 : softmax / rescale / epilogue of tile 0; thread = one query row (TMEM lane), so row
//   warps 4-7 : the same for tile 1                    maxima and sums need no cross-thread reduction
//   warp 8    : TMA producer: both Q tiles once, then K and V tiles (128 keys) through rings
//   warp 9    : tcgen05.mma issuer (one elected lane), owns the TMEM allocation
//   warps 10-11 only complete the third warpgroup, which hands most of its registers to the other two
//   (setmaxnreg: 224 per softmax thread, 56 for the rest; 256*224 + 128*56 = 384*168 as launched).
// Tensor memory (512 columns): S_0 at 0, S_1 at 128 (128 x 128 fp32 each), O_0 at 256, O_1 at 256 + D.
// P_t (bf16, two per column) is written over the first 64 columns of S_t and is the A operand of
// the P V product straight from tensor memory.  MMAs execute in issue order, so the issue sequence
//   S_0(0) S_1(0) | P_0 ready: O_0 += P_0 V_0, S_0(1) | P_1 ready: O_1 += P_1 V_0, S_1(1) | ...
// keeps every hazard (P_t read before S_t is overwritten, O_t complete before it is rescaled) safe:
// the barrier that announces S_t(j+1) also covers the completion of every earlier MMA.
// O is rescaled in TMEM only when a row's maximum grows by more than 2^8 (the stale maximum is
// kept otherwise; the final division by l uses the same reference, so the result is unchanged).
// Q and K are K-major operands, V [keys, D] is the MN-major B operand of P V.
#include <cuda_bf16.h>

#include <type_traits>

#include "forge_common.cuh"
#include "sm100_ptx.cuh"
#include "tmap.cuh"

namespace forge {
namespace {

using namespace ptx;

constexpr int kBM = 128;          // query rows per tile
constexpr int kTilesPerCta = 2;
constexpr int kBN = 128;          // keys per tile
constexpr int kThreads = 384;
constexpr int kSoftmaxThreads = 128;  // per query tile
constexpr int kTmemCols = 512;
constexpr int kColS = 0;          // S_t at t * 128
constexpr int kColO = 256;        // O_t at 256 + t * D
constexpr float kRescaleThreshold = 8.0f;  // log2 units

template <int D>
struct AttnSmem {
    static constexpr int kChunkBytes = 128 * 128;              // 128 rows x 64 bf16 (one swizzle span wide)
    static constexpr int kTileBytes = (D / 64) * kChunkBytes;  // a Q, K or V tile
    static constexpr int kKVStages = (D == 64) ? 4 : 2;
    static constexpr int kQOff = 0;
    static constexpr int kKOff = kQOff + kTilesPerCta * kTileBytes;
    static constexpr int kVOff = kKOff + kKVStages * kTileBytes;
    static constexpr int kOutOff = kVOff + kKVStages * kTileBytes;  // output staging: 128 rows x 64 bf16 per query tile
    static constexpr int kBarOff = kOutOff + kTilesPerCta * kChunkBytes;
    // q_full, k/v full+empty per stage, s_full[2], p_ready[2], pv_done[2]
    static constexpr int kNumBars = 2 + 4 * kKVStages + 10;
    static constexpr int kTotal = kBarOff + kNumBars * 8 + 16;
    static constexpr int kAlloc = kTotal + 1024;
};

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// 3-input maximum and packed two-wide fp32 arithmetic (one instruction for two elements)
__device__ __forceinline__ float max3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
__device__ __forceinline__ float2 ffma2(float2 a, float2 b, float2 c) {
    float2 d;
    asm("{\n\t.reg .b64 ra, rb, rc, rd;\n\t"
        "mov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %5};\n\tmov.b64 rc, {%6, %7};\n\t"
        "fma.rn.f32x2 rd, ra, rb, rc;\n\t"
        "mov.b64 {%0, %1}, rd;\n\t}"
        : "=f"(d.x), "=f"(d.y)
        : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y), "f"(c.x), "f"(c.y));
    return d;
}
__device__ __forceinline__ float2 fadd2(float2 a, float2 b) {
    float2 d;
    asm("{\n\t.reg .b64 ra, rb, rd;\n\t"
        "mov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %5};\n\t"
        "add.rn.f32x2 rd, ra, rb;\n\t"
        "mov.b64 {%0, %1}, rd;\n\t}"
        : "=f"(d.x), "=f"(d.y)
        : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y));
    return d;
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

struct AttnParams {
    __nv_bfloat16* out;
    const int32_t* lens;
    int B, Hq, Hkv, Sq, Skv;
    int mask_kind;
    float scale_log2;
    int* status;
};

// What one CTA needs to know about a work item (a pair of query tiles of one head).
struct ItemInfo {
    int b, kvlen;
    int kvh[kTilesPerCta];      // KV head of each tile (equal unless the tiles read separate K/V streams)
    int q0[kTilesPerCta];       // first query row of each of the two tiles
    int h[kTilesPerCta];        // query head of each tile
    int n_tiles[kTilesPerCta];  // KV tiles visible to at least one row of each query tile (0: tile beyond Sq)
    int n_max;
};

template <int D>
__global__ void __launch_bounds__(kThreads, 1)
attn_bf16_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
                 const __grid_constant__ CUtensorMap tmap_v, const __grid_constant__ CUtensorMap tmap_o,
                 const AttnParams p) {
    using L = AttnSmem<D>;
    constexpr int kKVStages = L::kKVStages;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* sQ = smem + L::kQOff;
    uint8_t* sK = smem + L::kKOff;
    uint8_t* sV = smem + L::kVOff;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::kBarOff);
    uint64_t* q_full = bars;
    uint64_t* q_empty = bars + 1;
    uint64_t* k_full = bars + 2;
    uint64_t* k_empty = k_full + kKVStages;
    uint64_t* v_full = k_empty + kKVStages;
    uint64_t* v_empty = v_full + kKVStages;
    uint64_t* s_full = v_empty + kKVStages;  // [2] per query tile
    uint64_t* p_ready = s_full + 2;          // [2]
    uint64_t* pv_done = p_ready + 2;         // [2]
    uint64_t* o_free = pv_done + 2;          // [2]
    uint64_t* wg_bar = o_free + 2;           // [2] meeting point of a tile's four softmax warps
    uint32_t* tmem_base_slot = reinterpret_cast<uint32_t*>(wg_bar + 2);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // The two tiles of an item: with an even number of query heads per KV head, the same 128 query rows of
    // two heads that share K and V (equal causal lengths, so neither tile waits for the other); otherwise
    // two consecutive 128-row tiles of one head.
    const int G = p.Hq / p.Hkv;
    const bool pair_heads = (G % 2) == 0;
    // With an odd group size and D = 64 (where shared memory has room for it) the two tiles are still two
    // heads on the same query rows, each with its own K/V stream through half of the stage ring.
    const bool two_streams = !pair_heads && kKVStages >= 4;
    const int ring_len = two_streams ? kKVStages / 2 : kKVStages;
    const int num_q_tiles = (p.Sq + kBM - 1) / kBM;
    const int head_pairs = (p.Hq + 1) / 2;
    const int rows_of_items = (pair_heads || two_streams) ? num_q_tiles : (num_q_tiles + 1) / 2;
    const int heads = (pair_heads || two_streams) ? head_pairs * p.B : p.Hq * p.B;  // items per query step
    const int num_items = rows_of_items * heads;
    // ring slot and phase of the g-th KV tile of stream u
    auto kv_slot = [&](int u, int g) { return (two_streams ? u * ring_len : 0) + g % ring_len; };
    auto kv_phase = [&](int g) { return (uint32_t)((g / ring_len) & 1); };
    const int causal_off = p.Skv - p.Sq;
    const bool causal = (p.mask_kind & FORGE_MASK_CAUSAL) != 0;

    // Persistent schedule.  Items are ordered longest first (the last query-tile pair of every head, then
    // the one before, ...); CTA c takes item c of every round of gridDim.x items, in alternating direction
    // from round to round, which keeps the per-CTA sums of causal work close together.
    auto item_of_round = [&](int r) {
        const int c = (r & 1) ? (int)gridDim.x - 1 - (int)blockIdx.x : (int)blockIdx.x;
        return r * (int)gridDim.x + c;
    };
    auto decode = [&](int i) {
        ItemInfo it;
        const int qstep = rows_of_items - 1 - i / heads;  // longest (causal) first
        const int hb = i % heads;
        if (pair_heads || two_streams) {
            const int hp = hb % head_pairs;
            it.b = hb / head_pairs;
            it.h[0] = 2 * hp;
            it.h[1] = min(2 * hp + 1, p.Hq - 1);
            it.q0[0] = it.q0[1] = qstep * kBM;
            if (2 * hp + 1 >= p.Hq) it.q0[1] = num_q_tiles * kBM;  // odd head count: no second tile
        } else {
            it.b = hb / p.Hq;
            it.h[0] = it.h[1] = hb % p.Hq;
            it.q0[0] = 2 * qstep * kBM; it.q0[1] = (2 * qstep + 1) * kBM;
        }
        it.kvh[0] = it.h[0] / G;
        it.kvh[1] = it.h[1] / G;
        it.kvlen = p.Skv;
        if (p.mask_kind & FORGE_MASK_PADDING) it.kvlen = min(max(p.lens[it.b], 0), p.Skv);
        it.n_max = 0;
#pragma unroll
        for (int t = 0; t < kTilesPerCta; ++t) {
            const int q0 = it.q0[t];
            int kv_end = it.kvlen;
            if (causal) kv_end = min(kv_end, min(q0 + kBM, p.Sq) + causal_off);
            if (q0 >= p.Sq) kv_end = 0;
            kv_end = max(kv_end, 0);
            it.n_tiles[t] = (kv_end + kBN - 1) / kBN;
            it.n_max = max(it.n_max, it.n_tiles[t]);
        }
        return it;
    };

    if (threadIdx.x == 0) {
        mbar_init(q_full, 1);
        mbar_init(q_empty, 1);
        for (int i = 0; i < kKVStages; ++i) {
            mbar_init(&k_full[i], 1); mbar_init(&k_empty[i], 1);
            mbar_init(&v_full[i], 1); mbar_init(&v_empty[i], 1);
        }
        for (int t = 0; t < 2; ++t) {
            mbar_init(&s_full[t], 1); mbar_init(&p_ready[t], kSoftmaxThreads / 32);
            mbar_init(&pv_done[t], 1); mbar_init(&o_free[t], kSoftmaxThreads / 32);
            mbar_init(&wg_bar[t], kSoftmaxThreads / 32);
        }
        fence_mbar_init();
        prefetch_tmap(&tmap_q); prefetch_tmap(&tmap_k); prefetch_tmap(&tmap_v); prefetch_tmap(&tmap_o);
    }
    if (warp == 9) {
        tmem_alloc(tmem_base_slot, kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_base_slot;
    bool failed = false;

    if (warp >= 8) {
      asm volatile("setmaxnreg.dec.sync.aligned.u32 56;");
      if (warp == 8) {
        // ------------------------------------------------------------------ TMA producer
        if (elect_one()) {
            int kvn[2] = {0, 0};  // KV tiles loaded so far per stream (ring position), across items
            int items = 0;        // items with work so far
            for (int r = 0; !failed; ++r) {
                const int i = item_of_round(r);
                if (i >= num_items) break;
                const ItemInfo it = decode(i);
                if (it.n_max == 0) continue;
                // the previous item's last S = Q K^T has been issued and completed: Q may be replaced
                if (!mbar_wait(q_empty, (items & 1) ^ 1)) { failed = true; break; }
                mbar_expect_tx(q_full, kTilesPerCta * L::kTileBytes);
#pragma unroll
                for (int t = 0; t < kTilesPerCta; ++t)
#pragma unroll
                    for (int c = 0; c < D / 64; ++c)  // rows beyond Sq are zero-filled by the TMA unit
                        tma_load_3d(sQ + t * L::kTileBytes + c * L::kChunkBytes, &tmap_q, q_full, c * 64,
                                    it.q0[t], it.b * p.Hq + it.h[t]);
                for (int j = 0; j < it.n_max && !failed; ++j) {
                    for (int u = 0; u < (two_streams ? 2 : 1); ++u) {
                        if (two_streams && j >= it.n_tiles[u]) continue;
                        const int g = kvn[u]++, st = kv_slot(u, g);
                        const uint32_t ph = kv_phase(g);
                        const int kv_row = it.b * p.Hkv + it.kvh[u];
                        if (!mbar_wait(&k_empty[st], ph ^ 1)) { failed = true; break; }
                        mbar_expect_tx(&k_full[st], L::kTileBytes);
#pragma unroll
                        for (int c = 0; c < D / 64; ++c)
                            tma_load_3d(sK + st * L::kTileBytes + c * L::kChunkBytes, &tmap_k, &k_full[st], c * 64,
                                        j * kBN, kv_row);
                        if (!mbar_wait(&v_empty[st], ph ^ 1)) { failed = true; break; }
                        mbar_expect_tx(&v_full[st], L::kTileBytes);
#pragma unroll
                        for (int c = 0; c < D / 64; ++c)
                            tma_load_3d(sV + st * L::kTileBytes + c * L::kChunkBytes, &tmap_v, &v_full[st], c * 64,
                                        j * kBN, kv_row);
                    }
                }
                ++items;
            }
        }
      } else if (warp == 9) {
        // ------------------------------------------------------------------ MMA issuer
        if (elect_one()) {
            constexpr uint32_t idesc_s = make_idesc_bf16(kBM, kBN, false, false);
            constexpr uint32_t idesc_o = make_idesc_bf16(kBM, D, false, true);
            const uint32_t q_addr = smem_u32(sQ), k_addr = smem_u32(sK), v_addr = smem_u32(sV);
            int kvbase[2] = {0, 0};          // per stream: ring position of the item's first KV tile
            int k_waited[2] = {-1, -1}, v_waited[2] = {-1, -1};  // highest ring position seen to have arrived
            int items = 0;                  // items with work so far
            int its[kTilesPerCta] = {0, 0};     // tile iterations issued so far per query tile (barrier phases)
            int used[kTilesPerCta] = {0, 0};    // items in which each query tile had work (phase of o_free)

            for (int r = 0; !failed; ++r) {
                const int i = item_of_round(r);
                if (i >= num_items) break;
                const ItemInfo it = decode(i);
                if (it.n_max == 0) continue;

                int qk_issued = 0;
                const int qk_total = it.n_tiles[0] + it.n_tiles[1];
                // S_t(j) = Q_t K_j^T; the last tile that uses K_j releases its stage
                auto issue_qk = [&](int t, int j) -> bool {
                    const int u = two_streams ? t : 0, g = kvbase[u] + j, st = kv_slot(u, g);
                    if (g > k_waited[u]) {
                        if (!mbar_wait(&k_full[st], kv_phase(g))) return false;
                        k_waited[u] = g;
                    }
                    tc_fence_after_sync();
                    // descriptors differ only in the start-address field: build one per operand, then add
                    // (byte offset >> 4) for each 16-wide K step (the field cannot overflow below 256 KB)
                    const uint64_t qd = make_smem_desc(q_addr + t * L::kTileBytes, 16, 1024);
                    const uint64_t kd = make_smem_desc(k_addr + st * L::kTileBytes, 16, 1024);
#pragma unroll
                    for (int kk = 0; kk < D / 16; ++kk) {
                        const uint32_t off = ((kk / 4) * L::kChunkBytes + (kk % 4) * 32) >> 4;
                        mma_ss(tmem_base + kColS + t * kBN, qd + off, kd + off, idesc_s, kk != 0);
                    }
                    bool last = true;  // no later tile reads this K tile (always so with separate streams)
                    for (int t2 = t + 1; t2 < kTilesPerCta && !two_streams; ++t2) last = last && !(j < it.n_tiles[t2]);
                    if (last) mma_commit(&k_empty[st]);
                    mma_commit(&s_full[t]);
                    // the item's last S = Q K^T: once it completes, the next item's Q tiles may be loaded
                    if (++qk_issued == qk_total) mma_commit(q_empty);
                    return true;
                };
                // O_t += P_t(j) V_j with P_t read from tensor memory
                auto issue_pv = [&](int t, int j) -> bool {
                    const int u = two_streams ? t : 0, g = kvbase[u] + j, st = kv_slot(u, g);
                    if (!mbar_wait(&p_ready[t], its[t] & 1)) return false;
                    if (g > v_waited[u]) {
                        if (!mbar_wait(&v_full[st], kv_phase(g))) return false;
                        v_waited[u] = g;
                    }
                    // the first product of an item overwrites O_t: the previous item's epilogue must have read it
                    if (j == 0 && !mbar_wait(&o_free[t], (used[t] & 1) ^ 1)) return false;
                    tc_fence_after_sync();
                    // P: 16 keys = 8 columns of packed bf16 pairs.  V: MN-major, 16 keys = two 1024-byte groups
                    // (2048 bytes per step); the 64-wide chunks of D are 16 KB apart.
                    const uint64_t vd = make_smem_desc(v_addr + st * L::kTileBytes, L::kChunkBytes, 1024);
                    const uint32_t o_tmem = tmem_base + kColO + t * D, p_tmem = tmem_base + kColS + t * kBN;
                    if (j == 0) mma_ts(o_tmem, p_tmem, vd, idesc_o, 0u);
                    else mma_ts(o_tmem, p_tmem, vd, idesc_o, 1u);
#pragma unroll
                    for (int kk = 1; kk < kBN / 16; ++kk) mma_ts(o_tmem, p_tmem + kk * 8, vd + kk * (2048 >> 4), idesc_o, 1u);
                    bool last = true;
                    for (int t2 = t + 1; t2 < kTilesPerCta && !two_streams; ++t2) last = last && !(j < it.n_tiles[t2]);
                    if (last) mma_commit(&v_empty[st]);
                    mma_commit(&pv_done[t]);
                    ++its[t];
                    return true;
                };

                if (!mbar_wait(q_full, items & 1)) { failed = true; break; }
                for (int t = 0; t < kTilesPerCta && !failed; ++t)
                    if (it.n_tiles[t] > 0 && !issue_qk(t, 0)) failed = true;
                for (int j = 0; j < it.n_max && !failed; ++j) {
                    for (int t = 0; t < kTilesPerCta && !failed; ++t) {
                        if (j >= it.n_tiles[t]) continue;
                        if (!issue_pv(t, j)) { failed = true; break; }
                        if (j + 1 < it.n_tiles[t] && !issue_qk(t, j + 1)) { failed = true; break; }
                    }
                }
                for (int t = 0; t < kTilesPerCta; ++t) used[t] += it.n_tiles[t] > 0;
                if (two_streams) { kvbase[0] += it.n_tiles[0]; kvbase[1] += it.n_tiles[1]; }
                else kvbase[0] += it.n_max;
                ++items;
            }
        }
      }
    } else {
        // ------------------------------------------------------------------ softmax / rescale / epilogue
        asm volatile("setmaxnreg.inc.sync.aligned.u32 224;");
        const int t = warp >> 2;       // query tile of this warp group
        const int quarter = warp & 3;  // TMEM lane quarter this warp may access
        const int row = quarter * 32 + lane;
        const int wg_tid = threadIdx.x & 127;  // index inside the warp group of this tile
        const uint32_t lane_base = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
        const uint32_t col_s = kColS + t * kBN, col_o = kColO + t * D;
        const float sl2 = p.scale_log2;
        int its = 0;  // tile iterations done so far (barrier phases run across items)
        uint32_t wg_phase = 0;
        // the four warps of this tile meet on an mbarrier: unlike bar.sync, the wait is bounded
        auto wg_sync = [&]() -> bool {
            __syncwarp();
            if (lane == 0) mbar_arrive(&wg_bar[t]);
            const bool ok = warp_wait(&wg_bar[t], wg_phase);
            wg_phase ^= 1;
            return ok;
        };

        for (int r = 0; !failed; ++r) {
            const int i = item_of_round(r);
            if (i >= num_items) break;
            const ItemInfo it = decode(i);
            const int q0 = it.q0[t];
            const int qi = q0 + row;
            const int nt = it.n_tiles[t];
            __nv_bfloat16* orow = p.out + ((size_t)(it.b * p.Hq + it.h[t]) * p.Sq + qi) * D;
            if (nt == 0) {  // no visible key for any row of this tile (or the tile lies beyond Sq)
                if (qi < p.Sq) {
#pragma unroll
                    for (int c = 0; c < D / 8; ++c) reinterpret_cast<uint4*>(orow)[c] = make_uint4(0, 0, 0, 0);
                }
                continue;
            }
            float m_run = -INFINITY;  // running maximum of the raw scores (reference of the exponentials)
            float l_run = 0.f;
            const int row_limit = causal ? qi + causal_off : 0x7fffffff;  // last visible key of this row
            for (int j = 0; j < nt; ++j, ++its) {
                // S_t(j) is complete, and so is every MMA issued before it: O_t holds all earlier P V
                // products and P_t(j-1) has been consumed.
                if (!warp_wait(&s_full[t], its & 1)) { failed = true; break; }
                tc_fence_after_sync();
                float s[kBN];
#pragma unroll
                for (int c = 0; c < kBN / 32; ++c) {
                    uint32_t r[32];
                    tmem_ld_x32(lane_base + col_s + c * 32, r);
#pragma unroll
                    for (int i = 0; i < 32; ++i) s[c * 32 + i] = __uint_as_float(r[i]);
                }
                tmem_ld_wait();

                const int j0 = j * kBN;
                const bool need_mask = (j0 + kBN > it.kvlen) || (causal && (j0 + kBN - 1 > q0 + causal_off));
                if (need_mask) {
                    const int lim = min(it.kvlen - 1, row_limit) - j0;  // last visible column of this tile
#pragma unroll
                    for (int i = 0; i < kBN; ++i) s[i] = (i <= lim) ? s[i] : -INFINITY;
                }
                const float2 sl2v = make_float2(sl2, sl2);
                // Fast path (full tiles once every row has a finite reference): exponentials against the
                // current reference in the same pass that finds the tile maximum.  Valid as long as no row's
                // maximum exceeds its reference by more than the threshold, which is what the lazy rescale
                // tolerates anyway; otherwise the tile is redone below with a new reference.
                bool done = false;
                if (!need_mask && __all_sync(0xffffffffu, m_run != -INFINITY)) {
                    const float2 neg_m = make_float2(-m_run * sl2, -m_run * sl2);
                    float2 lsum[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
                    float mx[4] = {s[0], s[1], s[2], s[3]};
#pragma unroll
                    for (int half = 0; half < 2; ++half) {
                        uint32_t packed[32];
#pragma unroll
                        for (int i = 0; i < 32; ++i) {
                            const float s0 = s[half * 64 + 2 * i], s1 = s[half * 64 + 2 * i + 1];
                            mx[i & 3] = max3(mx[i & 3], s0, s1);
                            const float2 x = ffma2(make_float2(s0, s1), sl2v, neg_m);
                            const float2 pr = make_float2(ex2(x.x), ex2(x.y));
                            lsum[i & 1] = fadd2(lsum[i & 1], pr);
                            packed[i] = pack_bf16(pr.x, pr.y);
                        }
                        tmem_st_x32(lane_base + col_s + half * 32, packed);
                    }
                    const float m_tile = max3(fmaxf(mx[0], mx[1]), mx[2], mx[3]);
                    if (!__any_sync(0xffffffffu, (m_tile - m_run) * sl2 > kRescaleThreshold)) {
                        l_run += (lsum[0].x + lsum[0].y) + (lsum[1].x + lsum[1].y);
                        done = true;
                    }
                }
                if (!done) {
                    // row maximum: four independent chains of 3-input maxima
                    float mx[4] = {s[0], s[1], s[2], s[3]};
    #pragma unroll
                    for (int i = 4; i + 7 < kBN; i += 8) {
                        mx[0] = max3(mx[0], s[i], s[i + 1]);
                        mx[1] = max3(mx[1], s[i + 2], s[i + 3]);
                        mx[2] = max3(mx[2], s[i + 4], s[i + 5]);
                        mx[3] = max3(mx[3], s[i + 6], s[i + 7]);
                    }
                    mx[0] = max3(mx[0], s[kBN - 4], s[kBN - 3]);
                    mx[1] = max3(mx[1], s[kBN - 2], s[kBN - 1]);
                    const float m_tile = max3(fmaxf(mx[0], mx[1]), mx[2], mx[3]);

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
                    if (j > 0 && __any_sync(0xffffffffu, alpha != 1.f)) {
                        // rare after the first tiles: small chunks, not unrolled, to keep register pressure low
    #pragma unroll 1
                        for (int c = 0; c < D / 16; ++c) {
                            uint32_t r[16];
                            tmem_ld_x16(lane_base + col_o + c * 16, r);
                            tmem_ld_wait();
    #pragma unroll
                            for (int i = 0; i < 16; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * alpha);
                            tmem_st_x16(lane_base + col_o + c * 16, r);
                        }
                    }
                    const float m_ref = (m_run == -INFINITY) ? 0.f : m_run;
                    const float2 neg_m = make_float2(-m_ref * sl2, -m_ref * sl2);
                    float2 lsum[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
                    // P = 2^(s * sl2 - m * sl2) as packed bf16 pairs, written over the first 64 columns of S_t
                    // in two halves.  In masked tiles the probability of a masked key is forced to exactly 0
                    // (that also covers sl2 == 0, where -inf * 0 would be NaN); full tiles skip the selects.
                    auto exp_and_store = [&](auto masked_tag) {
                        constexpr bool kMasked = decltype(masked_tag)::value;
    #pragma unroll
                        for (int half = 0; half < 2; ++half) {
                            uint32_t packed[32];
    #pragma unroll
                            for (int i = 0; i < 32; ++i) {
                                const float s0 = s[half * 64 + 2 * i], s1 = s[half * 64 + 2 * i + 1];
                                const float2 x = ffma2(make_float2(s0, s1), sl2v, neg_m);
                                float2 pr = make_float2(ex2(x.x), ex2(x.y));
                                if constexpr (kMasked) {
                                    pr.x = (s0 == -INFINITY) ? 0.f : pr.x;
                                    pr.y = (s1 == -INFINITY) ? 0.f : pr.y;
                                }
                                lsum[i & 1] = fadd2(lsum[i & 1], pr);
                                packed[i] = pack_bf16(pr.x, pr.y);
                            }
                            tmem_st_x32(lane_base + col_s + half * 32, packed);
                        }
                    };
                    if (need_mask) exp_and_store(std::true_type{});
                    else exp_and_store(std::false_type{});
                    const float l_tile = (lsum[0].x + lsum[0].y) + (lsum[1].x + lsum[1].y);
                    l_run = l_run * alpha + l_tile;
                }
                tmem_st_wait();
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(&p_ready[t]);  // one arrival per warp
            }
            if (failed) break;
            if (!warp_wait(&pv_done[t], (its - 1) & 1)) { failed = true; break; }
            tc_fence_after_sync();
            // O_t -> registers, then hand O_t back to the MMA warp before the stores go out
            uint32_t o[D];
#pragma unroll
            for (int c = 0; c < D / 32; ++c) {
                uint32_t rr[32];
                tmem_ld_x32(lane_base + col_o + c * 32, rr);
#pragma unroll
                for (int k = 0; k < 32; ++k) o[c * 32 + k] = rr[k];
            }
            tmem_ld_wait();
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&o_free[t]);
            // O / l as bf16 through a 128-byte-swizzled staging buffer and one TMA store per 64 columns
            // (rows beyond Sq are clipped by the TMA unit).  The store drains while the next item starts.
            {
                const float inv = l_run > 0.f ? 1.f / l_run : 0.f;  // no visible key: zeros
                uint8_t* stage_out = smem + L::kOutOff + t * L::kChunkBytes;
#pragma unroll
                for (int cb = 0; cb < D / 64; ++cb) {
                    if (wg_tid == 0) tma_store_wait_read<0>();  // the previous store has read the buffer
                    if (!wg_sync()) { failed = true; break; }
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        uint32_t w[4];
#pragma unroll
                        for (int k = 0; k < 4; ++k)
                            w[k] = pack_bf16(__uint_as_float(o[cb * 64 + c * 8 + 2 * k]) * inv,
                                             __uint_as_float(o[cb * 64 + c * 8 + 2 * k + 1]) * inv);
                        *reinterpret_cast<uint4*>(stage_out + row * 128 + ((c ^ (row & 7)) << 4)) =
                            make_uint4(w[0], w[1], w[2], w[3]);
                    }
                    fence_proxy_async_smem();
                    if (!wg_sync()) { failed = true; break; }
                    if (wg_tid == 0) {
                        tma_store_3d(&tmap_o, stage_out, cb * 64, q0, it.b * p.Hq + it.h[t]);
                        tma_store_commit();
                    }
                }
            }
        }
        if (wg_tid == 0) tma_store_wait_all<0>();  // every output tile has left shared memory and is written
    }

    if (failed) {
        atomicExch(p.status, 1);
        for (int i = 0; i < 2000; ++i) __nanosleep(1000);  // let copies and MMAs in flight land
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 9) {
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
    CUtensorMap to;
    {
        const uint64_t dims[3] = {(uint64_t)D, (uint64_t)Sq, (uint64_t)B * Hq};
        const uint64_t strides[2] = {(uint64_t)D * 2, (uint64_t)Sq * D * 2};
        if (!encode_tmap_bf16_sw128(&to, out, 3, dims, strides, box)) return FORGE_ERR_CUDA;
    }
    AttnParams p;
    p.out = static_cast<__nv_bfloat16*>(out);
    p.lens = lens;
    p.B = B; p.Hq = Hq; p.Hkv = Hkv; p.Sq = Sq; p.Skv = Skv;
    p.mask_kind = mask_kind;
    p.scale_log2 = scale * 1.4426950408889634f;
    p.status = device_status_word();
    if (!p.status) return FORGE_ERR_CUDA;
    auto kernel = attn_bf16_kernel<D>;
    FORGE_SET_SMEM_ONCE(kernel, L::kAlloc);
    const int sms = sm_count();
    if (sms <= 0) return FORGE_ERR_CUDA;
    const int q_tiles = (Sq + kBM - 1) / kBM;
    const bool head_pairs = ((Hq / Hkv) % 2 == 0) || L::kKVStages >= 4;  // same rule as in the kernel
    const long long items = head_pairs ? (long long)((Hq + 1) / 2) * B * q_tiles
                                       : (long long)Hq * B * ((q_tiles + 1) / 2);
    const int grid = items < sms ? (int)items : sms;
    kernel<<<grid, kThreads, L::kAlloc, s>>>(tq, tk, tv, to, p);
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
    if ((long long)Hq * B * ((Sq + 255) / 256) > 2147483647LL) return FORGE_ERR_UNSUPPORTED;
    if (!(scale >= 0.f)) return FORGE_ERR_UNSUPPORTED;  // the running maximum is taken on unscaled scores
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    return D == 64 ? launch_attn<64>(q, k, v, out, B, Hq, Hkv, Sq, Skv, mask_kind, lens, scale, s)
                   : launch_attn<128>(q, k, v, out, B, Hq, Hkv, Sq, Skv, mask_kind, lens, scale, s);
}
