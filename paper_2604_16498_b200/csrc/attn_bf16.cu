// Fused attention, 16-bit in / fp32 accumulate / 16-bit out (Eq. 8 / Eq. 9): scores, mask, online
// softmax and the product with V in one kernel; S and P never reach global memory.  The element type
// is bf16 or fp16 (a template parameter: the MMA operand format and the two conversions differ).
//
// One work item = two 128-row query tiles (see the item decoding below).  Every 128-key tile of S is
// computed, normalised and multiplied with V in two 64-key halves with their own barriers, so each
// query tile has two independent half-step streams and the CTA has four: while a softmax thread works
// on one half, the tensor core multiplies the other half's P with V and produces that half's next S.
// Warp roles:
//   warps 0-3 : softmax / rescale / epilogue of tile 0; thread = one query row (TMEM lane), so row
//   warps 4-7 : the same for tile 1                    maxima and sums need no cross-thread reduction
//   warp 8    : TMA producer: Q tiles, then K and V tiles (64 keys, one per half-step) through rings;
//               it sleeps between barrier polls (a spinning thread takes issue slots from the softmax
//               warp of its scheduler: 1.2 % of the kernel)
//   warp 9    : tcgen05.mma issuer of tile 0 (one elected lane), owns the TMEM allocation
//   warp 10   : tcgen05.mma issuer of tile 1
//   warp 11 only completes the third warpgroup, which hands registers to the other two
//   (setmaxnreg: 208 per softmax thread, 88 for the rest; 256*208 + 128*88 = 384*168 as launched).
// Tensor memory (512 columns): S_t at t*128 (half h at +64h, 64 fp32 columns each), O_0 at 256,
// O_1 at 256 + D.  P (bf16, two per column) of half h is written over the first 32 columns of that
// half of S and is the A operand of the P V product straight from tensor memory.  A tile's issuer
// thread issues, per half-step g (key tile g/2, half g%2):  O += P(g) V(g), then S(g+2) = Q K(g+2)^T.
// MMAs of one thread execute in issue order, so P(g) is read before S(g+2) overwrites it, and the
// barrier that announces S(g+2) also covers the completion of the P V products up to g.
// O is rescaled in TMEM only when a row's maximum grows by more than 2^8 (the stale maximum is
// kept otherwise; the final division by l uses the same reference, so the result is unchanged).
// Q and K are K-major operands, V [keys, D] is the MN-major B operand of P V.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <type_traits>

#include "attn_wide.cuh"
#include "forge_common.cuh"
#include "sm100_ptx.cuh"
#include "tmap.cuh"

namespace forge {
namespace {

using namespace ptx;

constexpr int kBM = 128;          // query rows per tile
constexpr int kTilesPerCta = 2;
constexpr int kBN = 128;          // keys per tile of S (two half-steps)
constexpr int kHalf = 64;         // keys per half-step and per K/V tile in shared memory
constexpr int kThreads = 384;
constexpr int kTmemCols = 512;
constexpr int kColS = 0;          // S_t at t * 128
constexpr int kColO = 256;        // O_t at 256 + t * D
constexpr float kRescaleThreshold = 8.0f;  // log2 units
#ifndef FORGE_ATTN_FMA_EXP_PAIRS
#define FORGE_ATTN_FMA_EXP_PAIRS 2
#endif
// of the 32 score pairs of a half-step, how many take their exponentials on the FMA pipe (unmasked steps)
constexpr int kFmaExpPairs = FORGE_ATTN_FMA_EXP_PAIRS;

template <int D>
struct AttnSmem {
    static constexpr int kChunkBytes = 128 * 128;              // Q: 128 rows x 64 bf16 (one swizzle span wide)
    static constexpr int kTileBytes = (D / 64) * kChunkBytes;  // a Q tile
    static constexpr int kKVChunkBytes = kHalf * 128;          // K, V: 64 keys x 64 bf16
    static constexpr int kKVTileBytes = (D / 64) * kKVChunkBytes;
    static constexpr int kKVStages = (D == 64) ? 8 : 3;
    static constexpr int kQOff = 0;
    static constexpr int kKOff = kQOff + kTilesPerCta * kTileBytes;
    static constexpr int kVOff = kKOff + kKVStages * kKVTileBytes;
    // output staging: 32 rows x 64 bf16 per softmax warp and 64-column block of D
    static constexpr int kOutOff = kVOff + kKVStages * kKVTileBytes;
    static constexpr int kOutWarpBytes = (D / 64) * 4096;
    static constexpr int kBarOff = kOutOff + 8 * kOutWarpBytes;
    // q_full[2], q_empty[2], k/v full+empty per stage, s_full[4], p_ready[4], pv_done[4], o_free[2]
    static constexpr int kNumBars = 4 + 4 * kKVStages + 14;
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

// 2^x for two values on the FMA and integer pipes instead of the special-function unit (which is the
// narrowest pipe of the softmax): x = n + f with n = round(x), f in [-0.5, 0.5]; 2^f by a cubic with a
// relative error of 7.6e-5 (far below the bf16 rounding of P); n is added to the exponent field.
// Inputs below -125 give 2^-125 rather than 0, so this is used only where no score is masked.
__device__ __forceinline__ float2 ex2_fma2(float2 x) {
    const float kMagic = 12582912.f;  // 1.5 * 2^23: adding it leaves round(x) in the low mantissa bits
    x.x = fmaxf(x.x, -125.f);
    x.y = fmaxf(x.y, -125.f);
    const float2 t = fadd2(x, make_float2(kMagic, kMagic));
    const float2 n = fadd2(t, make_float2(-kMagic, -kMagic));
    const float2 f = ffma2(n, make_float2(-1.f, -1.f), x);
    float2 q = ffma2(f, make_float2(0.05520550534f, 0.05520550534f), make_float2(0.2426139712f, 0.2426139712f));
    q = ffma2(q, f, make_float2(0.6932547688f, 0.6932547688f));
    q = ffma2(q, f, make_float2(0.9999276996f, 0.9999276996f));
    return make_float2(__int_as_float(__float_as_int(q.x) + (__float_as_int(t.x) << 23)),
                       __int_as_float(__float_as_int(q.y) + (__float_as_int(t.y) << 23)));
}

// two fp32 values rounded to nearest even and packed as bf16 (F16 = false) or fp16 (F16 = true)
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

// Division by a divisor fixed at launch: floor(n / d) = high 64 bits of n * ceil(2^64 / d) for 0 <= n < 2^32.
struct FastDiv {
    unsigned long long m;  // ceil(2^64 / d); unused for d == 1
    int d;
};
inline FastDiv make_fastdiv(int d) {
    FastDiv f;
    f.d = d;
    f.m = d > 1 ? ~0ull / (unsigned long long)d + 1ull : 0ull;
    return f;
}
__device__ __forceinline__ int fast_div(int n, const FastDiv& f) {
    return f.d == 1 ? n : (int)__umul64hi((unsigned long long)(unsigned)n, f.m);
}

struct AttnParams {
    uint16_t* out;  // bf16 or fp16 elements
    long long o_sb, o_sh, o_ss;  // element strides of out between batch entries, heads and rows
    const int32_t* lens;
    const float* bias;  // additive bias on the scaled scores [B, bias_heads, Sq, Skv], or nullptr
    int bias_heads;     // 1 (shared by all heads) or Hq
    float inv_scale;    // 1 / scale: the bias is added to the unscaled scores as bias / scale
    int B, Hq, Hkv, Sq, Skv;
    int head_dim;  // elements per row in memory (<= the kernel's D; the TMA unit zero-fills the difference)
    int mask_kind;
    float scale_log2;  // > 0 (a zero scale is passed as the smallest normal number: every product flushes to 0)
    FastDiv div_heads;  // by the number of items per query step
    FastDiv div_inner;  // by the head pairs (or heads) per batch entry
    FastDiv div_group;  // by the query heads per KV head
    int* status;
};

// What one CTA needs to know about a work item (a pair of query tiles).
struct ItemInfo {
    int b, kvlen;
    int kvh[kTilesPerCta];      // KV head of each tile (equal unless the tiles read separate K/V streams)
    int q0[kTilesPerCta];       // first query row of each of the two tiles
    int h[kTilesPerCta];        // query head of each tile
    int nh[kTilesPerCta];       // 64-key half-steps visible to at least one row of each query tile (0: no work)
    int n_max;                  // the larger of the two
};

// element t of a two-element array without dynamic indexing (keeps the array in registers)
__device__ __forceinline__ int pick(const int (&a)[kTilesPerCta], int t) { return t ? a[1] : a[0]; }

template <int D, bool F16, bool BIAS>
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
    uint64_t* q_full = bars;                 // [2] per query tile
    uint64_t* q_empty = bars + 2;            // [2]
    uint64_t* k_full = bars + 4;
    uint64_t* k_empty = k_full + kKVStages;
    uint64_t* v_full = k_empty + kKVStages;
    uint64_t* v_empty = v_full + kKVStages;
    uint64_t* s_full = v_empty + kKVStages;  // [4] query tile t, half h at t * 2 + h
    uint64_t* p_ready = s_full + 4;          // [4]
    uint64_t* pv_done = p_ready + 4;         // [4] one completion per P V product of that tile and half
    uint64_t* o_free = pv_done + 4;          // [2] per query tile
    uint32_t* tmem_base_slot = reinterpret_cast<uint32_t*>(o_free + 2);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // The two tiles of an item: with an even number of query heads per KV head, the same 128 query rows of
    // two heads that share K and V (equal causal lengths, so neither tile waits for the other); otherwise
    // two consecutive 128-row tiles of one head.
    const int G = p.Hq / p.Hkv;
    const bool pair_heads = (G % 2) == 0;
    // With an odd group size and D = 64 (where shared memory has room for it) the two tiles are still two
    // heads on the same query rows, each with its own K/V stream through half of the stage ring.
    const bool two_streams = !pair_heads && kKVStages >= 8;
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
        const int round_q = fast_div(i, p.div_heads);
        const int qstep = rows_of_items - 1 - round_q;  // longest (causal) first
        const int hb = i - round_q * heads;
        it.b = fast_div(hb, p.div_inner);
        if (pair_heads || two_streams) {
            const int hp = hb - it.b * head_pairs;
            it.h[0] = 2 * hp;
            it.h[1] = min(2 * hp + 1, p.Hq - 1);
            it.q0[0] = it.q0[1] = qstep * kBM;
            if (2 * hp + 1 >= p.Hq) it.q0[1] = num_q_tiles * kBM;  // odd head count: no second tile
        } else {
            it.h[0] = it.h[1] = hb - it.b * p.Hq;
            it.q0[0] = 2 * qstep * kBM; it.q0[1] = (2 * qstep + 1) * kBM;
        }
        it.kvh[0] = fast_div(it.h[0], p.div_group);
        it.kvh[1] = fast_div(it.h[1], p.div_group);
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
            it.nh[t] = (kv_end + kHalf - 1) / kHalf;
            it.n_max = max(it.n_max, it.nh[t]);
        }
        return it;
    };

    if (threadIdx.x == 0) {
        for (int t = 0; t < 2; ++t) { mbar_init(&q_full[t], 1); mbar_init(&q_empty[t], 1); }
        // a shared K/V stage is released by both tiles' issuer threads, a private one by its own
        const uint32_t releases = two_streams ? 1 : 2;
        for (int i = 0; i < kKVStages; ++i) {
            mbar_init(&k_full[i], 1); mbar_init(&k_empty[i], releases);
            mbar_init(&v_full[i], 1); mbar_init(&v_empty[i], releases);
        }
        for (int i = 0; i < 4; ++i) { mbar_init(&s_full[i], 1); mbar_init(&p_ready[i], 4); mbar_init(&pv_done[i], 1); }
        for (int t = 0; t < 2; ++t) mbar_init(&o_free[t], 4);
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
    // set-up done: the next kernel may move in as SMs free up; nothing global is touched before the
    // previous kernel has completed
    pdl_launch_dependents();
    pdl_wait();

    if (warp >= 8) {
      asm volatile("setmaxnreg.dec.sync.aligned.u32 88;");
      if (warp == 8) {
        // ------------------------------------------------------------------ TMA producer
        if (elect_one()) {
            int kvn[2] = {0, 0};     // KV tiles loaded so far per stream (ring position), across items
            int q_loads[2] = {0, 0}; // Q tiles loaded so far per query tile
            for (int r = 0; !failed; ++r) {
                const int i = item_of_round(r);
                if (i >= num_items) break;
                const ItemInfo it = decode(i);
                if (it.n_max == 0) continue;
#pragma unroll
                for (int t = 0; t < kTilesPerCta; ++t) {
                    if (it.nh[t] == 0) continue;
                    // the tile's last S = Q K^T of its previous item has completed: Q may be replaced
                    if (!mbar_wait_relaxed(&q_empty[t], (q_loads[t] & 1) ^ 1)) { failed = true; break; }
                    ++q_loads[t];
                    mbar_expect_tx(&q_full[t], L::kTileBytes);
#pragma unroll
                    for (int c = 0; c < D / 64; ++c)  // rows beyond Sq are zero-filled by the TMA unit
                        tma_load_4d(sQ + t * L::kTileBytes + c * L::kChunkBytes, &tmap_q, &q_full[t], c * 64,
                                    it.q0[t], it.h[t], it.b);
                }
                // The next item's Q tiles are asked into L2 now, a whole item ahead: Q can only be copied to
                // shared memory once this item's last scores are done, and a copy that then has to come from
                // HBM leaves the tensor core idle for a microsecond or two at every item boundary.
                {
                    const int i_next = item_of_round(r + 1);
                    if (i_next < num_items) {
                        const ItemInfo nx = decode(i_next);
#pragma unroll
                        for (int t = 0; t < kTilesPerCta; ++t) {
                            if (nx.nh[t] == 0) continue;
#pragma unroll
                            for (int c = 0; c < D / 64; ++c) tma_prefetch_l2_4d(&tmap_q, c * 64, nx.q0[t], nx.h[t], nx.b);
                        }
                    }
                }
                for (int j = 0; j < it.n_max && !failed; ++j) {
#pragma unroll
                    for (int u = 0; u < 2; ++u) {
                        if (u == 1 && !two_streams) continue;
                        if (two_streams && j >= it.nh[u]) continue;
                        const int g = kvn[u]++, st = kv_slot(u, g);
                        const uint32_t ph = kv_phase(g);
                        const int kvh = it.kvh[u];
                        if (!mbar_wait_relaxed(&k_empty[st], ph ^ 1)) { failed = true; break; }
                        mbar_expect_tx(&k_full[st], L::kKVTileBytes);
#pragma unroll
                        for (int c = 0; c < D / 64; ++c)
                            tma_load_4d(sK + st * L::kKVTileBytes + c * L::kKVChunkBytes, &tmap_k, &k_full[st], c * 64,
                                        j * kHalf, kvh, it.b);
                        if (!mbar_wait_relaxed(&v_empty[st], ph ^ 1)) { failed = true; break; }
                        mbar_expect_tx(&v_full[st], L::kKVTileBytes);
#pragma unroll
                        for (int c = 0; c < D / 64; ++c)
                            tma_load_4d(sV + st * L::kKVTileBytes + c * L::kKVChunkBytes, &tmap_v, &v_full[st], c * 64,
                                        j * kHalf, kvh, it.b);
                    }
                }
            }
        }
      } else if (warp <= 10) {
        // ------------------------------------------------------------------ MMA issuer of query tile t
        if (elect_one()) {
            const int t = warp - 9;
            const int u = two_streams ? t : 0;
            constexpr uint32_t idesc_s = F16 ? make_idesc_f16(kBM, kHalf, false, false) : make_idesc_bf16(kBM, kHalf, false, false);
            constexpr uint32_t idesc_o = F16 ? make_idesc_f16(kBM, D, false, true) : make_idesc_bf16(kBM, D, false, true);
            const uint32_t q_addr = smem_u32(sQ) + t * L::kTileBytes, k_addr = smem_u32(sK), v_addr = smem_u32(sV);
            const uint32_t s_tmem = tmem_base + kColS + t * kBN, o_tmem = tmem_base + kColO + t * D;
            // descriptors differ only in the start-address field: build one per operand, then add
            // (byte offset >> 4) for each step (the field cannot overflow below 256 KB)
            const uint64_t qd = make_smem_desc(q_addr, 16, 1024);
            int kvbase = 0;      // ring position of the item's first KV tile in this tile's stream
            int q_uses = 0;      // items in which this tile had work (phases of q_full, o_free)
            int steps0 = 0, steps1 = 0;  // half-steps issued so far per half (phases of p_ready)

            ItemInfo it;
            int i_cur = item_of_round(0);
            if (i_cur < num_items) it = decode(i_cur);
            for (int r = 0; !failed && i_cur < num_items; ++r) {
                const int i_next = item_of_round(r + 1);
                ItemInfo it_next;
                if (it.n_max == 0) {
                    if (i_next < num_items) it_next = decode(i_next);
                    it = it_next; i_cur = i_next;
                    continue;
                }
                const int nh = pick(it.nh, t);

                // A barrier poll costs a few hundred cycles even on a completed phase, so the operands of a step
                // (V(g) for the product, K(g + 2) for the next scores) are waited for before the probabilities,
                // while this thread has nothing to issue; once P(g) arrives the MMAs go out back to back.
                auto wait_k = [&](int g) -> bool {
                    const int pos = kvbase + g;
                    return mbar_wait(&k_full[kv_slot(u, pos)], kv_phase(pos));
                };
                auto wait_v = [&](int g) -> bool {
                    const int pos = kvbase + g;
                    return mbar_wait(&v_full[kv_slot(u, pos)], kv_phase(pos));
                };
                // S(g) = Q K(g)^T into half g % 2 of S_t (K(g) has landed)
                auto issue_qk = [&](int g) -> bool {
                    const int hh = g & 1, pos = kvbase + g, st = kv_slot(u, pos);
                    tc_fence_after_sync();
                    const uint64_t kd = make_smem_desc(k_addr + st * L::kKVTileBytes, 16, 1024);
#pragma unroll
                    for (int kk = 0; kk < D / 16; ++kk) {
                        const uint32_t qoff = ((kk / 4) * L::kChunkBytes + (kk % 4) * 32) >> 4;
                        const uint32_t koff = ((kk / 4) * L::kKVChunkBytes + (kk % 4) * 32) >> 4;
                        mma_ss(s_tmem + hh * kHalf, qd + qoff, kd + koff, idesc_s, kk != 0);
                    }
                    mma_commit(&s_full[t * 2 + hh]);
                    mma_commit(&k_empty[st]);                  // this tile is done with the K tile
                    if (g == nh - 1) mma_commit(&q_empty[t]);  // and, after the item's last S, with Q
                    return true;
                };
                // O_t += P(g) V(g) with P read from tensor memory (V(g) has landed)
                auto issue_pv = [&](int g) -> bool {
                    const int hh = g & 1, pos = kvbase + g, st = kv_slot(u, pos);
                    if (!mbar_wait(&p_ready[t * 2 + hh], (hh ? steps1 : steps0) & 1)) return false;
                    if (hh) ++steps1; else ++steps0;
                    // the first product of an item overwrites O_t: the previous item's epilogue must have read it
                    if (g == 0 && !mbar_wait(&o_free[t], (q_uses & 1) ^ 1)) return false;
                    tc_fence_after_sync();
                    // P: 16 keys = 8 columns of packed bf16 pairs.  V: MN-major, 16 keys = two 1024-byte groups
                    // (2048 bytes per step); the 64-wide chunks of D are 8 KB apart.
                    const uint64_t vd = make_smem_desc(v_addr + st * L::kKVTileBytes, L::kKVChunkBytes, 1024);
                    const uint32_t p_tmem = s_tmem + hh * kHalf;
                    if (g == 0) mma_ts(o_tmem, p_tmem, vd, idesc_o, 0u);
                    else mma_ts(o_tmem, p_tmem, vd, idesc_o, 1u);
#pragma unroll
                    for (int kk = 1; kk < kHalf / 16; ++kk) mma_ts(o_tmem, p_tmem + kk * 8, vd + kk * (2048 >> 4), idesc_o, 1u);
                    mma_commit(&pv_done[t * 2 + hh]);
                    mma_commit(&v_empty[st]);
                    return true;
                };

                if (nh > 0) {
                    if (!mbar_wait(&q_full[t], q_uses & 1)) { failed = true; break; }
                    if (!wait_k(0) || !issue_qk(0)) { failed = true; break; }
                    if (nh > 1 && (!wait_k(1) || !issue_qk(1))) { failed = true; break; }
                }
                // the next item's coordinates, worked out while the softmax warps are busy with the first S
                if (i_next < num_items) it_next = decode(i_next);
                if (nh > 0) {
                    for (int g = 0; g < nh; ++g) {
                        if (!wait_v(g) || (g + 2 < nh && !wait_k(g + 2))) { failed = true; break; }
                        if (!issue_pv(g)) { failed = true; break; }
                        if (g + 2 < nh && !issue_qk(g + 2)) { failed = true; break; }
                    }
                    if (failed) break;
                    ++q_uses;
                }
                if (two_streams) {
                    kvbase += nh;
                } else {
                    // K/V tiles that only the other query tile reads: release them once they have landed
                    for (int j = nh; j < it.n_max; ++j) {
                        const int pos = kvbase + j, st = kv_slot(0, pos);
                        if (!mbar_wait(&k_full[st], kv_phase(pos))) { failed = true; break; }
                        mbar_arrive(&k_empty[st]);
                        if (!mbar_wait(&v_full[st], kv_phase(pos))) { failed = true; break; }
                        mbar_arrive(&v_empty[st]);
                    }
                    kvbase += it.n_max;
                }
                it = it_next; i_cur = i_next;
            }
        }
      }
    } else {
        // ------------------------------------------------------------------ softmax / rescale / epilogue
        asm volatile("setmaxnreg.inc.sync.aligned.u32 208;");
        const int t = warp >> 2;       // query tile of this warp group
        const int quarter = warp & 3;  // TMEM lane quarter this warp may access
        const int row = quarter * 32 + lane;
        const uint32_t lane_base = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
        const uint32_t col_s = kColS + t * kBN, col_o = kColO + t * D;
        const float sl2 = p.scale_log2;
        const float2 sl2v = make_float2(sl2, sl2);
        uint8_t* stage_out = smem + L::kOutOff + warp * L::kOutWarpBytes;  // this warp's 32 rows x 128 bytes per block
        int steps0 = 0, steps1 = 0;  // half-steps done so far per half (barrier phases run across items)
        const int u = two_streams ? t : 0;  // K/V stream of this tile
        int kvbase = 0;              // ring position of the item's first KV tile in that stream
        const bool padding = (p.mask_kind & FORGE_MASK_PADDING) != 0;

        ItemInfo it;
        int i_cur = item_of_round(0);
        if (i_cur < num_items) it = decode(i_cur);
        for (int r = 0; !failed && i_cur < num_items; ++r) {
            const int i_next = item_of_round(r + 1);
            ItemInfo it_next;
            const int q0 = pick(it.q0, t);
            const int qi = q0 + row;
            const int nh = pick(it.nh, t);
            const int head = pick(it.h, t);
            if (nh == 0) {  // no visible key for any row of this tile (or the tile lies beyond Sq)
                if (qi < p.Sq) {
                    uint16_t* orow = p.out + it.b * p.o_sb + head * p.o_sh + qi * p.o_ss;
                    for (int c = 0; c < p.head_dim / 8; ++c) reinterpret_cast<uint4*>(orow)[c] = make_uint4(0, 0, 0, 0);
                }
                if (i_next < num_items) it_next = decode(i_next);
                if (!two_streams) kvbase += it.n_max;  // the tiles the other query tile of the item reads
                it = it_next; i_cur = i_next;
                continue;
            }
            float m_run = -INFINITY;  // running maximum of the raw scores (reference of the exponentials)
            float l_run = 0.f;
            // last visible key of this row
            const int row_limit = min(it.kvlen - 1, causal ? qi + causal_off : 0x7fffffff);
#pragma unroll 1
            for (int g = 0; g < nh; ++g) {
                const int hh = g & 1;
                const uint32_t col_h = col_s + hh * kHalf;
                // S(g) is complete, and so is every MMA this tile's issuer issued before it: O_t holds the
                // P V products up to g - 2 and P(g - 2) has been consumed.
                if (!warp_wait(&s_full[t * 2 + hh], (hh ? steps1 : steps0) & 1)) { failed = true; break; }
                if (hh) ++steps1; else ++steps0;
                tc_fence_after_sync();
                float s[kHalf];
#pragma unroll
                for (int c = 0; c < kHalf / 32; ++c) {
                    uint32_t rr[32];
                    tmem_ld_x32(lane_base + col_h + c * 32, rr);
#pragma unroll
                    for (int k = 0; k < 32; ++k) s[c * 32 + k] = __uint_as_float(rr[k]);
                }
                tmem_ld_wait();

                const int key0 = (g >> 1) * kBN + hh * kHalf;
                const bool need_mask = (key0 + kHalf > it.kvlen) || (causal && (key0 + kHalf - 1 > q0 + causal_off)) ||
                                       BIAS;  // a bias may hold -inf: the path that tolerates it
                if constexpr (BIAS) {
                    // Eq. 8's mask node as a tensor: scale * s + bias = scale * (s + bias / scale)
                    const int hb = p.bias_heads == 1 ? 0 : pick(it.h, t);
                    const float* brow = p.bias + (((size_t)it.b * p.bias_heads + hb) * p.Sq + min(qi, p.Sq - 1)) * (size_t)p.Skv + key0;
                    const int nvalid = min(kHalf, p.Skv - key0);  // columns beyond Skv are masked below
                    if ((p.Skv & 3) == 0) {  // rows start on 16-byte boundaries
#pragma unroll
                        for (int c = 0; c < kHalf / 4; ++c) {
                            if (c * 4 < nvalid) {
                                const float4 bv = __ldg(reinterpret_cast<const float4*>(brow) + c);
                                s[4 * c] = fmaf(bv.x, p.inv_scale, s[4 * c]);
                                s[4 * c + 1] = fmaf(bv.y, p.inv_scale, s[4 * c + 1]);
                                s[4 * c + 2] = fmaf(bv.z, p.inv_scale, s[4 * c + 2]);
                                s[4 * c + 3] = fmaf(bv.w, p.inv_scale, s[4 * c + 3]);
                            }
                        }
                    } else {
#pragma unroll
                        for (int k = 0; k < kHalf; ++k)
                            if (k < nvalid) s[k] = fmaf(__ldg(brow + k), p.inv_scale, s[k]);
                    }
                }
                bool stored = false;
                if (need_mask) {
                    const int lim = row_limit - key0;  // last visible column of this half
                    if (__all_sync(0xffffffffu, lim < 0)) {
                        // nothing visible for any row of this warp: P = 0
                        uint32_t zeros[32];
#pragma unroll
                        for (int k = 0; k < 32; ++k) zeros[k] = 0u;
                        tmem_st_x32(lane_base + col_h, zeros);
                        stored = true;
                    } else {
                        // a masked score of -inf gives a probability of exactly 0 below (the scale is > 0)
#pragma unroll
                        for (int k = 0; k < kHalf; ++k) s[k] = (k <= lim) ? s[k] : -INFINITY;
                    }
                }
                // Fast path (once every row of the warp has a finite reference): exponentials against the
                // current reference in the same pass that finds the maximum.  Valid as long as no row's
                // maximum exceeds its reference by more than the threshold, which is what the lazy rescale
                // tolerates anyway; otherwise the half is redone below with a new reference.
                if (!stored && __all_sync(0xffffffffu, m_run != -INFINITY)) {
                    auto fast_path = [&](auto fma_tag) {
                        constexpr bool kUseFma = decltype(fma_tag)::value;
                        const float2 neg_m = make_float2(-m_run * sl2, -m_run * sl2);
                        float2 lsum[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
                        float mx[4] = {s[0], s[1], s[2], s[3]};
                        uint32_t packed[32];
#pragma unroll
                        for (int k = 0; k < 32; ++k) {
                            const float s0 = s[2 * k], s1 = s[2 * k + 1];
                            mx[k & 3] = max3(mx[k & 3], s0, s1);
                            const float2 x = ffma2(make_float2(s0, s1), sl2v, neg_m);
                            // evenly spaced pairs go to the FMA pipe, the rest to the special-function unit
                            const bool on_fma = kUseFma && ((k + 1) * kFmaExpPairs / 32) != (k * kFmaExpPairs / 32);
                            const float2 pr = on_fma ? ex2_fma2(x) : make_float2(ex2(x.x), ex2(x.y));
                            lsum[k & 1] = fadd2(lsum[k & 1], pr);
                            packed[k] = pack16<F16>(pr.x, pr.y);
                        }
                        const float m_tile = max3(fmaxf(mx[0], mx[1]), mx[2], mx[3]);
                        if (!__any_sync(0xffffffffu, (m_tile - m_run) * sl2 > kRescaleThreshold)) {
                            tmem_st_x32(lane_base + col_h, packed);
                            l_run += (lsum[0].x + lsum[0].y) + (lsum[1].x + lsum[1].y);
                            stored = true;
                        }
                    };
                    if (need_mask) fast_path(std::false_type{});
                    else fast_path(std::true_type{});
                }
                if (!stored) {
                    // row maximum: four independent chains of 3-input maxima
                    float mx[4] = {s[0], s[1], s[2], s[3]};
#pragma unroll
                    for (int k = 4; k + 7 < kHalf; k += 8) {
                        mx[0] = max3(mx[0], s[k], s[k + 1]);
                        mx[1] = max3(mx[1], s[k + 2], s[k + 3]);
                        mx[2] = max3(mx[2], s[k + 4], s[k + 5]);
                        mx[3] = max3(mx[3], s[k + 6], s[k + 7]);
                    }
                    mx[0] = max3(mx[0], s[kHalf - 4], s[kHalf - 3]);
                    mx[1] = max3(mx[1], s[kHalf - 2], s[kHalf - 1]);
                    const float m_tile = max3(fmaxf(mx[0], mx[1]), mx[2], mx[3]);

                    // Keep the old reference unless this half's maximum exceeds it by more than the
                    // threshold (in log2 units of the scaled scores); then every later exponent is <= 8.
                    float alpha = 1.f;
                    bool grow = (m_tile - m_run) * sl2 > kRescaleThreshold || m_run == -INFINITY;
                    if (m_tile == -INFINITY) grow = false;
                    if (grow) {
                        // first visible keys of this row: nothing accumulated yet, nothing to rescale
                        alpha = (m_run == -INFINITY) ? 1.f : ex2((m_run - m_tile) * sl2);
                        m_run = m_tile;
                    }
                    if (g > 0 && __any_sync(0xffffffffu, alpha != 1.f)) {
                        // O_t must hold every product issued so far and none may be in flight: the product of
                        // half-step g - 1 (the other half's latest) is the only one the barrier above does not cover.
                        if (!warp_wait(&pv_done[t * 2 + (hh ^ 1)], ((hh ? steps0 : steps1) - 1) & 1)) { failed = true; break; }
                        tc_fence_after_sync();
                        // rare after the first steps: small chunks, not unrolled, to keep register pressure low
#pragma unroll 1
                        for (int c = 0; c < D / 16; ++c) {
                            uint32_t rr[16];
                            tmem_ld_x16(lane_base + col_o + c * 16, rr);
                            tmem_ld_wait();
#pragma unroll
                            for (int k = 0; k < 16; ++k) rr[k] = __float_as_uint(__uint_as_float(rr[k]) * alpha);
                            tmem_st_x16(lane_base + col_o + c * 16, rr);
                        }
                    }
                    const float m_ref = (m_run == -INFINITY) ? 0.f : m_run;
                    const float2 neg_m = make_float2(-m_ref * sl2, -m_ref * sl2);
                    float2 lsum[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
                    // P = 2^(s * sl2 - m * sl2) as packed bf16 pairs, written over the first 32 columns of this
                    // half of S_t
                    uint32_t packed[32];
#pragma unroll
                    for (int k = 0; k < 32; ++k) {
                        const float2 x = ffma2(make_float2(s[2 * k], s[2 * k + 1]), sl2v, neg_m);
                        const float2 pr = make_float2(ex2(x.x), ex2(x.y));
                        lsum[k & 1] = fadd2(lsum[k & 1], pr);
                        packed[k] = pack16<F16>(pr.x, pr.y);
                    }
                    tmem_st_x32(lane_base + col_h, packed);
                    const float l_tile = (lsum[0].x + lsum[0].y) + (lsum[1].x + lsum[1].y);
                    l_run = l_run * alpha + l_tile;
                }
                // Rows of the V tile at and beyond lens[b] were copied from the caller's padding, which may hold
                // anything; their probabilities are exactly 0, but 0 x NaN is NaN on the tensor core.  The four
                // warps of the tile zero those rows in shared memory before the product is allowed to start (the
                // issuer needs all four arrivals below).  Rows beyond Skv were zero-filled by the copy itself.
                if (padding && key0 + kHalf > it.kvlen && it.kvlen < p.Skv) {
                    const int pos = kvbase + g, st = kv_slot(u, pos);
                    if (!warp_wait(&v_full[st], kv_phase(pos))) { failed = true; break; }
                    const int first = max(it.kvlen - key0, 0);       // first padded row of this tile
                    const int per_chunk = (kHalf - first) * 8;        // 16-byte pieces to clear per 64-column chunk
                    uint8_t* vt = sV + st * L::kKVTileBytes;
                    for (int i = quarter * 32 + lane; i < (D / 64) * per_chunk; i += 128) {
                        const int c = i / per_chunk, rem = i - c * per_chunk;
                        *reinterpret_cast<uint4*>(vt + c * L::kKVChunkBytes + (first + (rem >> 3)) * 128 + ((rem & 7) << 4)) =
                            make_uint4(0, 0, 0, 0);
                    }
                    fence_proxy_async_smem();  // the tensor core reads what these threads wrote
                }
                tmem_st_wait();
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(&p_ready[t * 2 + hh]);  // one arrival per warp
            }
            if (failed) break;
            // the next item's coordinates, worked out while the last products are still running
            if (i_next < num_items) it_next = decode(i_next);
            // The last product of either half (every S barrier seen covers that half's product before the
            // latest, so each wait is at most one completion behind and the phase parity identifies it).
            if (steps0 > 0 && !warp_wait(&pv_done[t * 2], (steps0 - 1) & 1)) { failed = true; break; }
            if (steps1 > 0 && !warp_wait(&pv_done[t * 2 + 1], (steps1 - 1) & 1)) { failed = true; break; }
            tc_fence_after_sync();
            // O / l as bf16 through this warp's 128-byte-swizzled staging rows (32 rows x 64 columns per
            // block of D) and one TMA store per block; rows beyond Sq are clipped by the TMA unit.  A short
            // rolled loop: the code runs once per item, so its footprint matters more than its issue count.
            {
                const float inv = l_run > 0.f ? 1.f / l_run : 0.f;  // no visible key: zeros
                if (lane == 0) tma_store_wait_read<0>();  // the previous item's stores have read the staging rows
                __syncwarp();
                uint32_t cur[32];
                tmem_ld_x32(lane_base + col_o, cur);
#pragma unroll 1
                for (int c32 = 0; c32 < D / 32; ++c32) {
                    tmem_ld_wait();
                    uint32_t w[16];
#pragma unroll
                    for (int k = 0; k < 16; ++k)
                        w[k] = pack16<F16>(__uint_as_float(cur[2 * k]) * inv, __uint_as_float(cur[2 * k + 1]) * inv);
                    if (c32 + 1 < D / 32) tmem_ld_x32(lane_base + col_o + (c32 + 1) * 32, cur);
                    // 32 columns = four 16-byte chunks of this row's 128-byte line in block c32 / 2
                    uint8_t* line = stage_out + (c32 >> 1) * 4096 + lane * 128;
#pragma unroll
                    for (int c = 0; c < 4; ++c)
                        *reinterpret_cast<uint4*>(line + ((((c32 & 1) * 4 + c) ^ (lane & 7)) << 4)) =
                            make_uint4(w[4 * c], w[4 * c + 1], w[4 * c + 2], w[4 * c + 3]);
                }
                // O_t is in shared memory: hand it back to the issuer before the stores go out
                tc_fence_before_sync();
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(&o_free[t]);
                    const int row0 = q0 + quarter * 32;
                    if (row0 < p.Sq) {
#pragma unroll
                        for (int cb = 0; cb < D / 64; ++cb) tma_store_4d(&tmap_o, stage_out + cb * 4096, cb * 64, row0, head, it.b);
                        tma_store_commit();
                    }
                }
            }
            kvbase += two_streams ? nh : it.n_max;
            it = it_next; i_cur = i_next;
        }
        if (lane == 0) tma_store_wait_all<0>();  // every output tile has left shared memory and is written
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

// Element strides of a [B, H, S, D] tensor between batch entries, heads and rows (the D elements of a row are
// contiguous).  Dense tensors have {H * S * D, S * D, D}; the strided entry point passes the caller's.
struct Strides {
    long long b, h, s;
};
inline Strides dense_strides(int H, int S, int D) { return {(long long)H * S * D, (long long)S * D, (long long)D}; }

// D: the kernel's head dimension (64 or 128); head_dim <= D: the tensors' (a multiple of 8).  Columns beyond
// head_dim are zero-filled on load and clipped on store by the TMA unit, so a padded head costs time, not memory.
template <int D, bool F16, bool BIAS = false>
int launch_attn(const void* q, const void* k, const void* v, void* out, int B, int Hq, int Hkv, int Sq, int Skv,
                int head_dim, int mask_kind, const int32_t* lens, float scale, cudaStream_t s, const float* bias = nullptr,
                int bias_heads = 1, const Strides* sq_ = nullptr, const Strides* sk_ = nullptr, const Strides* sv_ = nullptr,
                const Strides* so_ = nullptr) {
    using L = AttnSmem<D>;
    const Strides sq = sq_ ? *sq_ : dense_strides(Hq, Sq, head_dim), so = so_ ? *so_ : dense_strides(Hq, Sq, head_dim);
    const Strides sk = sk_ ? *sk_ : dense_strides(Hkv, Skv, head_dim), sv = sv_ ? *sv_ : dense_strides(Hkv, Skv, head_dim);
    // every tensor as a 4-D map (D, rows, heads, batch): the strides carry the layout
    auto encode = [&](CUtensorMap* m, const void* base, int H, int S, const Strides& st, uint32_t box_rows) {
        const uint32_t box[4] = {64, box_rows, 1, 1};
        const uint64_t dims[4] = {(uint64_t)head_dim, (uint64_t)S, (uint64_t)H, (uint64_t)B};
        const uint64_t strides[3] = {(uint64_t)st.s * 2, (uint64_t)st.h * 2, (uint64_t)st.b * 2};
        return encode_tmap_bf16_sw128(m, base, 4, dims, strides, box);
    };
    CUtensorMap tq, tk, tv, to;
    if (!encode(&tq, q, Hq, Sq, sq, 128)) return FORGE_ERR_CUDA;
    if (!encode(&tk, k, Hkv, Skv, sk, kHalf)) return FORGE_ERR_CUDA;
    if (!encode(&tv, v, Hkv, Skv, sv, kHalf)) return FORGE_ERR_CUDA;
    if (!encode(&to, out, Hq, Sq, so, 32)) return FORGE_ERR_CUDA;  // the output leaves in boxes of 32 rows, one per softmax warp
    AttnParams p;
    p.out = static_cast<uint16_t*>(out);
    p.o_sb = so.b; p.o_sh = so.h; p.o_ss = so.s;
    p.lens = lens;
    p.bias = bias;
    p.bias_heads = bias_heads;
    p.inv_scale = scale > 0.f ? 1.f / scale : 0.f;
    p.head_dim = head_dim;
    p.B = B; p.Hq = Hq; p.Hkv = Hkv; p.Sq = Sq; p.Skv = Skv;
    p.mask_kind = mask_kind;
    p.scale_log2 = scale * 1.4426950408889634f;
    // scale = 0 (uniform weights): any positive multiplier whose products with the scores flush to zero
    if (!(p.scale_log2 > 0.f)) p.scale_log2 = 1.17549435e-38f;
    p.status = device_status_word();
    if (!p.status) return FORGE_ERR_CUDA;
    {
        const int G = Hq / Hkv;
        const bool by_pairs = (G % 2 == 0) || L::kKVStages >= 8;  // same rule as in the kernel
        const int inner = by_pairs ? (Hq + 1) / 2 : Hq;
        p.div_heads = make_fastdiv(inner * B);
        p.div_inner = make_fastdiv(inner);
        p.div_group = make_fastdiv(G);
    }
    auto kernel = attn_bf16_kernel<D, F16, BIAS>;
    FORGE_SET_SMEM_ONCE(kernel, L::kAlloc);
    const int sms = sm_count();
    if (sms <= 0) return FORGE_ERR_CUDA;
    const int q_tiles = (Sq + kBM - 1) / kBM;
    const bool head_pairs = ((Hq / Hkv) % 2 == 0) || L::kKVStages >= 8;  // same rule as in the kernel
    const long long items = head_pairs ? (long long)((Hq + 1) / 2) * B * q_tiles
                                       : (long long)Hq * B * ((q_tiles + 1) / 2);
    const int grid = items < sms ? (int)items : sms;
    FORGE_CUDA_TRY(launch_pdl(kernel, dim3(grid), dim3(kThreads), L::kAlloc, s, tq, tk, tv, to, p));
    return finish_launch(1);
}

// Head sizes above 128 run on the one-tile-per-CTA kernel of attn_wide.cu.
int wide_dense(bool f16, const void* q, const void* k, const void* v, void* out, int B, int Hq, int Hkv, int Sq, int Skv,
               int D, int mask_kind, const int32_t* lens, float scale, cudaStream_t s) {
    const Strides a = dense_strides(Hq, Sq, D), c = dense_strides(Hkv, Skv, D);
    const long long st[4][3] = {{a.b, a.h, a.s}, {c.b, c.h, c.s}, {c.b, c.h, c.s}, {a.b, a.h, a.s}};
    return attn_wide(f16, q, k, v, out, B, Hq, Hkv, Sq, Skv, D, mask_kind, lens, scale, st, s);
}

}  // namespace
}  // namespace forge

extern "C" int forge_attn_fused(const void* q, const void* k, const void* v, void* out,
                                int B, int Hq, int Hkv, int Sq, int Skv, int D,
                                int mask_kind, const int32_t* lens, float scale, void* stream) {
    using namespace forge;
    int st = check_attn_args(q, k, v, out, B, Hq, Hkv, Sq, Skv, D, mask_kind, lens, /*any_head_dim=*/true, 256);
    if (st != FORGE_OK) return st;
    if ((long long)Hq * B * ((Sq + 127) / 128) > 2147483647LL) return FORGE_ERR_UNSUPPORTED;
    if (!(scale >= 0.f)) return FORGE_ERR_UNSUPPORTED;  // the running maximum is taken on unscaled scores
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (D > 128) return wide_dense(false, q, k, v, out, B, Hq, Hkv, Sq, Skv, D, mask_kind, lens, scale, s);
    return D <= 64 ? launch_attn<64, false>(q, k, v, out, B, Hq, Hkv, Sq, Skv, D, mask_kind, lens, scale, s)
                   : launch_attn<128, false>(q, k, v, out, B, Hq, Hkv, Sq, Skv, D, mask_kind, lens, scale, s);
}

extern "C" int forge_attn_fused_f16(const void* q, const void* k, const void* v, void* out,
                                    int B, int Hq, int Hkv, int Sq, int Skv, int D,
                                    int mask_kind, const int32_t* lens, float scale, void* stream) {
    using namespace forge;
    int st = check_attn_args(q, k, v, out, B, Hq, Hkv, Sq, Skv, D, mask_kind, lens, /*any_head_dim=*/true, 256);
    if (st != FORGE_OK) return st;
    if ((long long)Hq * B * ((Sq + 127) / 128) > 2147483647LL) return FORGE_ERR_UNSUPPORTED;
    if (!(scale >= 0.f)) return FORGE_ERR_UNSUPPORTED;  // the running maximum is taken on unscaled scores
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (D > 128) return wide_dense(true, q, k, v, out, B, Hq, Hkv, Sq, Skv, D, mask_kind, lens, scale, s);
    return D <= 64 ? launch_attn<64, true>(q, k, v, out, B, Hq, Hkv, Sq, Skv, D, mask_kind, lens, scale, s)
                   : launch_attn<128, true>(q, k, v, out, B, Hq, Hkv, Sq, Skv, D, mask_kind, lens, scale, s);
}

extern "C" int forge_attn_fused_bias(const void* q, const void* k, const void* v, void* out,
                                     int B, int Hq, int Hkv, int Sq, int Skv, int D,
                                     int mask_kind, const int32_t* lens, const float* bias, int bias_heads,
                                     float scale, void* stream) {
    using namespace forge;
    int st = check_attn_args(q, k, v, out, B, Hq, Hkv, Sq, Skv, D, mask_kind, lens, /*any_head_dim=*/true);
    if (st != FORGE_OK) return st;
    if (!bias || (reinterpret_cast<uintptr_t>(bias) & 15u)) return FORGE_ERR_INVALID_ARG;
    if (bias_heads != 1 && bias_heads != Hq) return FORGE_ERR_INVALID_ARG;
    if ((long long)Hq * B * ((Sq + 255) / 256) > 2147483647LL) return FORGE_ERR_UNSUPPORTED;
    if (!(scale > 0.f)) return FORGE_ERR_UNSUPPORTED;  // the bias enters the kernel as bias / scale
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    return D <= 64 ? launch_attn<64, false, true>(q, k, v, out, B, Hq, Hkv, Sq, Skv, D, mask_kind, lens, scale, s, bias, bias_heads)
                   : launch_attn<128, false, true>(q, k, v, out, B, Hq, Hkv, Sq, Skv, D, mask_kind, lens, scale, s, bias, bias_heads);
}

extern "C" int forge_attn_fused_strided(const void* q, const void* k, const void* v, void* out,
                                        int B, int Hq, int Hkv, int Sq, int Skv, int D,
                                        const int64_t* q_strides, const int64_t* k_strides, const int64_t* v_strides,
                                        const int64_t* out_strides, int mask_kind, const int32_t* lens, float scale,
                                        void* stream) {
    using namespace forge;
    int st = check_attn_args(q, k, v, out, B, Hq, Hkv, Sq, Skv, D, mask_kind, lens, /*any_head_dim=*/true, 256);
    if (st != FORGE_OK) return st;
    if (!q_strides || !k_strides || !v_strides || !out_strides) return FORGE_ERR_INVALID_ARG;
    if ((long long)Hq * B * ((Sq + 127) / 128) > 2147483647LL) return FORGE_ERR_UNSUPPORTED;
    if (!(scale >= 0.f)) return FORGE_ERR_UNSUPPORTED;  // the running maximum is taken on unscaled scores
    Strides str[4];
    const int64_t* in[4] = {q_strides, k_strides, v_strides, out_strides};
    for (int i = 0; i < 4; ++i) {
        str[i] = {in[i][0], in[i][1], in[i][2]};
        // rows must not overlap their own elements, and every stride must keep rows on 16-byte boundaries
        if (str[i].b <= 0 || str[i].h <= 0 || str[i].s < D) return FORGE_ERR_INVALID_ARG;
        if ((str[i].b % 8) || (str[i].h % 8) || (str[i].s % 8)) return FORGE_ERR_UNSUPPORTED;
        if (str[i].b >= (1LL << 38) || str[i].h >= (1LL << 38) || str[i].s >= (1LL << 38)) return FORGE_ERR_UNSUPPORTED;
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (D > 128) {
        long long w[4][3];
        for (int i = 0; i < 4; ++i) { w[i][0] = str[i].b; w[i][1] = str[i].h; w[i][2] = str[i].s; }
        return attn_wide(false, q, k, v, out, B, Hq, Hkv, Sq, Skv, D, mask_kind, lens, scale, w, s);
    }
    return D <= 64 ? launch_attn<64, false>(q, k, v, out, B, Hq, Hkv, Sq, Skv, D, mask_kind, lens, scale, s, nullptr, 1,
                                            &str[0], &str[1], &str[2], &str[3])
                   : launch_attn<128, false>(q, k, v, out, B, Hq, Hkv, Sq, Skv, D, mask_kind, lens, scale, s, nullptr, 1,
                                             &str[0], &str[1], &str[2], &str[3]);
}
